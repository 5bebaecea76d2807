// Attention of each emulated shard over its own heads (Sec. 3).  Shards own contiguous head
// ranges, so one launch over all heads IS the T per-shard attentions side by side; nothing
// crosses a shard boundary here.  K and V are always read from the paged cache.
#include "common.cuh"

namespace spd {

// 16-byte-or-less vector load of VEC consecutive elements into floats.
template <typename T, int VEC> struct VecLoad;
template <> struct VecLoad<float, 4> {
    static __device__ __forceinline__ void ld(const float *p, float *o)
    { float4 v = *(const float4 *)p; o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
};
template <> struct VecLoad<float, 2> {
    static __device__ __forceinline__ void ld(const float *p, float *o)
    { float2 v = *(const float2 *)p; o[0] = v.x; o[1] = v.y; }
};
template <> struct VecLoad<float, 1> {
    static __device__ __forceinline__ void ld(const float *p, float *o) { o[0] = *p; }
};
template <> struct VecLoad<bf16, 4> {
    static __device__ __forceinline__ void ld(const bf16 *p, float *o)
    {
        uint2 v = *(const uint2 *)p;
        float2 a = __bfloat1622float2(*(const __nv_bfloat162 *)&v.x), b = __bfloat1622float2(*(const __nv_bfloat162 *)&v.y);
        o[0] = a.x; o[1] = a.y; o[2] = b.x; o[3] = b.y;
    }
};
template <> struct VecLoad<bf16, 2> {
    static __device__ __forceinline__ void ld(const bf16 *p, float *o)
    { float2 a = __bfloat1622float2(*(const __nv_bfloat162 *)p); o[0] = a.x; o[1] = a.y; }
};
template <> struct VecLoad<bf16, 1> {
    static __device__ __forceinline__ void ld(const bf16 *p, float *o) { o[0] = __bfloat162float(*p); }
};

__device__ __forceinline__ long page_row(const PageTable &pt, int b, int kvh, int t, int d, int *err)
{
    int page = pt.block_table[(long)b * pt.max_pages + t / pt.block];
    if (page < 0 || page >= pt.n_pages) { atomicOr(err, ERR_PAGE_RANGE); page = 0; }
    return (((long)page * pt.n_kv_heads + kvh) * pt.block + t % pt.block) * d;
}

// One warp per (query token, query head); lane l owns dims [l*VEC, (l+1)*VEC), d = 32*VEC.
// Online softmax over cache positions [t_begin, t_end).
template <typename T, int VEC>
__device__ __forceinline__ void attend_range(const float *q, const T *kp, const T *vp, const PageTable &pt,
                                             int b, int kvh, int t_begin, int t_end, float scale,
                                             float &mx, float &den, float *o, int *err)
{
    const int d = 32 * VEC, lane = threadIdx.x & 31;
    for (int t = t_begin; t < t_end; ++t) {
        long row = page_row(pt, b, kvh, t, d, err) + lane * VEC;
        float kf[VEC], vf[VEC];
        VecLoad<T, VEC>::ld(kp + row, kf);
        VecLoad<T, VEC>::ld(vp + row, vf);
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < VEC; ++i) s = fmaf(q[i], kf[i], s);
        s = warp_sum(s) * scale;
        float nm = fmaxf(mx, s);
        float corr = __expf(mx - nm), p = __expf(s - nm);
        den = den * corr + p;
#pragma unroll
        for (int i = 0; i < VEC; ++i) o[i] = fmaf(o[i], corr, p * vf[i]);
        mx = nm;
    }
}

template <typename T, int VEC>
__global__ void __launch_bounds__(128) prefill_attention_kernel(AttnArgs a)
{
    const int d = 32 * VEC, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int m = blockIdx.x * 4 + warp, hq = blockIdx.y;
    if (m >= a.M) return;
    int b, pos;
    a.tm.locate(m, b, pos);
    if (pos < 0 || pos / a.pt.block >= a.pt.max_pages) { if (lane == 0) atomicOr(a.err, ERR_CAPACITY); return; }
    const int kvh = hq / (a.n_q_heads / a.pt.n_kv_heads);
    float q[VEC], o[VEC];
    VecLoad<T, VEC>::ld((const T *)a.q + ((long)m * a.n_q_heads + hq) * d + lane * VEC, q);
#pragma unroll
    for (int i = 0; i < VEC; ++i) o[i] = 0.f;
    float mx = -INFINITY, den = 0.f;
    attend_range<T, VEC>(q, (const T *)a.k_pages, (const T *)a.v_pages, a.pt, b, kvh, 0, pos + 1,
                         rsqrtf((float)d), mx, den, o, a.err);
    T *out = (T *)a.out + ((long)m * a.n_q_heads + hq) * d + lane * VEC;
    float inv = 1.f / den;
#pragma unroll
    for (int i = 0; i < VEC; ++i) out[i] = from_f<T>(o[i] * inv);
}

template <typename T> cudaError_t launch_prefill_attention(const AttnArgs &a, cudaStream_t st)
{
    if (a.M <= 0) return cudaSuccess;
    dim3 grid((a.M + 3) / 4, a.n_q_heads);
    switch (a.head_dim) {
    case 128: prefill_attention_kernel<T, 4><<<grid, 128, 0, st>>>(a); break;
    case 64: prefill_attention_kernel<T, 2><<<grid, 128, 0, st>>>(a); break;
    case 32: prefill_attention_kernel<T, 1><<<grid, 128, 0, st>>>(a); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}
template cudaError_t launch_prefill_attention<float>(const AttnArgs &, cudaStream_t);
template cudaError_t launch_prefill_attention<bf16>(const AttnArgs &, cudaStream_t);

// Decode: grid (n_q_heads, B, splits); the 4 warps of a CTA interleave the tokens of the
// split's range, then merge through shared memory; splits are merged by the next kernel.
template <typename T, int VEC>
__global__ void __launch_bounds__(128) decode_attention_kernel(AttnArgs a)
{
    const int d = 32 * VEC, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hq = blockIdx.x, b = blockIdx.y, sp = blockIdx.z;
    __shared__ float sm_o[4][32 * VEC];
    __shared__ float sm_ml[4][2];
    const int ctx = a.tm.seq_lens[b] + 1;
    float *po = a.part_o + (((long)b * a.n_q_heads + hq) * a.splits + sp) * d;
    float *pml = a.part_ml + (((long)b * a.n_q_heads + hq) * a.splits + sp) * 2;
    const bool bad = ctx > a.max_context || (ctx - 1) / a.pt.block >= a.pt.max_pages || ctx < 1;
    // tokens per split, rounded to whole pages
    int per = (a.max_context + a.splits - 1) / a.splits;
    per = (per + a.pt.block - 1) / a.pt.block * a.pt.block;
    const int t0 = sp * per, t1 = min(ctx, t0 + per);
    if (bad || t0 >= t1) {
        if (bad && threadIdx.x == 0) atomicOr(a.err, ERR_CAPACITY);
        for (int i = threadIdx.x; i < d; i += blockDim.x) po[i] = 0.f;
        if (threadIdx.x == 0) { pml[0] = -INFINITY; pml[1] = 0.f; }
        return;
    }
    const int kvh = hq / (a.n_q_heads / a.pt.n_kv_heads);
    float q[VEC], o[VEC];
    VecLoad<T, VEC>::ld((const T *)a.q + ((long)b * a.n_q_heads + hq) * d + lane * VEC, q);
#pragma unroll
    for (int i = 0; i < VEC; ++i) o[i] = 0.f;
    float mx = -INFINITY, den = 0.f;
    const float scale = rsqrtf((float)d);
    // warp w takes pages w, w+4, ... of the range
    for (int p0 = t0 + warp * a.pt.block; p0 < t1; p0 += 4 * a.pt.block)
        attend_range<T, VEC>(q, (const T *)a.k_pages, (const T *)a.v_pages, a.pt, b, kvh, p0,
                             min(t1, p0 + a.pt.block), scale, mx, den, o, a.err);
#pragma unroll
    for (int i = 0; i < VEC; ++i) sm_o[warp][lane * VEC + i] = o[i];
    if (lane == 0) { sm_ml[warp][0] = mx; sm_ml[warp][1] = den; }
    __syncthreads();
    float gm = fmaxf(fmaxf(sm_ml[0][0], sm_ml[1][0]), fmaxf(sm_ml[2][0], sm_ml[3][0]));
    float gden = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) gden += sm_ml[w][1] * ((sm_ml[w][0] == -INFINITY) ? 0.f : __expf(sm_ml[w][0] - gm));
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) acc += sm_o[w][i] * ((sm_ml[w][0] == -INFINITY) ? 0.f : __expf(sm_ml[w][0] - gm));
        po[i] = acc; // un-normalised
    }
    if (threadIdx.x == 0) { pml[0] = gm; pml[1] = gden; }
}

// grid (n_q_heads, B): combine the splits' (max, denominator, numerator) triples.
template <typename T> __global__ void decode_merge_kernel(AttnArgs a)
{
    const int hq = blockIdx.x, b = blockIdx.y, d = a.head_dim;
    const float *po = a.part_o + (((long)b * a.n_q_heads + hq) * a.splits) * d;
    const float *pml = a.part_ml + (((long)b * a.n_q_heads + hq) * a.splits) * 2;
    float gm = -INFINITY;
    for (int s = 0; s < a.splits; ++s) gm = fmaxf(gm, pml[2 * s]);
    float den = 0.f;
    for (int s = 0; s < a.splits; ++s)
        if (pml[2 * s] != -INFINITY) den += pml[2 * s + 1] * __expf(pml[2 * s] - gm);
    T *out = (T *)a.out + ((long)b * a.n_q_heads + hq) * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < a.splits; ++s)
            if (pml[2 * s] != -INFINITY) acc += po[(long)s * d + i] * __expf(pml[2 * s] - gm);
        out[i] = from_f<T>(den > 0.f ? acc / den : 0.f);
    }
}

template <typename T> cudaError_t launch_decode_attention(const AttnArgs &a, cudaStream_t st)
{
    if (a.B <= 0) return cudaSuccess;
    dim3 grid(a.n_q_heads, a.B, a.splits);
    switch (a.head_dim) {
    case 128: decode_attention_kernel<T, 4><<<grid, 128, 0, st>>>(a); break;
    case 64: decode_attention_kernel<T, 2><<<grid, 128, 0, st>>>(a); break;
    case 32: decode_attention_kernel<T, 1><<<grid, 128, 0, st>>>(a); break;
    default: return cudaErrorInvalidValue;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    decode_merge_kernel<T><<<dim3(a.n_q_heads, a.B), a.head_dim >= 64 ? 64 : 32, 0, st>>>(a);
    return cudaGetLastError();
}
template cudaError_t launch_decode_attention<float>(const AttnArgs &, cudaStream_t);
template cudaError_t launch_decode_attention<bf16>(const AttnArgs &, cudaStream_t);

} // namespace spd
