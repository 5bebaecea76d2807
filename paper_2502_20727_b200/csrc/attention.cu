// Attention of each emulated shard over its own heads (Sec. 3).  Shards own contiguous head
// ranges, so one launch over all heads IS the T per-shard attentions side by side; nothing
// crosses a shard boundary here.  K and V are always read from the paged cache.
#include "common.cuh"
#include "tc_ptx.cuh"
#include "trace.cuh"

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
    pdl_launch_dependents();
    pdl_wait();
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
    case 128: return launch_kernel(prefill_attention_kernel<T, 4>, grid, dim3(128), 0, st, 0, a);
    case 64: return launch_kernel(prefill_attention_kernel<T, 2>, grid, dim3(128), 0, st, 0, a);
    case 32: return launch_kernel(prefill_attention_kernel<T, 1>, grid, dim3(128), 0, st, 0, a);
    default: return cudaErrorInvalidValue;
    }
}
template cudaError_t launch_prefill_attention<float>(const AttnArgs &, cudaStream_t);
template cudaError_t launch_prefill_attention<bf16>(const AttnArgs &, cudaStream_t);

// ---------------------------------------------------------------------------------------
// Paged decode attention: one query token per sequence.
// grid (n_q_heads / GT, B, splits).  A CTA serves GT query heads that share one KV head
// (grouped-query attention reads each K/V row once for the whole tile) over one slice of the
// context.  Every K/V row is fetched with 16-byte loads, LPT = row_bytes / 16 lanes per token,
// so a warp instruction covers TPW = 32 / LPT whole rows; NG such instructions per operand are
// issued back to back before any arithmetic.  Scores are reduced with warp shuffles, the
// softmax is the online form per token slot, slots / warps / splits are merged at the end
// (the last CTA of a (sequence, head tile) to finish merges the splits, in a fixed order).
template <typename T> struct Row16;
template <> struct Row16<float> {
    static constexpr int E = 4;
    static __device__ __forceinline__ void cvt(const uint4 &u, float *o)
    { o[0] = __uint_as_float(u.x); o[1] = __uint_as_float(u.y); o[2] = __uint_as_float(u.z); o[3] = __uint_as_float(u.w); }
};
template <> struct Row16<bf16> {
    static constexpr int E = 8;
    static __device__ __forceinline__ void cvt(const uint4 &u, float *o)
    {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { o[2 * i] = __uint_as_float(w[i] << 16); o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
    }
};

// Ring of the bulk-copy decode kernel: K and V page per slot, 32 KB in all (measured better than
// 64 KB: four thread blocks per SM keep every block of a step resident at once).
template <typename T, int D> struct DecodeRing {
    static constexpr int PAGE_BYTES = 16 * D * (int)sizeof(T);
    static constexpr int SLOTS = (32 * 1024) / (2 * PAGE_BYTES) > 16 ? 16 : (32 * 1024) / (2 * PAGE_BYTES);
};

template <typename T, int D, int GT>
__global__ void __launch_bounds__(128) decode_attention_kernel(AttnArgs a)
{
    pdl_launch_dependents();
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_START);
    pdl_wait();
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_DEP_DONE);
    constexpr int E = Row16<T>::E, LPT = D / E, TPW = 32 / LPT, NG = 8, CHUNK = NG * TPW;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int slot = lane / LPT, li = lane % LPT;
    const int hq0 = blockIdx.x * GT, b = blockIdx.y, sp = blockIdx.z;
    const int kvh = hq0 / (a.n_q_heads / a.pt.n_kv_heads);
    __shared__ float sm_o[4][GT][D];
    __shared__ float sm_ml[4][GT][2];
    __shared__ int sm_last;

    const int ctx = a.tm.seq_lens[b] + 1;
    const bool bad = ctx < 1 || ctx > a.max_context || (ctx - 1) / a.pt.block >= a.pt.max_pages;
    int per = (a.max_context + a.splits - 1) / a.splits;
    per = (per + CHUNK - 1) / CHUNK * CHUNK;
    const int t0 = sp * per, t1 = bad ? t0 : min(ctx, t0 + per);
    if (bad && threadIdx.x == 0) atomicOr(a.err, ERR_CAPACITY);

    // query tile, pre-scaled so that the softmax can use exp2
    float q[GT][E];
    {
        const float sc = rsqrtf((float)D) * 1.4426950408889634f;
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            const T *qp = (const T *)a.q + ((long)b * a.n_q_heads + hq0 + g) * D + li * E;
            uint4 u = *(const uint4 *)qp;
            Row16<T>::cvt(u, q[g]);
#pragma unroll
            for (int e = 0; e < E; ++e) q[g][e] *= sc;
        }
    }
    float mx[GT], den[GT], o[GT][E];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        mx[g] = -INFINITY; den[g] = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) o[g][e] = 0.f;
    }
    const T *kp = (const T *)a.k_pages, *vp = (const T *)a.v_pages;
    for (int c0 = t0 + warp * CHUNK; c0 < t1; c0 += 4 * CHUNK) {
        uint4 kr[NG], vr[NG];
        bool valid[NG];
#pragma unroll
        for (int i = 0; i < NG; ++i) {
            const int t = c0 + i * TPW + slot;
            valid[i] = t < t1;
            kr[i] = make_uint4(0, 0, 0, 0);
            vr[i] = make_uint4(0, 0, 0, 0);
            if (valid[i]) {
                int page = a.pt.block_table[(long)b * a.pt.max_pages + t / a.pt.block];
                if (page < 0 || page >= a.pt.n_pages) { atomicOr(a.err, ERR_PAGE_RANGE); page = 0; }
                const long row = (((long)page * a.pt.n_kv_heads + kvh) * a.pt.block + t % a.pt.block) * D + li * E;
                kr[i] = *(const uint4 *)(kp + row);
                vr[i] = *(const uint4 *)(vp + row);
            }
        }
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            float s[NG], cmax = -INFINITY;
#pragma unroll
            for (int i = 0; i < NG; ++i) {
                float kf[E], acc = 0.f;
                Row16<T>::cvt(kr[i], kf);
#pragma unroll
                for (int e = 0; e < E; ++e) acc = fmaf(q[g][e], kf[e], acc);
#pragma unroll
                for (int off = LPT / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                s[i] = valid[i] ? acc : -INFINITY;
                cmax = fmaxf(cmax, s[i]);
            }
            const float nm = fmaxf(mx[g], cmax);
            if (nm == -INFINITY) continue; // nothing valid in this slot so far
            const float corr = exp2f(mx[g] - nm);
            mx[g] = nm;
            den[g] *= corr;
#pragma unroll
            for (int e = 0; e < E; ++e) o[g][e] *= corr;
#pragma unroll
            for (int i = 0; i < NG; ++i) {
                const float p = exp2f(s[i] - nm); // 0 for masked tokens
                den[g] += p;
                float vf[E];
                Row16<T>::cvt(vr[i], vf);
#pragma unroll
                for (int e = 0; e < E; ++e) o[g][e] = fmaf(p, vf[e], o[g][e]);
            }
        }
    }
    // merge the token slots of the warp
#pragma unroll
    for (int off = LPT; off < 32; off <<= 1) {
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            const float om = __shfl_xor_sync(0xffffffffu, mx[g], off), od = __shfl_xor_sync(0xffffffffu, den[g], off);
            const float nm = fmaxf(mx[g], om);
            const float ca = (mx[g] == -INFINITY) ? 0.f : exp2f(mx[g] - nm), cb = (om == -INFINITY) ? 0.f : exp2f(om - nm);
            den[g] = den[g] * ca + od * cb;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const float oo = __shfl_xor_sync(0xffffffffu, o[g][e], off);
                o[g][e] = o[g][e] * ca + oo * cb;
            }
            mx[g] = nm;
        }
    }
    if (slot == 0) {
#pragma unroll
        for (int g = 0; g < GT; ++g) {
#pragma unroll
            for (int e = 0; e < E; ++e) sm_o[warp][g][li * E + e] = o[g][e];
            if (li == 0) { sm_ml[warp][g][0] = mx[g]; sm_ml[warp][g][1] = den[g]; }
        }
    }
    __syncthreads();
    // merge the 4 warps; thread -> (head of the tile, dim)
    const long pbase = ((long)b * a.n_q_heads + hq0) * a.splits + sp;
    for (int idx = threadIdx.x; idx < GT * D; idx += blockDim.x) {
        const int g = idx / D, dd = idx % D;
        float gm = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) gm = fmaxf(gm, sm_ml[w][g][0]);
        float acc = 0.f, gden = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float c = (sm_ml[w][g][0] == -INFINITY) ? 0.f : exp2f(sm_ml[w][g][0] - gm);
            acc += sm_o[w][g][dd] * c;
            gden += sm_ml[w][g][1] * c;
        }
        if (a.splits == 1) {
            ((T *)a.out)[((long)b * a.n_q_heads + hq0 + g) * D + dd] = from_f<T>(gden > 0.f ? acc / gden : 0.f);
        } else {
            const long pi = pbase + (long)g * a.splits;
            a.part_o[pi * D + dd] = acc; // un-normalised
            if (dd == 0) { a.part_ml[pi * 2] = gm; a.part_ml[pi * 2 + 1] = gden; }
        }
    }
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_MAIN_DONE);
    if (a.splits == 1) return;
    // the last CTA of this (sequence, head tile) to arrive merges the splits
    __threadfence();
    __syncthreads();
    int *cnt = a.counters + (long)b * gridDim.x + blockIdx.x;
    if (threadIdx.x == 0) sm_last = (atomicAdd(cnt, 1) == a.splits - 1);
    __syncthreads();
    if (!sm_last) return;
    __threadfence();
    for (int idx = threadIdx.x; idx < GT * D; idx += blockDim.x) {
        const int g = idx / D, dd = idx % D;
        const long p0 = ((long)b * a.n_q_heads + hq0 + g) * a.splits;
        float gm = -INFINITY;
        for (int s2 = 0; s2 < a.splits; ++s2) gm = fmaxf(gm, __ldcg(a.part_ml + (p0 + s2) * 2));
        float acc = 0.f, gden = 0.f;
        for (int s2 = 0; s2 < a.splits; ++s2) {
            const float m2 = __ldcg(a.part_ml + (p0 + s2) * 2);
            const float c = (m2 == -INFINITY) ? 0.f : exp2f(m2 - gm);
            acc += __ldcg(a.part_o + (p0 + s2) * D + dd) * c;
            gden += __ldcg(a.part_ml + (p0 + s2) * 2 + 1) * c;
        }
        ((T *)a.out)[((long)b * a.n_q_heads + hq0 + g) * D + dd] = from_f<T>(gden > 0.f ? acc / gden : 0.f);
    }
    if (threadIdx.x == 0) *cnt = 0; // ready for the next launch
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_END);
}

// ---------------------------------------------------------------------------------------
// Paged decode attention fed by bulk copies.  With 16-token pages the K (and V) rows of one
// (page, kv head) are one contiguous block, so a producer warp streams whole pages into a
// shared-memory ring with cp.async.bulk (completion on an mbarrier) and the four compute
// warps take pages round-robin; a page is released back to the producer by the warp that
// read it.  Every page of the thread block's range is requested as early as the ring allows,
// independent of the arithmetic, and pages that hold only earlier steps' tokens are requested
// before the dependency wait (only the page receiving this step's token is written by the
// preceding kernel).  grid (n_q_heads / GT, B, splits); GT query heads share the KV head.
template <typename T, int D, int GT>
__global__ void __launch_bounds__(160) decode_attention_ring_kernel(AttnArgs a)
{
    using namespace tc;
    constexpr int E = Row16<T>::E, LPT = D / E, TPW = 32 / LPT, BLK = 16, NG = BLK / TPW;
    constexpr int PAGE_BYTES = BLK * D * (int)sizeof(T);
    constexpr int R = DecodeRing<T, D>::SLOTS;
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t *ring = smem;
    float(*sm_o)[GT][D] = (float(*)[GT][D])(smem + R * 2 * PAGE_BYTES);
    float(*sm_ml)[GT][2] = (float(*)[GT][2])(smem + R * 2 * PAGE_BYTES + 4 * GT * D * 4);
    uint8_t *tail = smem + R * 2 * PAGE_BYTES + 4 * GT * D * 4 + 4 * GT * 2 * 4;
    const uint32_t bars = smem_u32(tail);             // full[R], empty[R]
    int *sm_bt = (int *)(tail + 2 * R * 8);           // pages of this block's range
    volatile int *abort_flag = (volatile int *)(sm_bt + DECODE_MAX_PAGES_PER_BLOCK);
    int *sm_last = (int *)(sm_bt + DECODE_MAX_PAGES_PER_BLOCK + 1);
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (R + s); };

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hq0 = blockIdx.x * GT, b = blockIdx.y, sp = blockIdx.z;
    const int kvh = hq0 / (a.n_q_heads / a.pt.n_kv_heads);

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        SPD_TRACE_EVENT(TRK_ATTN, TR_START);
        for (int s = 0; s < R; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // seq_lens and the block table are written before the step starts, never by its kernels
    const int ctx = a.tm.seq_lens[b] + 1;
    const bool bad = ctx < 1 || ctx > a.max_context || (ctx - 1) / BLK >= a.pt.max_pages;
    const int pages_bucket = (a.max_context + BLK - 1) / BLK;
    const int per = (pages_bucket + a.splits - 1) / a.splits;   // pages per split (<= DECODE_MAX_PAGES_PER_BLOCK)
    const int p0 = sp * per;
    const int ctx_pages = bad ? 0 : (ctx + BLK - 1) / BLK;
    const int n_pages = max(0, min(ctx_pages, p0 + per) - p0);
    const int new_page = (ctx - 1) / BLK;                        // the page this step's token lands in
    if (bad && threadIdx.x == 0) atomicOr(a.err, ERR_CAPACITY);

    if (warp == 4) {
        // producer
        for (int i = lane; i < n_pages; i += 32) {
            int page = a.pt.block_table[(long)b * a.pt.max_pages + p0 + i];
            if (page < 0 || page >= a.pt.n_pages) { atomicOr(a.err, ERR_PAGE_RANGE); page = 0; }
            sm_bt[i] = page;
        }
        __syncwarp();
        if (lane == 0) {
            const T *kp = (const T *)a.k_pages, *vp = (const T *)a.v_pages;
            bool waited = false;
            for (int i = 0; i < n_pages; ++i) {
                const int s = i % R;
                if (!waited && p0 + i >= new_page) { pdl_wait(); waited = true; }
                if (i >= R && !mbar_wait(empty_bar(s), ((i / R) & 1) ^ 1, a.err, abort_flag)) break;
                const long off = ((long)sm_bt[i] * a.pt.n_kv_heads + kvh) * (BLK * D);
                const uint32_t dst = smem_u32(ring + s * 2 * PAGE_BYTES);
                mbar_expect_tx(full_bar(s), 2 * PAGE_BYTES);
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(dst), "l"(kp + off), "r"(PAGE_BYTES), "r"(full_bar(s)) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(dst + PAGE_BYTES), "l"(vp + off), "r"(PAGE_BYTES), "r"(full_bar(s)) : "memory");
            }
        }
        __syncwarp();
    }
    pdl_wait(); // q comes from the preceding kernel
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_DEP_DONE);

    float mx[GT], den[GT], o[GT][E];
    const int slot = lane / LPT, li = lane % LPT;
    if (warp < 4) {
        // query tile, pre-scaled so that the softmax can use exp2
        float q[GT][E];
        {
            const float sc = rsqrtf((float)D) * 1.4426950408889634f;
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                const T *qp = (const T *)a.q + ((long)b * a.n_q_heads + hq0 + g) * D + li * E;
                uint4 u = *(const uint4 *)qp;
                Row16<T>::cvt(u, q[g]);
#pragma unroll
                for (int e = 0; e < E; ++e) q[g][e] *= sc;
            }
        }
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            mx[g] = -INFINITY; den[g] = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) o[g][e] = 0.f;
        }
        for (int pi = warp; pi < n_pages; pi += 4) {
            const int s = pi % R;
            if (!mbar_wait(full_bar(s), (pi / R) & 1, a.err, abort_flag)) break;
            const uint8_t *kb = ring + s * 2 * PAGE_BYTES, *vb = kb + PAGE_BYTES;
            const int tbase = (p0 + pi) * BLK;
            uint4 kr[NG], vr[NG];
            bool valid[NG];
#pragma unroll
            for (int i = 0; i < NG; ++i) {
                const int tl = i * TPW + slot;
                valid[i] = tbase + tl < ctx;
                kr[i] = *(const uint4 *)(kb + ((long)tl * D + li * E) * sizeof(T));
                vr[i] = *(const uint4 *)(vb + ((long)tl * D + li * E) * sizeof(T));
            }
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(s)) : "memory");
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                float sc[NG], cmax = -INFINITY;
#pragma unroll
                for (int i = 0; i < NG; ++i) {
                    float kf[E], acc = 0.f;
                    Row16<T>::cvt(kr[i], kf);
#pragma unroll
                    for (int e = 0; e < E; ++e) acc = fmaf(q[g][e], kf[e], acc);
#pragma unroll
                    for (int off = LPT / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                    sc[i] = valid[i] ? acc : -INFINITY;
                    cmax = fmaxf(cmax, sc[i]);
                }
                const float nm = fmaxf(mx[g], cmax);
                if (nm == -INFINITY) continue; // nothing valid in this slot so far
                const float corr = exp2f(mx[g] - nm);
                mx[g] = nm;
                den[g] *= corr;
#pragma unroll
                for (int e = 0; e < E; ++e) o[g][e] *= corr;
#pragma unroll
                for (int i = 0; i < NG; ++i) {
                    const float p = exp2f(sc[i] - nm); // 0 for masked tokens
                    den[g] += p;
                    float vf[E];
                    Row16<T>::cvt(vr[i], vf);
#pragma unroll
                    for (int e = 0; e < E; ++e) o[g][e] = fmaf(p, vf[e], o[g][e]);
                }
            }
        }
        // merge the token slots of the warp
#pragma unroll
        for (int off = LPT; off < 32; off <<= 1) {
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                const float om = __shfl_xor_sync(0xffffffffu, mx[g], off), od = __shfl_xor_sync(0xffffffffu, den[g], off);
                const float nm = fmaxf(mx[g], om);
                const float ca = (mx[g] == -INFINITY) ? 0.f : exp2f(mx[g] - nm), cb = (om == -INFINITY) ? 0.f : exp2f(om - nm);
                den[g] = den[g] * ca + od * cb;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const float oo = __shfl_xor_sync(0xffffffffu, o[g][e], off);
                    o[g][e] = o[g][e] * ca + oo * cb;
                }
                mx[g] = nm;
            }
        }
        if (slot == 0) {
#pragma unroll
            for (int g = 0; g < GT; ++g) {
#pragma unroll
                for (int e = 0; e < E; ++e) sm_o[warp][g][li * E + e] = o[g][e];
                if (li == 0) { sm_ml[warp][g][0] = mx[g]; sm_ml[warp][g][1] = den[g]; }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_MAIN_DONE);
    // merge the 4 warps; thread -> (head of the tile, dim)
    const long pbase = ((long)b * a.n_q_heads + hq0) * a.splits + sp;
    for (int idx = threadIdx.x; idx < GT * D; idx += blockDim.x) {
        const int g = idx / D, dd = idx % D;
        float gm = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) gm = fmaxf(gm, sm_ml[w][g][0]);
        float acc = 0.f, gden = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float c = (sm_ml[w][g][0] == -INFINITY) ? 0.f : exp2f(sm_ml[w][g][0] - gm);
            acc += sm_o[w][g][dd] * c;
            gden += sm_ml[w][g][1] * c;
        }
        if (a.splits == 1) {
            ((T *)a.out)[((long)b * a.n_q_heads + hq0 + g) * D + dd] = from_f<T>(gden > 0.f ? acc / gden : 0.f);
        } else {
            const long pi = pbase + (long)g * a.splits;
            a.part_o[pi * D + dd] = acc; // un-normalised
            if (dd == 0) { a.part_ml[pi * 2] = gm; a.part_ml[pi * 2 + 1] = gden; }
        }
    }
    if (a.splits == 1) return;
    // the last block of this (sequence, head tile) to arrive merges the splits
    __threadfence();
    __syncthreads();
    int *cnt = a.counters + (long)b * gridDim.x + blockIdx.x;
    if (threadIdx.x == 0) *sm_last = (atomicAdd(cnt, 1) == a.splits - 1);
    __syncthreads();
    if (!*sm_last) return;
    __threadfence();
    for (int idx = threadIdx.x; idx < GT * D; idx += blockDim.x) {
        const int g = idx / D, dd = idx % D;
        const long q0 = ((long)b * a.n_q_heads + hq0 + g) * a.splits;
        float gm = -INFINITY;
        for (int s2 = 0; s2 < a.splits; ++s2) gm = fmaxf(gm, __ldcg(a.part_ml + (q0 + s2) * 2));
        float acc = 0.f, gden = 0.f;
        for (int s2 = 0; s2 < a.splits; ++s2) {
            const float m2 = __ldcg(a.part_ml + (q0 + s2) * 2);
            const float c = (m2 == -INFINITY) ? 0.f : exp2f(m2 - gm);
            acc += __ldcg(a.part_o + (q0 + s2) * D + dd) * c;
            gden += __ldcg(a.part_ml + (q0 + s2) * 2 + 1) * c;
        }
        ((T *)a.out)[((long)b * a.n_q_heads + hq0 + g) * D + dd] = from_f<T>(gden > 0.f ? acc / gden : 0.f);
    }
    if (threadIdx.x == 0) *cnt = 0; // ready for the next launch
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_END);
}

template <typename T, int D, int GT> cudaError_t launch_ring(const AttnArgs &a, cudaStream_t st)
{
    constexpr int PAGE_BYTES = 16 * D * (int)sizeof(T), R = DecodeRing<T, D>::SLOTS;
    constexpr int SMEM = R * 2 * PAGE_BYTES + 4 * GT * D * 4 + 4 * GT * 2 * 4 + 2 * R * 8 + (DECODE_MAX_PAGES_PER_BLOCK + 2) * 4;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(decode_attention_ring_kernel<T, D, GT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        // ask for the largest shared-memory carve-out so that four blocks fit an SM
        e = cudaFuncSetAttribute(decode_attention_ring_kernel<T, D, GT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    dim3 grid(a.n_q_heads / GT, a.B, a.splits);
    return launch_kernel(decode_attention_ring_kernel<T, D, GT>, grid, dim3(160), SMEM, st, 0, a);
}

template <typename T, int D> cudaError_t launch_decode_d(const AttnArgs &a, cudaStream_t st)
{
    const int group = a.n_q_heads / a.pt.n_kv_heads;
    const int pages_bucket = (a.max_context + 15) / 16;
    if (a.pt.block == 16 && (pages_bucket + a.splits - 1) / a.splits <= DECODE_MAX_PAGES_PER_BLOCK) {
        switch (decode_heads_per_block(group)) {
        case 4: return launch_ring<T, D, 4>(a, st);
        case 2: return launch_ring<T, D, 2>(a, st);
        default: return launch_ring<T, D, 1>(a, st);
        }
    }
    const int gt = (group % 4 == 0) ? 4 : ((group % 2 == 0) ? 2 : 1);
    dim3 grid(a.n_q_heads / gt, a.B, a.splits);
    if (gt == 4) return launch_kernel(decode_attention_kernel<T, D, 4>, grid, dim3(128), 0, st, 0, a);
    if (gt == 2) return launch_kernel(decode_attention_kernel<T, D, 2>, grid, dim3(128), 0, st, 0, a);
    return launch_kernel(decode_attention_kernel<T, D, 1>, grid, dim3(128), 0, st, 0, a);
}

template <typename T> cudaError_t launch_decode_attention(const AttnArgs &a, cudaStream_t st)
{
    if (a.B <= 0) return cudaSuccess;
    switch (a.head_dim) {
    case 128: return launch_decode_d<T, 128>(a, st);
    case 64: return launch_decode_d<T, 64>(a, st);
    case 32: return launch_decode_d<T, 32>(a, st);
    default: return cudaErrorInvalidValue;
    }
}
template cudaError_t launch_decode_attention<float>(const AttnArgs &, cudaStream_t);
template cudaError_t launch_decode_attention<bf16>(const AttnArgs &, cudaStream_t);

} // namespace spd
