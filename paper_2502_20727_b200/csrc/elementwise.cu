// Row-wise kernels between the GEMMs: the residual adds and RMSNorms of the TP and SPD
// blocks (Sec. 3; Sec. 4.1.1: MLP input X + Y_i per shard, output X + sum_i (Y_i + Z_i)),
// the rotary embedding + KV-page append, and SwiGLU.
#include "common.cuh"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace spd {

constexpr int MAX_T = 8;

__device__ __forceinline__ float block_sum(float v, float *red)
{
    v = warp_sum(v);
    int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = (l < nw) ? red[l] : 0.f;
    return warp_sum(t);
}

template <typename T> __device__ __forceinline__ float4 load4(const T *p);
template <> __device__ __forceinline__ float4 load4<float>(const float *p) { return *(const float4 *)p; }
template <> __device__ __forceinline__ float4 load4<bf16>(const bf16 *p)
{
    uint2 v = *(const uint2 *)p;
    float2 a = __bfloat1622float2(*(const __nv_bfloat162 *)&v.x), b = __bfloat1622float2(*(const __nv_bfloat162 *)&v.y);
    return make_float4(a.x, a.y, b.x, b.y);
}
template <typename T> __device__ __forceinline__ void store4(T *p, float4 v);
template <> __device__ __forceinline__ void store4<float>(float *p, float4 v) { *(float4 *)p = v; }
template <> __device__ __forceinline__ void store4<bf16>(bf16 *p, float4 v)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *(uint32_t *)&a;
    u.y = *(uint32_t *)&b;
    *(uint2 *)p = u;
}

__device__ __forceinline__ float4 f4add(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }

__device__ __forceinline__ float4 group_sum4(const NormArgs &a, int g, long idx)
{
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.part)
        for (int p = 0; p < a.per_group; ++p)
            acc = f4add(acc, *(const float4 *)(a.part + (long)(g * a.per_group + p) * a.part_stride + idx));
    return acc;
}

// One CTA per token row; float4 column chunks.
//   res_out  = base + sum over ALL partial planes   (base = x_in or res_in; res_out != res_in)
//   h_out[g] = rmsnorm(base + sum of group g's planes) * gain
// n_groups == 1 is the synchronous block's "all-reduce, residual add, norm"; n_groups == T is
// the SPD block, where shard g only ever sees its own partial attention output Y_g while the
// residual carried to the block output still collects every Y_g.  The second pass re-reads the
// planes (cache resident) instead of holding T x hidden values in registers.
template <typename T>
__global__ void __launch_bounds__(512) residual_norm_kernel(NormArgs a)
{
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float red[32];
    const int m = blockIdx.x, H = a.H, G = a.n_groups, H4 = H >> 2;
    const bool ln = a.shift != nullptr;
    float ss[MAX_T], sm[MAX_T];
#pragma unroll
    for (int g = 0; g < MAX_T; ++g) { ss[g] = 0.f; sm[g] = 0.f; }
    auto base_of = [&](int c, long idx) {
        float4 base = a.x_in ? load4<T>((const T *)a.x_in + idx) : *(const float4 *)(a.res_in + idx);
        if (a.bias) base = f4add(base, load4<T>((const T *)a.bias + 4 * c)); // the row-split layer's bias, once
        return base;
    };
    for (int c = threadIdx.x; c < H4; c += blockDim.x) {
        const long idx = (long)m * H + 4 * c;
        const float4 base = base_of(c, idx);
        float4 tot = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int g = 0; g < MAX_T; ++g) {
            if (g >= G) continue;
            const float4 y = group_sum4(a, g, idx);
            tot = f4add(tot, y);
            const float4 r = f4add(base, y);
            ss[g] += r.x * r.x + r.y * r.y + r.z * r.z + r.w * r.w;
            sm[g] += r.x + r.y + r.z + r.w;
        }
        const float4 r = f4add(base, tot);
        if (a.res_out) *(float4 *)(a.res_out + idx) = r;
        if (a.final_out) store4<T>((T *)a.final_out + idx, r);
    }
    if (!a.h_out) return;
    float rs[MAX_T], mu[MAX_T];
#pragma unroll
    for (int g = 0; g < MAX_T; ++g) {
        rs[g] = 0.f;
        mu[g] = 0.f;
        if (g >= G) continue;
        const float q = block_sum(ss[g], red) / (float)H;
        if (ln) {
            mu[g] = block_sum(sm[g], red) / (float)H;
            rs[g] = rsqrtf(fmaxf(q - mu[g] * mu[g], 0.f) + a.eps);
        } else {
            rs[g] = rsqrtf(q + a.eps);
        }
    }
    const T *gain = (const T *)a.gain;
    for (int c = threadIdx.x; c < H4; c += blockDim.x) {
        const long idx = (long)m * H + 4 * c;
        const float4 base = base_of(c, idx);
        const float4 gj = load4<T>(gain + 4 * c);
        const float4 sh = ln ? load4<T>((const T *)a.shift + 4 * c) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int g = 0; g < MAX_T; ++g) {
            if (g >= G) continue;
            const float4 r = f4add(base, group_sum4(a, g, idx));
            store4<T>((T *)a.h_out + (long)g * a.h_stride + idx,
                      make_float4((r.x - mu[g]) * rs[g] * gj.x + sh.x, (r.y - mu[g]) * rs[g] * gj.y + sh.y,
                                  (r.z - mu[g]) * rs[g] * gj.z + sh.z, (r.w - mu[g]) * rs[g] * gj.w + sh.w));
        }
    }
}

// The same computation with a thread-block cluster of CS CTAs per token row: each CTA owns
// hidden/CS columns, keeps its chunks in registers (single pass over the planes) and the
// row's sums of squares are combined through distributed shared memory.
template <typename T, int NCH>
__global__ void __launch_bounds__(256) residual_norm_cluster_kernel(NormArgs a)
{
    pdl_launch_dependents();
    pdl_wait();
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int m = blockIdx.x / CS, H = a.H, G = a.n_groups, P = a.per_group;
    const int cpc = (H >> 2) / CS; // float4 chunks per CTA
    __shared__ float warp_ss[8][2 * MAX_T];
    __shared__ float cta_ss[2 * MAX_T]; // sums of squares, then (LayerNorm) sums
    const bool ln = a.shift != nullptr;
    float4 base[NCH], y[NCH][MAX_T];
    float ss[MAX_T], sm[MAX_T];
#pragma unroll
    for (int g = 0; g < MAX_T; ++g) { ss[g] = 0.f; sm[g] = 0.f; }
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int lc = threadIdx.x + i * blockDim.x;
        if (lc >= cpc) continue;
        const long idx = (long)m * H + 4 * (rank * cpc + lc);
        base[i] = a.x_in ? load4<T>((const T *)a.x_in + idx) : *(const float4 *)(a.res_in + idx);
        if (a.bias) base[i] = f4add(base[i], load4<T>((const T *)a.bias + 4 * (rank * cpc + lc))); // the row-split layer's bias, once
        float4 tot = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int g = 0; g < MAX_T; ++g) {
            if (g >= G) continue;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            if (a.part) {
#pragma unroll 4
                for (int p = 0; p < P; ++p)
                    acc = f4add(acc, *(const float4 *)(a.part + (long)(g * P + p) * a.part_stride + idx));
            }
            y[i][g] = acc;
            tot = f4add(tot, acc);
            const float4 r = f4add(base[i], acc);
            ss[g] += r.x * r.x + r.y * r.y + r.z * r.z + r.w * r.w;
            sm[g] += r.x + r.y + r.z + r.w;
        }
        const float4 r = f4add(base[i], tot);
        if (a.res_out) *(float4 *)(a.res_out + idx) = r;
        if (a.final_out) store4<T>((T *)a.final_out + idx, r);
    }
    if (!a.h_out) return; // uniform over the whole grid: no CTA of the cluster waits below
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
#pragma unroll
    for (int g = 0; g < MAX_T; ++g) {
        if (g >= G) continue;
        const float v = warp_sum(ss[g]), u = warp_sum(sm[g]);
        if (lane == 0) { warp_ss[warp][g] = v; warp_ss[warp][MAX_T + g] = u; }
    }
    __syncthreads();
    if (threadIdx.x < 2 * MAX_T) {
        float v = 0.f;
        if ((int)(threadIdx.x % MAX_T) < G)
            for (int w = 0; w < nw; ++w) v += warp_ss[w][threadIdx.x];
        cta_ss[threadIdx.x] = v;
    }
    cluster.sync();
    float rs[MAX_T], mu[MAX_T];
#pragma unroll
    for (int g = 0; g < MAX_T; ++g) {
        rs[g] = 0.f;
        mu[g] = 0.f;
        if (g >= G) continue;
        float tot = 0.f, tsum = 0.f;
        for (int r = 0; r < CS; ++r) { tot += cluster.map_shared_rank(cta_ss, r)[g]; tsum += cluster.map_shared_rank(cta_ss, r)[MAX_T + g]; }
        if (ln) {
            mu[g] = tsum / (float)H;
            rs[g] = rsqrtf(fmaxf(tot / (float)H - mu[g] * mu[g], 0.f) + a.eps);
        } else {
            rs[g] = rsqrtf(tot / (float)H + a.eps);
        }
    }
    cluster.sync(); // no CTA may exit while its shared memory is still being read
    const T *gain = (const T *)a.gain;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int lc = threadIdx.x + i * blockDim.x;
        if (lc >= cpc) continue;
        const int col = 4 * (rank * cpc + lc);
        const long idx = (long)m * H + col;
        const float4 gj = load4<T>(gain + col);
        const float4 sh = ln ? load4<T>((const T *)a.shift + col) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int g = 0; g < MAX_T; ++g) {
            if (g >= G) continue;
            const float4 r = f4add(base[i], y[i][g]);
            store4<T>((T *)a.h_out + (long)g * a.h_stride + idx,
                      make_float4((r.x - mu[g]) * rs[g] * gj.x + sh.x, (r.y - mu[g]) * rs[g] * gj.y + sh.y,
                                  (r.z - mu[g]) * rs[g] * gj.z + sh.z, (r.w - mu[g]) * rs[g] * gj.w + sh.w));
        }
    }
}

template <typename T> cudaError_t launch_residual_norm(const NormArgs &a, cudaStream_t st)
{
    if (a.M <= 0) return cudaSuccess;
    if (a.H % 4 || a.n_groups > MAX_T) return cudaErrorInvalidValue;
    const int h4 = a.H / 4;
    constexpr int CS = 8;
    if (h4 % CS == 0 && h4 / CS <= 512 && (long)a.M * CS < 2147483647L) {
        const int cpc = h4 / CS;
        const int threads = cpc >= 256 ? 256 : (cpc + 31) / 32 * 32;
        const dim3 grid((unsigned)(a.M * CS));
        if (cpc <= threads) return launch_kernel(residual_norm_cluster_kernel<T, 1>, grid, dim3(threads), 0, st, CS, a);
        return launch_kernel(residual_norm_cluster_kernel<T, 2>, grid, dim3(threads), 0, st, CS, a);
    }
    const int threads = h4 >= 512 ? 512 : (h4 + 31) / 32 * 32;
    return launch_kernel(residual_norm_kernel<T>, dim3(a.M), dim3(threads), 0, st, 0, a);
}
template cudaError_t launch_residual_norm<float>(const NormArgs &, cudaStream_t);
template cudaError_t launch_residual_norm<bf16>(const NormArgs &, cudaStream_t);

// Block with bias: the two vectors that let a LayerNorm commute with the projection that follows it,
// wg[n] = sum_k g[k] W[n][k] and wb[n] = sum_k beta[k] W[n][k] + b[n] (one warp per weight row, fp32 sums of the
// exact bf16 products).  Run once per projection when the context is created.
__global__ void __launch_bounds__(256) ln_fold_kernel(const bf16 *W, int N, int K, const bf16 *g, const bf16 *beta, const bf16 *b, float *wg,
                                                      float *wb)
{
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (n >= N) return;
    float sg = 0.f, sb = 0.f;
    for (int k = lane; k < K; k += 32) {
        const float w = __bfloat162float(W[(long)n * K + k]);
        sg = fmaf(__bfloat162float(g[k]), w, sg);
        sb = fmaf(__bfloat162float(beta[k]), w, sb);
    }
    sg = warp_sum(sg);
    sb = warp_sum(sb);
    if (lane == 0) { wg[n] = sg; wb[n] = sb + (b ? __bfloat162float(b[n]) : 0.f); }
}

cudaError_t launch_ln_fold(const void *W, int N, int K, const void *g, const void *beta, const void *b, float *wg, float *wb, cudaStream_t st)
{
    if (N <= 0) return cudaSuccess;
    ln_fold_kernel<<<(N + 7) / 8, 256, 0, st>>>((const bf16 *)W, N, K, (const bf16 *)g, (const bf16 *)beta, (const bf16 *)b, wg, wb);
    return cudaGetLastError();
}

// cos/sin of pos * base^(-2j/d), evaluated in double once per call and shared by all layers.
__global__ void rope_table_kernel(float2 *table, TokMap tm, int M, int half, double log_base, int d, unsigned long long *stamp)
{
    pdl_launch_dependents();
    if (threadIdx.x == 0) stamp_entry(stamp);
    pdl_wait();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < M * half) {
        int m = i / half, j = i % half, b, pos;
        tm.locate(m, b, pos);
        double theta = exp(-2.0 * (double)j / (double)d * log_base);
        double s, c;
        sincos((double)pos * theta, &s, &c);
        table[i] = make_float2((float)c, (float)s);
    }
    if (threadIdx.x == 0) stamp_exit(stamp);
}

cudaError_t launch_rope_table(float2 *table, TokMap tm, int M, int head_dim, float base, cudaStream_t st, unsigned long long *stamp)
{
    int n = M * (head_dim / 2);
    if (n <= 0) return cudaSuccess;
    return launch_kernel(rope_table_kernel, dim3((n + 255) / 256), dim3(256), 0, st, 0, table, tm, M, head_dim / 2,
                         log((double)base), head_dim, stamp);
}

// grid (M, n_q_heads + n_kv_heads): sums the split-K planes of one head's projection, rotates
// q and k (pairs (j, j + d/2)), stores q for the attention kernel and k, v into their page.
template <typename T> __global__ void rope_kv_kernel(RopeKvArgs a)
{
    pdl_launch_dependents();
    pdl_wait();
    const int m = blockIdx.x, head = blockIdx.y, d = a.head_dim, half = d / 2;
    const int nq = a.n_q_heads, nkv = a.pt.n_kv_heads;
    int b, pos;
    a.tm.locate(m, b, pos);
    const bool is_q = head < nq;
    const int kvh = head - nq;
    long kv_off = 0;
    if (!is_q) {
        int pi = pos / a.pt.block;
        if (pos < 0 || pi >= a.pt.max_pages) { if (threadIdx.x == 0) atomicOr(a.err, ERR_CAPACITY); return; }
        int page = a.pt.block_table[(long)b * a.pt.max_pages + pi];
        if (page < 0 || page >= a.pt.n_pages) { if (threadIdx.x == 0) atomicOr(a.err, ERR_PAGE_RANGE); return; }
        kv_off = (((long)page * nkv + kvh) * a.pt.block + pos % a.pt.block) * d;
    }
    const long col_q = (long)head * d;                 // q or k column of this head
    const long col_v = (long)(nq + nkv + kvh) * d;     // v column (kv heads only)
    for (int j = threadIdx.x; j < half; j += blockDim.x) {
        float x0 = 0.f, x1 = 0.f, v0 = 0.f, v1 = 0.f;
        for (int s = 0; s < a.splits; ++s) {
            const float *row = a.qkv + (long)s * a.split_stride + (long)m * a.ldq;
            x0 += row[col_q + j];
            x1 += row[col_q + j + half];
            if (!is_q) { v0 += row[col_v + j]; v1 += row[col_v + j + half]; }
        }
        if (is_q && a.bq) { x0 += to_f<T>(((const T *)a.bq)[col_q + j]); x1 += to_f<T>(((const T *)a.bq)[col_q + j + half]); }
        if (!is_q && a.bk) { x0 += to_f<T>(((const T *)a.bk)[(long)kvh * d + j]); x1 += to_f<T>(((const T *)a.bk)[(long)kvh * d + j + half]); }
        if (!is_q && a.bv) { v0 += to_f<T>(((const T *)a.bv)[(long)kvh * d + j]); v1 += to_f<T>(((const T *)a.bv)[(long)kvh * d + j + half]); }
        float c = 1.f, sn = 0.f;
        if (a.use_rope) { float2 cs = a.table[(long)m * half + j]; c = cs.x; sn = cs.y; }
        float r0 = x0 * c - x1 * sn, r1 = x1 * c + x0 * sn;
        if (is_q) {
            T *q = (T *)a.q_out + (long)m * nq * d + (long)head * d;
            q[j] = from_f<T>(r0);
            q[j + half] = from_f<T>(r1);
        } else {
            T *kp = (T *)a.k_pages + kv_off, *vp = (T *)a.v_pages + kv_off;
            kp[j] = from_f<T>(r0);
            kp[j + half] = from_f<T>(r1);
            vp[j] = from_f<T>(v0);
            vp[j + half] = from_f<T>(v1);
        }
    }
}

template <typename T> cudaError_t launch_rope_kv(const RopeKvArgs &a, cudaStream_t st)
{
    if (a.M <= 0) return cudaSuccess;
    dim3 grid(a.M, a.n_q_heads + a.pt.n_kv_heads);
    int threads = a.head_dim / 2 >= 64 ? 64 : 32;
    return launch_kernel(rope_kv_kernel<T>, grid, dim3(threads), 0, st, 0, a);
}
template cudaError_t launch_rope_kv<float>(const RopeKvArgs &, cudaStream_t);
template cudaError_t launch_rope_kv<bf16>(const RopeKvArgs &, cudaStream_t);

// act = silu(sum_s gate_s) * (sum_s up_s)
template <typename T> __global__ void silu_mul_kernel(SiluMulArgs a)
{
    pdl_launch_dependents();
    pdl_wait();
    long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long n = (long)a.M * a.F;
    if (i >= n) return;
    long m = i / a.F, f = i % a.F;
    float g = 0.f, u = 0.f;
    for (int s = 0; s < a.splits; ++s) {
        g += a.gate[(long)s * a.split_stride + m * a.ld + f];
        if (!a.relu) u += a.up[(long)s * a.split_stride + m * a.ld + f];
    }
    if (a.bias) g += to_f<T>(((const T *)a.bias)[f]);
    float act = a.relu ? fmaxf(g, 0.f) : g / (1.f + __expf(-g)) * u;
    ((T *)a.act)[i] = from_f<T>(act);
}

template <typename T> cudaError_t launch_silu_mul(const SiluMulArgs &a, cudaStream_t st)
{
    long n = (long)a.M * a.F;
    if (n <= 0) return cudaSuccess;
    return launch_kernel(silu_mul_kernel<T>, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, 0, a);
}
template cudaError_t launch_silu_mul<float>(const SiluMulArgs &, cudaStream_t);
template cudaError_t launch_silu_mul<bf16>(const SiluMulArgs &, cudaStream_t);

} // namespace spd
