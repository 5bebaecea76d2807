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

// ---------------------------------------------------------------------------------------
// Causal prefill attention on tensor cores (bf16): one thread block per 128 query rows of one
// (sequence, query head); K/V tiles of 64 cached tokens are gathered from their pages into
// double-buffered, XOR-swizzled shared memory with cp.async; each of the 8 warps owns 16 query
// rows: S = Q K^T and O += P V as m16n8k16 MMAs with fp32 accumulators, online softmax in
// base 2 on the accumulator fragments, P re-used in registers as the A operand of the second
// product.  Chunked prefill: queries at positions s0.. attend to every cached position <= their own.
namespace fa {

constexpr int NW = 8, BQ = 16 * NW, BKV = 64, FA_THREADS = 32 * NW;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? 16 : 0; // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(uint32_t *)&v;
}
// byte offset of 16-byte chunk `c` of row `r` in a [rows][D] bf16 tile (chunks XOR-swizzled by row)
template <int D> __device__ __forceinline__ uint32_t tile_off(int r, int c) { return (uint32_t)(r * D * 2 + ((c ^ (r & 7)) << 4)); }

template <int D>
__global__ void __launch_bounds__(FA_THREADS, 2) prefill_attention_mma_kernel(AttnArgs a)
{
    constexpr int CH = D / 8;       // 16-byte chunks per row
    constexpr int KS = D / 16;      // k-steps of Q K^T
    constexpr int NT = BKV / 8;     // n-tiles of S
    constexpr int DT = D / 8;       // n-tiles of O
    extern __shared__ __align__(128) uint8_t fa_smem[];
    const uint32_t sQ = tc::smem_u32(fa_smem), sK = sQ + BQ * D * 2, sV = sK + 2 * BKV * D * 2;
    pdl_launch_dependents();
    if (threadIdx.x == 0) stamp_entry(a.stamp);
    pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int q0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * BQ, hq = blockIdx.y, bi = blockIdx.z; // longest rows first
    const int ns = a.tm.ns, s0 = a.tm.s0, b = a.tm.b0 + bi;
    const int kvh = hq / (a.n_q_heads / a.pt.n_kv_heads);
    const int q_rows = min(BQ, ns - q0);
    const int kv_len = s0 + q0 + q_rows;                 // keys 0 .. last query position of the tile
    const int n_tiles = (kv_len + BKV - 1) / BKV;
    const bf16 *kp = (const bf16 *)a.k_pages, *vp = (const bf16 *)a.v_pages;

    auto load_kv = [&](int tile, int buf) {
        const uint32_t dK = sK + buf * BKV * D * 2, dV = sV + buf * BKV * D * 2;
#pragma unroll
        for (int i = 0; i < BKV * CH / FA_THREADS; ++i) {
            const int idx = tid + i * FA_THREADS, r = idx / CH, c = idx % CH, tkn = tile * BKV + r;
            const bool valid = tkn < kv_len;
            long off = 0;
            if (valid) {
                int page = a.pt.block_table[(long)b * a.pt.max_pages + tkn / a.pt.block];
                if (page < 0 || page >= a.pt.n_pages) { atomicOr(a.err, ERR_PAGE_RANGE); page = 0; }
                off = (((long)page * a.pt.n_kv_heads + kvh) * a.pt.block + tkn % a.pt.block) * D + c * 8;
            }
            cp_async16(dK + tile_off<D>(r, c), kp + off, valid);
            cp_async16(dV + tile_off<D>(r, c), vp + off, valid);
        }
    };
    // Q tile
#pragma unroll
    for (int i = 0; i < BQ * CH / FA_THREADS; ++i) {
        const int idx = tid + i * FA_THREADS, r = idx / CH, c = idx % CH;
        const bool valid = r < q_rows;
        const bf16 *src = (const bf16 *)a.q + ((long)(bi * ns + q0 + (valid ? r : 0)) * a.n_q_heads + hq) * D + c * 8;
        cp_async16(sQ + tile_off<D>(r, c), src, valid);
    }
    cp_async_commit();
    load_kv(0, 0);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    // the A fragments of this warp's 16 query rows are re-read from the Q tile for every K tile
    // (keeps the register count at two thread blocks per SM)
    const uint32_t q_addr_row = warp * 16 + (lane & 15);
    float o[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const float sc = rsqrtf((float)D) * 1.4426950408889634f;
    // positions of this thread's two rows (g and g + 8 of the warp's 16); -1 for rows past the tile
    int pos_q[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = warp * 16 + g + 8 * h;
        pos_q[h] = r < q_rows ? s0 + q0 + r : -1;
    }
    for (int j = 0; j < n_tiles; ++j) {
        const int buf = j & 1;
        if (j + 1 < n_tiles) load_kv(j + 1, buf ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t bK = sK + buf * BKV * D * 2, bV = sV + buf * BKV * D * 2;
        float s[NT][4];
#pragma unroll
        for (int i = 0; i < NT; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
            uint32_t qf[4];
            ldsm_x4(qf, sQ + tile_off<D>(q_addr_row, kk * 2 + (lane >> 4)));
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
                // matrices: (tokens np*16 + 0..7, dims kk*16 + 0..7), (same tokens, dims + 8), (tokens + 8, dims), (tokens + 8, dims + 8)
                uint32_t kf[4];
                const int r = np * 16 + (lane & 7) + ((lane >> 4) << 3), c = kk * 2 + ((lane >> 3) & 1);
                ldsm_x4(kf, bK + tile_off<D>(r, c));
                mma_bf16(s[2 * np], qf, kf[0], kf[1]);
                mma_bf16(s[2 * np + 1], qf, kf[2], kf[3]);
            }
        }
        // scale, causal mask (only tiles that reach past this warp's first query position), running max
        float m_new[2] = {m_run[0], m_run[1]};
        const bool need_mask = (j + 1) * BKV - 1 > s0 + q0 + warp * 16 || q0 + warp * 16 + 16 > q_rows;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = j * BKV + nt * 8 + 2 * t4 + (e & 1), h = e >> 1;
                const float v = (!need_mask || key <= pos_q[h]) ? s[nt][e] * sc : -INFINITY;
                s[nt][e] = v;
                m_new[h] = fmaxf(m_new[h], v);
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            m_new[h] = fmaxf(m_new[h], __shfl_xor_sync(0xffffffffu, m_new[h], 1));
            m_new[h] = fmaxf(m_new[h], __shfl_xor_sync(0xffffffffu, m_new[h], 2));
        }
        float corr[2], base[2], rs[2] = {0.f, 0.f};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            base[h] = m_new[h] == -INFINITY ? 0.f : m_new[h];
            corr[h] = m_run[h] == -INFINITY ? 0.f : exp2f(m_run[h] - base[h]);
            m_run[h] = m_new[h];
        }
        uint32_t pf[NT / 2][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                p[e] = exp2f(s[nt][e] - base[e >> 1]);
                rs[e >> 1] += p[e];
            }
            // accumulator layout of two adjacent n-tiles = A layout of one 16-wide k-step
            pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) l_run[h] = l_run[h] * corr[h] + rs[h];
#pragma unroll
        for (int dt = 0; dt < DT; ++dt) { o[dt][0] *= corr[0]; o[dt][1] *= corr[0]; o[dt][2] *= corr[1]; o[dt][3] *= corr[1]; }
#pragma unroll
        for (int k2 = 0; k2 < BKV / 16; ++k2) {
#pragma unroll
            for (int dp = 0; dp < DT / 2; ++dp) {
                // transposed loads: (tokens k2*16 + 0..7, dims dp*16 + 0..7), (tokens + 8, dims), (tokens, dims + 8), (tokens + 8, dims + 8)
                uint32_t vf[4];
                const int r = k2 * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), c = dp * 2 + (lane >> 4);
                ldsm_x4_t(vf, bV + tile_off<D>(r, c));
                mma_bf16(o[2 * dp], pf[k2], vf[0], vf[1]);
                mma_bf16(o[2 * dp + 1], pf[k2], vf[2], vf[3]);
            }
        }
        __syncthreads(); // this buffer is refilled two iterations from now
    }
    // row sums across the quad, normalise, store
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = warp * 16 + g + 8 * h;
        if (r >= q_rows) continue;
        const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;
        bf16 *dst = (bf16 *)a.out + ((long)(bi * ns + q0 + r) * a.n_q_heads + hq) * D;
#pragma unroll
        for (int dt = 0; dt < DT; ++dt)
            *(uint32_t *)(dst + dt * 8 + 2 * t4) = pack_bf16(o[dt][2 * h] * inv, o[dt][2 * h + 1] * inv);
    }
    if (threadIdx.x == 0) stamp_exit(a.stamp);
}

template <int D> cudaError_t launch(const AttnArgs &a, int n_seq, cudaStream_t st)
{
    constexpr int SMEM = (BQ + 4 * BKV) * D * 2;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(prefill_attention_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    dim3 grid((a.tm.ns + BQ - 1) / BQ, a.n_q_heads, n_seq);
    return launch_kernel(prefill_attention_mma_kernel<D>, grid, dim3(FA_THREADS), SMEM, st, 0, a);
}

} // namespace fa

template <typename T> cudaError_t launch_prefill_attention_tc(const AttnArgs &, cudaStream_t, bool &done) { done = false; return cudaSuccess; }
template <> cudaError_t launch_prefill_attention_tc<bf16>(const AttnArgs &a, cudaStream_t st, bool &done)
{
    done = false;
    if (a.tm.decode || a.tm.ns <= 0 || a.M % a.tm.ns) return cudaSuccess;
    done = true;
    if (a.head_dim == 128 && a.pt.block == 16 && a.q_map && a.k_map && a.v_map) return launch_prefill_attention_umma(a, st);
    switch (a.head_dim) {
    case 128: return fa::launch<128>(a, a.M / a.tm.ns, st);
    case 64: return fa::launch<64>(a, a.M / a.tm.ns, st);
    default: done = false; return cudaSuccess;
    }
}

template <typename T> cudaError_t launch_prefill_attention(const AttnArgs &a, cudaStream_t st)
{
    if (a.M <= 0) return cudaSuccess;
    bool done = false;
    cudaError_t e = launch_prefill_attention_tc<T>(a, st, done);
    if (done || e != cudaSuccess) return e;
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

// Merge of the context splits by the last thread block of a (sequence, head tile): the
// per-split maxima and denominators are turned into weights once (shared memory), then every
// thread adds up its output elements with the partial loads issued eight at a time.
// scratch: at least 2 * GT * splits floats of shared memory no longer in use.
template <typename T, int D, int GT>
__device__ __forceinline__ void merge_splits(const AttnArgs &a, int b, int hq0, float *scratch)
{
    const int S = a.splits;
    float *wgt = scratch, *inv = scratch + GT * S; // weight of split s2 for head g; 1 / denominator per head
    for (int i = threadIdx.x; i < GT * S; i += blockDim.x) {
        const int g = i / S;
        const long q0 = ((long)b * a.n_q_heads + hq0 + g) * S;
        wgt[i] = __ldcg(a.part_ml + (q0 + i % S) * 2); // the split's maximum for now
    }
    __syncthreads();
    if (threadIdx.x < GT) {
        const int g = threadIdx.x;
        const long q0 = ((long)b * a.n_q_heads + hq0 + g) * S;
        float gm = -INFINITY, den = 0.f;
        for (int s2 = 0; s2 < S; ++s2) gm = fmaxf(gm, wgt[g * S + s2]);
        for (int s2 = 0; s2 < S; ++s2) {
            const float m2 = wgt[g * S + s2];
            const float c = (m2 == -INFINITY) ? 0.f : exp2f(m2 - gm);
            wgt[g * S + s2] = c;
            den += __ldcg(a.part_ml + (q0 + s2) * 2 + 1) * c;
        }
        inv[g] = den > 0.f ? 1.f / den : 0.f;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < GT * D; idx += blockDim.x) {
        const int g = idx / D, dd = idx % D;
        const float *po = a.part_o + ((long)b * a.n_q_heads + hq0 + g) * S * D + dd;
        float acc = 0.f;
        for (int s0 = 0; s0 < S; s0 += 8) {
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = s0 + k < S ? __ldcg(po + (long)(s0 + k) * D) : 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) acc += v[k] * (s0 + k < S ? wgt[g * S + s0 + k] : 0.f);
        }
        ((T *)a.out)[((long)b * a.n_q_heads + hq0 + g) * D + dd] = from_f<T>(acc * inv[g]);
    }
}

// Tail of the paged decode kernels: merge the four compute warps of the block, then the context
// splits.  With up to 8 splits the blocks of one (sequence, head tile) form a thread-block cluster:
// each parks its merged, un-normalised partial in shared memory and, after one cluster barrier,
// block r finishes every splits-th output element from its peers' shared memory - no partial goes
// through global memory.  More splits: partials in global memory, last block to arrive merges.
template <typename T, int D, int GT>
__device__ __forceinline__ void finish_decode_attention(const AttnArgs &a, int b, int hq0, int sp, float (*sm_o)[GT][D],
                                                        float (*sm_ml)[GT][2], float *sm_pml, int *sm_last)
{
    const bool clustered = a.cluster_merge && a.splits > 1;
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
        } else if (clustered) {
            sm_o[0][g][dd] = acc; // only this thread reads (g, dd) of the warps' partials
            if (dd == 0) { sm_pml[2 * g] = gm; sm_pml[2 * g + 1] = gden; }
        } else {
            const long pi = pbase + (long)g * a.splits;
            a.part_o[pi * D + dd] = acc; // un-normalised
            if (dd == 0) { a.part_ml[pi * 2] = gm; a.part_ml[pi * 2 + 1] = gden; }
        }
    }
    if (a.splits == 1) return;
    if (clustered) {
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        const uint32_t o_base = tc::smem_u32(&sm_o[0][0][0]), ml_base = tc::smem_u32(sm_pml);
        auto peer_f = [](uint32_t addr, int rank) {
            uint32_t ra;
            float v;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(addr), "r"(rank));
            asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
            return v;
        };
        for (int idx = sp + a.splits * (int)threadIdx.x; idx < GT * D; idx += a.splits * (int)blockDim.x) {
            const int g = idx / D;
            float gm = -INFINITY;
            for (int s2 = 0; s2 < a.splits; ++s2) gm = fmaxf(gm, peer_f(ml_base + 8 * g, s2));
            float acc = 0.f, gden = 0.f;
            for (int s2 = 0; s2 < a.splits; ++s2) {
                const float m2 = peer_f(ml_base + 8 * g, s2);
                const float c = (m2 == -INFINITY) ? 0.f : exp2f(m2 - gm);
                acc += peer_f(o_base + 4 * idx, s2) * c;
                gden += peer_f(ml_base + 8 * g + 4, s2) * c;
            }
            ((T *)a.out)[((long)b * a.n_q_heads + hq0) * D + idx] = from_f<T>(gden > 0.f ? acc / gden : 0.f);
        }
        // no block may exit while a peer still reads its shared memory
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        return;
    }
    // the last block of this (sequence, head tile) to arrive merges the splits
    __threadfence();
    __syncthreads();
    int *cnt = a.counters + (long)b * gridDim.x + blockIdx.x;
    if (threadIdx.x == 0) *sm_last = (atomicAdd(cnt, 1) == a.splits - 1);
    __syncthreads();
    if (!*sm_last) return;
    __threadfence();
    merge_splits<T, D, GT>(a, b, hq0, &sm_o[0][0][0]);
    if (threadIdx.x == 0) *cnt = 0; // ready for the next launch
}

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
    if (threadIdx.x == 0) { SPD_TRACE_EVENT(TRK_ATTN, TR_START); stamp_entry(a.stamp); }
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
    if (threadIdx.x == 0) { SPD_TRACE_EVENT(TRK_ATTN, TR_MAIN_DONE); stamp_exit(a.stamp); }
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
    if (threadIdx.x == 0) { SPD_TRACE_EVENT(TRK_ATTN, TR_END); stamp_exit(a.stamp); }
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
// DENSE: compiled for five resident blocks per SM instead of four (72 registers); each block is a little slower,
// but a launch of 593-740 blocks (16 sequences x 40 heads, say) is resident at once instead of leaving a short
// second wave - chosen by the launcher.
template <typename T, int D, int GT, bool DENSE>
__global__ void __launch_bounds__(160, DENSE ? 5 : 4) decode_attention_ring_kernel(AttnArgs a)
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
    float *sm_pml = (float *)(sm_bt + DECODE_MAX_PAGES_PER_BLOCK + 2); // [GT][2] merged max, denominator of this block
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (R + s); };

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hq0 = blockIdx.x * GT, b = blockIdx.y, sp = blockIdx.z;
    const int kvh = hq0 / (a.n_q_heads / a.pt.n_kv_heads);

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        SPD_TRACE_EVENT(TRK_ATTN, TR_START);
        stamp_entry(a.stamp);
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
    finish_decode_attention<T, D, GT>(a, b, hq0, sp, sm_o, sm_ml, sm_pml, sm_last);
    if (threadIdx.x == 0) { SPD_TRACE_EVENT(TRK_ATTN, TR_END); stamp_exit(a.stamp); }
}

template <typename T, int D, int GT, bool DENSE> cudaError_t launch_ring_as(const AttnArgs &a, cudaStream_t st)
{
    constexpr int PAGE_BYTES = 16 * D * (int)sizeof(T), R = DecodeRing<T, D>::SLOTS;
    constexpr int SMEM = R * 2 * PAGE_BYTES + 4 * GT * D * 4 + 4 * GT * 2 * 4 + 2 * R * 8 + (DECODE_MAX_PAGES_PER_BLOCK + 2 + 2 * GT) * 4;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(decode_attention_ring_kernel<T, D, GT, DENSE>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        // ask for the largest shared-memory carve-out so that four (five) blocks fit an SM
        e = cudaFuncSetAttribute(decode_attention_ring_kernel<T, D, GT, DENSE>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    dim3 grid(a.n_q_heads / GT, a.B, a.splits);
    AttnArgs b = a;
    b.cluster_merge = a.splits > 1 && a.splits <= 8;
    return launch_kernel_z(decode_attention_ring_kernel<T, D, GT, DENSE>, grid, dim3(160), SMEM, st, b.cluster_merge ? a.splits : 1, b);
}

template <typename T, int D, int GT> cudaError_t launch_ring(const AttnArgs &a, cudaStream_t st)
{
    // five blocks per SM where that saves a wave (one query head per block only: the wider blocks would spill)
    const long SMS = sm_count();
    const long blocks = (long)(a.n_q_heads / GT) * a.B * a.splits;
    const bool dense = GT == 1 && (blocks + 5 * SMS - 1) / (5 * SMS) < (blocks + 4 * SMS - 1) / (4 * SMS);
    if (GT == 1 && dense) return launch_ring_as<T, D, 1, true>(a, st);
    return launch_ring_as<T, D, GT, false>(a, st);
}

// ---------------------------------------------------------------------------------------
// Grouped-query decode attention on tensor cores (bf16, head_dim 128, 16-token pages).  With a
// GQA group of 8 query heads per KV head the CUDA-core kernel above is bound by arithmetic
// (8 x 2 flops per cached element), not by the KV stream.  Here the group's query heads are the
// rows of an m16n8k16 MMA: S[heads x 16 tokens] = Q K^T and O[heads x 128] += P V per page.
// Pages arrive through TMA tensor copies (one box per page and tensor: 64 dims x 16 tokens x the two
// halves of the head dimension) in the 128-byte swizzle that ldmatrix reads without bank conflicts.  Warp roles and split merge: as in the bulk-copy kernel.  The page ring has more slots than
// compute warps (six or eight for four warps): page i goes to slot i % R and to warp i % 4, so a warp's next page is
// on its way while it works on the current one - with one slot per warp every page would cost a full memory latency.
// The warps' partial outputs are merged through the ring's own bytes once every page has been read.
// DENSE: compiled for four resident blocks per SM instead of three (96 registers, six slots instead of eight), taken
// by the launcher where it saves a wave.
template <bool DENSE> struct DecodeMmaRing { static constexpr int SLOTS = DENSE ? 6 : 8; };

template <int GT, bool DENSE>
__global__ void __launch_bounds__(160, DENSE ? 4 : 3) decode_attention_mma_kernel(const __grid_constant__ CUtensorMap tm_k,
                                                                   const __grid_constant__ CUtensorMap tm_v, AttnArgs a)
{
    using namespace tc;
    using fa::ldsm_x4;
    using fa::ldsm_x4_t;
    using fa::mma_bf16;
    using fa::pack_bf16;
    constexpr int D = 128, BLK = 16, R = DecodeMmaRing<DENSE>::SLOTS, SUB = 2048 /* 16 tokens x 64 dims */, SLOT = 4 * SUB;
    static_assert(R * SLOT >= 4 * GT * D * 4 + 4 * GT * 2 * 4, "the merge area lives in the ring");
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t ring = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t *gen = smem_dyn + (ring - smem_u32(smem_dyn));
    float(*sm_o)[GT][D] = (float(*)[GT][D])gen; // over the ring, after its last read
    float(*sm_ml)[GT][2] = (float(*)[GT][2])(gen + 4 * GT * D * 4);
    uint8_t *tail = gen + R * SLOT;
    const uint32_t bars = smem_u32(tail);             // full[R], empty[R]
    int *sm_bt = (int *)(tail + 2 * R * 8);
    volatile int *abort_flag = (volatile int *)(sm_bt + DECODE_MAX_PAGES_PER_BLOCK);
    int *sm_last = (int *)(sm_bt + DECODE_MAX_PAGES_PER_BLOCK + 1);
    float *sm_pml = (float *)(sm_bt + DECODE_MAX_PAGES_PER_BLOCK + 2); // [GT][2] merged max, denominator of this block
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (R + s); };

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t4 = lane & 3;
    const int hq0 = blockIdx.x * GT, b = blockIdx.y, sp = blockIdx.z;
    const int kvh = hq0 / (a.n_q_heads / a.pt.n_kv_heads);

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        SPD_TRACE_EVENT(TRK_ATTN, TR_START);
        stamp_entry(a.stamp);
        for (int s = 0; s < R; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int ctx = a.tm.seq_lens[b] + 1;
    const bool bad = ctx < 1 || ctx > a.max_context || (ctx - 1) / BLK >= a.pt.max_pages;
    const int pages_bucket = (a.max_context + BLK - 1) / BLK;
    const int per = (pages_bucket + a.splits - 1) / a.splits;
    const int p0 = sp * per;
    const int ctx_pages = bad ? 0 : (ctx + BLK - 1) / BLK;
    const int n_pages = max(0, min(ctx_pages, p0 + per) - p0);
    const int new_page = (ctx - 1) / BLK;
    if (bad && threadIdx.x == 0) atomicOr(a.err, ERR_CAPACITY);

    if (warp == 4) {
        for (int i = lane; i < n_pages; i += 32) {
            int page = a.pt.block_table[(long)b * a.pt.max_pages + p0 + i];
            if (page < 0 || page >= a.pt.n_pages) { atomicOr(a.err, ERR_PAGE_RANGE); page = 0; }
            sm_bt[i] = page;
        }
        __syncwarp();
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_k) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_v) : "memory");
            bool waited = false;
            for (int i = 0; i < n_pages; ++i) {
                const int s = i % R;
                if (!waited && p0 + i >= new_page) { pdl_wait(); waited = true; }
                if (i >= R && !mbar_wait(empty_bar(s), ((i / R) & 1) ^ 1, a.err, abort_flag)) break;
                const int row = (sm_bt[i] * a.pt.n_kv_heads + kvh) * BLK; // first of the page's 16 token rows
                const uint32_t dst = ring + s * SLOT;
                mbar_expect_tx(full_bar(s), SLOT);
                tma_load_3d(dst, &tm_k, 0, row, 0, full_bar(s));           // both halves of the head dimension: 2 x (16 x 64)
                tma_load_3d(dst + 2 * SUB, &tm_v, 0, row, 0, full_bar(s));
            }
        }
        __syncwarp();
    }
    pdl_wait(); // q comes from the preceding kernel
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_DEP_DONE);

    if (warp < 4) {
        // Tokens are the MMA rows and the group's query heads its 8 columns, so that no row of a 16 x 8 tile is
        // padding: S^T[16 tokens x 8 heads] = K Q^T and O^T[128 dims x 8 heads] += V^T P^T, 8 + 8 MMAs per page.
        // B fragments of Q^T: column g = query head hq0 + g (columns >= GT are padding), rows = 16 dims per step.
        uint32_t qb[8][2];
        {
            const bf16 *qp = (const bf16 *)a.q + ((long)b * a.n_q_heads + hq0 + g) * D;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                qb[kk][0] = g < GT ? *(const uint32_t *)(qp + kk * 16 + 2 * t4) : 0u;
                qb[kk][1] = g < GT ? *(const uint32_t *)(qp + kk * 16 + 8 + 2 * t4) : 0u;
            }
        }
        // this lane's share of O^T: dims dp*16 + g (o[dp][0..1]) and dp*16 + g + 8 (o[dp][2..3]), heads 2*t4 + {0,1}
        float o[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f}; // heads 2*t4 + {0,1}; l_run: this lane's tokens only
        const float sc = rsqrtf((float)D) * 1.4426950408889634f;
        for (int pi = warp; pi < n_pages; pi += 4) {
            const int s = pi % R;
            // Where the slots are not a multiple of the warps, the page that had this slot before (pi - R) belonged to
            // another warp, which may be behind: a parity wait can only tell a phase from the one next to it, so wait
            // until that page has been released (the slot's "empty" phase) before waiting for this one to be full.
            if (R % 4 != 0 && pi >= R && !mbar_wait(empty_bar(s), ((pi / R) & 1) ^ 1, a.err, abort_flag)) break;
            if (!mbar_wait(full_bar(s), (pi / R) & 1, a.err, abort_flag)) break;
            const uint32_t kb = ring + s * SLOT, vb = kb + 2 * SUB;
            float sv[4] = {0.f, 0.f, 0.f, 0.f}; // tokens g (sv[0..1]) and g + 8 (sv[2..3]) x heads 2*t4 + {0,1}
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                uint32_t kf[4]; // A fragment: tokens x 16 dims
                const int r = (lane & 7) + (((lane >> 3) & 1) << 3), c = (kk & 3) * 2 + (lane >> 4);
                ldsm_x4(kf, kb + (kk >> 2) * SUB + r * 128 + ((c ^ (r & 7)) << 4));
                mma_bf16(sv, kf, qb[kk][0], qb[kk][1]);
            }
            const int tbase = (p0 + pi) * BLK;
            const bool ok0 = tbase + g < ctx, ok1 = tbase + g + 8 < ctx;
            float pv[2][2], corr[2]; // [head][token g / g + 8]
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                pv[e][0] = ok0 ? sv[e] * sc : -INFINITY;
                pv[e][1] = ok1 ? sv[2 + e] * sc : -INFINITY;
                float mx = fmaxf(m_run[e], fmaxf(pv[e][0], pv[e][1]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                const float base = mx == -INFINITY ? 0.f : mx;
                corr[e] = m_run[e] == -INFINITY ? 0.f : exp2f(m_run[e] - base);
                m_run[e] = mx;
                pv[e][0] = exp2f(pv[e][0] - base);
                pv[e][1] = exp2f(pv[e][1] - base);
                l_run[e] = l_run[e] * corr[e] + pv[e][0] + pv[e][1];
            }
            // P^T as the B operand (16 tokens x 8 heads): the accumulator layout holds (token g; heads 2*t4, 2*t4+1),
            // the operand wants (head g; tokens 2*t4, 2*t4+1) - an 8 x 8 transpose across the warp per token half
            uint32_t pb0, pb1;
            {
                const uint32_t lo = pack_bf16(pv[0][0], pv[1][0]), hi = pack_bf16(pv[0][1], pv[1][1]);
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb0) : "r"(lo));
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb1) : "r"(hi));
            }
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                o[dp][0] *= corr[0]; o[dp][1] *= corr[1]; o[dp][2] *= corr[0]; o[dp][3] *= corr[1];
                uint32_t vf[4]; // A fragment of V^T: 16 dims x 16 tokens, read transposed from the [token][dim] page
                const int r = (lane & 7) + ((lane >> 4) << 3), c = (dp & 3) * 2 + ((lane >> 3) & 1);
                ldsm_x4_t(vf, vb + (dp >> 2) * SUB + r * 128 + ((c ^ (r & 7)) << 4));
                mma_bf16(o[dp], vf, pb0, pb1);
            }
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(s)) : "memory");
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 4);
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 8);
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 16);
        }
        asm volatile("bar.sync 1, 128;" ::: "memory"); // every compute warp is done with the ring: the merge area may overwrite it
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int h = 2 * t4 + e;
            if (h < GT) {
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {
                    sm_o[warp][h][dp * 16 + g] = o[dp][e];
                    sm_o[warp][h][dp * 16 + g + 8] = o[dp][2 + e];
                }
                if (g == 0) { sm_ml[warp][h][0] = m_run[e]; sm_ml[warp][h][1] = l_run[e]; }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_ATTN, TR_MAIN_DONE);
    finish_decode_attention<bf16, D, GT>(a, b, hq0, sp, sm_o, sm_ml, sm_pml, sm_last);
    if (threadIdx.x == 0) { SPD_TRACE_EVENT(TRK_ATTN, TR_END); stamp_exit(a.stamp); }
}

template <int GT, bool DENSE> cudaError_t launch_decode_mma_as(const AttnArgs &a, cudaStream_t st)
{
    constexpr int R = DecodeMmaRing<DENSE>::SLOTS;
    constexpr int SMEM = 1024 + R * 8192 + 2 * R * 8 + (DECODE_MAX_PAGES_PER_BLOCK + 2 + 2 * GT) * 4;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(decode_attention_mma_kernel<GT, DENSE>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(decode_attention_mma_kernel<GT, DENSE>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    dim3 grid(a.n_q_heads / GT, a.B, a.splits);
    AttnArgs b = a;
    b.cluster_merge = a.splits > 1 && a.splits <= 8;
    return launch_kernel_z(decode_attention_mma_kernel<GT, DENSE>, grid, dim3(160), SMEM, st, b.cluster_merge ? a.splits : 1,
                           *(const CUtensorMap *)a.k_map, *(const CUtensorMap *)a.v_map, b);
}

template <int GT> cudaError_t launch_decode_mma(const AttnArgs &a, cudaStream_t st)
{
    const long SMS = sm_count();
    const long blocks = (long)(a.n_q_heads / GT) * a.B * a.splits;
    if ((blocks + 4 * SMS - 1) / (4 * SMS) < (blocks + 3 * SMS - 1) / (3 * SMS)) return launch_decode_mma_as<GT, true>(a, st);
    return launch_decode_mma_as<GT, false>(a, st);
}

template <typename T, int D> cudaError_t launch_decode_d(const AttnArgs &a, cudaStream_t st)
{
    const int group = a.n_q_heads / a.pt.n_kv_heads;
    const int pages_bucket = (a.max_context + 15) / 16;
    const bool fits = (pages_bucket + a.splits - 1) / a.splits <= DECODE_MAX_PAGES_PER_BLOCK;
    if (fits && a.k_map && a.v_map && decode_uses_mma(group, D, sizeof(T) == 2, a.pt.block))
        return decode_heads_per_block_mma(group) == 8 ? launch_decode_mma<8>(a, st) : launch_decode_mma<4>(a, st);
    if (a.pt.block == 16 && fits) {
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
