// Causal prefill attention on the tcgen05 tensor cores (bf16, head_dim 128, 16-token pages):
// step a4 of the block for many query tokens (Sec. 3: every shard attends over its own heads).
//
// One thread block per (128 queries, query head, sequence).  Per tile of 128 cached keys:
//   S = Q K^T      tcgen05.mma, Q and K as K-major 128B-swizzled tiles (K pages land there as
//                  TMA boxes of 16 tokens x 64 dims), accumulator in tensor memory
//   P = softmax    warps 0-15: thread = (query row = TMEM lane, a quarter of the tile's 128 columns); the
//                  four threads of a row exchange their maxima through shared memory; running
//                  maximum and sums in base 2, P rounded to bf16 into a K-major swizzled tile
//   O += P V       tcgen05.mma with V as the MN-major operand: V pages are [token][dim], i.e.
//                  rows of the K dimension with the N dimension contiguous, exactly as TMA
//                  delivers them; O accumulates in tensor memory over all tiles and is rescaled
//                  there (load, multiply, store) only when the running maximum has grown by
//                  more than 2^8 since the last rescale; S of the next tile is computed meanwhile
// S is double-buffered in tensor memory, K and V tiles in two-stage rings (one for K, one for V).  19 warps:
// 0-15 softmax, 16 loads Q and the K tiles, 17 the V tiles (TMA), 18 issues the MMAs.  Every wait is bounded.
#include "common.cuh"
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace spd {

namespace {

using namespace tc;

constexpr int FQ = 128, FKV = 128, FD = 128;
constexpr int F_THREADS = 608;               // warps 0-15 softmax (four per accumulator row), 16 K loads, 17 V loads, 18 MMA
constexpr int HALF_TILE = 128 * 64 * 2;           // [128 rows][64 bf16]: one swizzled block
constexpr int TILE = 2 * HALF_TILE;               // 128 x 128 bf16
constexpr int OFF_Q = 0, OFF_KV = TILE, OFF_P = OFF_KV + 2 * 2 * TILE, OFF_RED = OFF_P + TILE, OFF_BAR = OFF_RED + 4096;
constexpr int F_SMEM = OFF_BAR + 256 + 1024;      // + alignment slack
constexpr uint32_t TMEM_COLS = 512;               // S0, S1 at columns 0 and 128, O at 256

// MN-major 128B-swizzled operand: 64 elements of the N dimension are contiguous (one 128-byte row
// per K index), 8 K rows form a 1024-byte swizzle atom; `lbo` = bytes between 64-wide N blocks,
// `sbo` = bytes between 8-row K groups.
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t smem_addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)(lbo >> 4) << 16;
    d |= (uint64_t)(sbo >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// 32 accumulator columns of this thread's row
__device__ __forceinline__ void tmem_ld32(uint32_t ta, float *v)
{
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%32];\n\t"
                 "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%33];\n\t"
                 "tcgen05.wait::ld.sync.aligned;"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(ta), "r"(ta + 16u)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// ... and back (the caller waits for the stores with tcgen05.wait::st)
__device__ __forceinline__ void tmem_st32(uint32_t ta, const float *v)
{
#pragma unroll
    for (int h = 0; h < 2; ++h)
        asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                     ::"r"(ta + 16u * h), "r"(__float_as_uint(v[16 * h + 0])), "r"(__float_as_uint(v[16 * h + 1])),
                       "r"(__float_as_uint(v[16 * h + 2])), "r"(__float_as_uint(v[16 * h + 3])), "r"(__float_as_uint(v[16 * h + 4])),
                       "r"(__float_as_uint(v[16 * h + 5])), "r"(__float_as_uint(v[16 * h + 6])), "r"(__float_as_uint(v[16 * h + 7])),
                       "r"(__float_as_uint(v[16 * h + 8])), "r"(__float_as_uint(v[16 * h + 9])), "r"(__float_as_uint(v[16 * h + 10])),
                       "r"(__float_as_uint(v[16 * h + 11])), "r"(__float_as_uint(v[16 * h + 12])), "r"(__float_as_uint(v[16 * h + 13])),
                       "r"(__float_as_uint(v[16 * h + 14])), "r"(__float_as_uint(v[16 * h + 15]))
                     : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(uint32_t *)&v;
}

__global__ void __launch_bounds__(F_THREADS, 1) prefill_attention_umma_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                                               const __grid_constant__ CUtensorMap tm_k,
                                                                               const __grid_constant__ CUtensorMap tm_v,
                                                                               const __grid_constant__ AttnArgs a)
{
    extern __shared__ uint8_t fa_raw[];
    const uint32_t base = (smem_u32(fa_raw) + 1023u) & ~1023u;
    uint8_t *gen = fa_raw + (base - smem_u32(fa_raw));
    const uint32_t sQ = base + OFF_Q, bars = base + OFF_BAR;
    auto sK = [&](int s) { return base + OFF_KV + (uint32_t)s * 2 * TILE; };
    auto sV = [&](int s) { return base + OFF_KV + (uint32_t)s * 2 * TILE + TILE; };
    const uint32_t sP = base + OFF_P;
    const uint32_t q_full = bars;
    // K and V tiles have rings of their own: a K slot is free once S of its tile is computed, long before the
    // tile's V slot, so the next K tile is on its way a whole tile earlier
    auto k_full = [&](int s) { return bars + 8u * (1 + s); };
    auto v_full = [&](int s) { return bars + 8u * (3 + s); };
    auto k_empty = [&](int s) { return bars + 8u * (5 + s); };
    auto v_empty = [&](int s) { return bars + 8u * (7 + s); };
    auto s_full = [&](int s) { return bars + 8u * (9 + s); };
    auto p_ready = [&](int s) { return bars + 8u * (11 + s); };
    auto o_full = [&](int s) { return bars + 8u * (13 + s); };
    uint32_t *tmem_slot = (uint32_t *)(gen + OFF_BAR + 128);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * FQ, hq = blockIdx.y, bi = blockIdx.z; // longest rows first
    const int ns = a.tm.ns, s0 = a.tm.s0, b = a.tm.b0 + bi;
    const int kvh = hq / (a.n_q_heads / a.pt.n_kv_heads);
    const int q_rows = min(FQ, ns - q0);
    const int kv_len = s0 + q0 + q_rows; // keys 0 .. last query position of the tile
    const int n_tiles = (kv_len + FKV - 1) / FKV;

    pdl_launch_dependents();
    if (threadIdx.x == 0) stamp_entry(a.stamp);
    // The two load warps set up the barriers themselves and only ARRIVE at the set-up barrier, so that the first
    // tiles are on their way while the others still wait for the tensor-memory allocation.
    uint32_t tmem = 0;
    if (warp == 16 || warp == 17) {
        if (lane == 0) {
            *abort_flag = 0;
            if (warp == 16) {
                mbar_init(q_full, 1);
                for (int s = 0; s < 2; ++s) {
                    mbar_init(k_full(s), 1);
                    mbar_init(k_empty(s), 1);
                    mbar_init(s_full(s), 1);
                    mbar_init(p_ready(s), 16);
                    mbar_init(o_full(s), 1);
                }
            } else {
                for (int s = 0; s < 2; ++s) {
                    mbar_init(v_full(s), 1);
                    mbar_init(v_empty(s), 1);
                }
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        asm volatile("bar.arrive 2, 608;" ::: "memory");
    } else {
        if (warp == 18) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("bar.sync 2, 608;" ::: "memory");
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tmem = *tmem_slot;
    }
    pdl_wait();

    if (warp == 16 || warp == 17) {
        // Warp 16 loads Q and the K tiles, warp 17 the V tiles.  The 16 boxes of a tile (8 pages x 2 halves of the
        // head) are one per lane: the eight page lookups of a tile go out together, and those of the next tile
        // before this one's ring slot is awaited.
        const bool is_v = warp == 17;
        const CUtensorMap *map = is_v ? &tm_v : &tm_k;
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
            if (!is_v) {
                asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_q) : "memory");
                mbar_expect_tx(q_full, TILE);
                for (int h = 0; h < 2; ++h) tma_load_3d(sQ + h * HALF_TILE, &tm_q, hq * FD + h * 64, bi * ns + q0, 0, q_full);
            }
        }
        const int pg = (lane >> 1) & 7, h = lane & 1;
        const int32_t *bt = a.pt.block_table + (long)b * a.pt.max_pages;
        auto lookup = [&](int j) {
            // pages past the last key are never looked up: their rows (masked keys) repeat the tile's first page
            const int tkn = j * FKV + pg * 16;
            int page = bt[(tkn < kv_len ? tkn : j * FKV) / 16];
            if (page < 0 || page >= a.pt.n_pages) { atomicOr(a.err, ERR_PAGE_RANGE); page = 0; }
            return page;
        };
        int page_next = n_tiles > 0 ? lookup(0) : 0;
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1, page = page_next;
            if (j + 1 < n_tiles) page_next = lookup(j + 1);
            bool ok = true;
            if (j >= 2) ok = mbar_wait(is_v ? v_empty(s) : k_empty(s), ((j >> 1) - 1) & 1, a.err, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            const uint32_t full = is_v ? v_full(s) : k_full(s);
            if (lane == 0) mbar_expect_tx(full, TILE);
            __syncwarp();
            if (lane < 16)
                tma_load_3d((is_v ? sV(s) : sK(s)) + h * HALF_TILE + pg * 2048, map, h * 64, (page * a.pt.n_kv_heads + kvh) * 16, 0, full);
        }
        __syncwarp();
    } else if (warp == 18) {
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc(FKV);                // Q, K: both K-major
            constexpr uint32_t idesc_o = make_idesc(FD) | (1u << 16);    // P K-major, V MN-major
            auto issue_s = [&](int j) {
                const int s = j & 1;
                const uint32_t acc = tmem + (uint32_t)s * 128u;
#pragma unroll
                for (int kk = 0; kk < FD / UMMA_K; ++kk) {
                    const uint64_t da = make_desc(sQ + (kk >> 2) * HALF_TILE) + (uint64_t)((kk & 3) * UMMA_K * 2 / 16);
                    const uint64_t db = make_desc(sK(s) + (kk >> 2) * HALF_TILE) + (uint64_t)((kk & 3) * UMMA_K * 2 / 16);
                    umma(acc, da, db, idesc_s, kk > 0 ? 1u : 0u);
                }
                umma_commit(s_full(s));
                umma_commit(k_empty(s));
            };
            bool ok = mbar_wait(q_full, 0, a.err, abort_flag) && mbar_wait(k_full(0), 0, a.err, abort_flag);
            if (ok) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                issue_s(0);
            }
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int s = j & 1;
                if (j + 1 < n_tiles) {
                    if (!mbar_wait(k_full(s ^ 1), ((j + 1) >> 1) & 1, a.err, abort_flag)) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    issue_s(j + 1);
                }
                if (!mbar_wait(p_ready(s), (j >> 1) & 1, a.err, abort_flag)) break;
                if (!mbar_wait(v_full(s), (j >> 1) & 1, a.err, abort_flag)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem + 256u; // O accumulates over the tiles
#pragma unroll
                for (int kk = 0; kk < FKV / UMMA_K; ++kk) {
                    const uint64_t da = make_desc(sP + (kk >> 2) * HALF_TILE) + (uint64_t)((kk & 3) * UMMA_K * 2 / 16);
                    const uint64_t db = make_desc_mn(sV(s) + kk * UMMA_K * 128, HALF_TILE, 1024);
                    umma(acc, da, db, idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(o_full(0));
                umma_commit(v_empty(s));
            }
        }
        __syncwarp();
    } else {
        // thread = (row, quarter): columns quarter*32 .. +31 of S (keys) and of O (head dims) of query row `row`
        const int row = threadIdx.x & 127, qt = threadIdx.x >> 7;
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const int pos_q = row < q_rows ? s0 + q0 + row : -1;
        const float sc = rsqrtf((float)FD) * 1.4426950408889634f;
        float *red = (float *)(gen + OFF_RED); // [2 tile parities][4 quarters][128 rows]
        // m_used: the maximum the accumulated O (in tensor memory) and the row sum are relative to.  It follows the
        // true running maximum lazily: O and the sum are only rescaled when the maximum has grown by more than
        // 2^rescale_log2 since (default 8: P stays below 2^8, exact enough in bf16 and far from fp32 overflow), which
        // is rare after the first tiles; 0 follows the maximum exactly.
        float m_used = -INFINITY, l_run = 0.f;
        bool ok = true;
        auto ex2 = [](float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; };
        const uint32_t t_o = tmem + lane_off + 256u + (uint32_t)qt * 32u;
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1;
            if (ok && !mbar_wait(s_full(s), (j >> 1) & 1, a.err, abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok); // warp-uniform: the tensor-memory accesses below are warp-wide
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int key0 = j * FKV + qt * 32;
            // keys of this tile beyond the row's own position are masked (only tiles that reach the diagonal)
            const bool need_mask = j * FKV + FKV - 1 > s0 + q0 || pos_q < 0;
            float sv[32];
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
            if (ok) {
                tmem_ld32(tmem + lane_off + (uint32_t)s * 128u + (uint32_t)qt * 32u, sv);
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    if (need_mask) {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (key0 + i + e > pos_q) sv[i + e] = -INFINITY;
                    }
                    mx0 = fmaxf(mx0, sv[i]); mx1 = fmaxf(mx1, sv[i + 1]); mx2 = fmaxf(mx2, sv[i + 2]); mx3 = fmaxf(mx3, sv[i + 3]);
                }
            }
            // the four threads of a row exchange the maxima of their quarters (sc > 0: maxima of the scaled scores)
            red[(s * 4 + qt) * 128 + row] = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sc;
            asm volatile("bar.sync 1, 512;" ::: "memory");
            float mx = m_used;
#pragma unroll
            for (int t = 0; t < 4; ++t) mx = fmaxf(mx, red[(s * 4 + t) * 128 + row]);
            float factor = 1.f;
            if (m_used == -INFINITY) m_used = mx;                 // nothing accumulated yet
            else if (mx > m_used + a.rescale_log2) { factor = ex2(m_used - mx); m_used = mx; }
            const float mbase = m_used == -INFINITY ? 0.f : m_used;
            float rs0 = 0.f, rs1 = 0.f;
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const float p0 = ex2(sv[i] * sc - mbase), p1 = ex2(sv[i + 1] * sc - mbase);
                rs0 += p0;
                rs1 += p1;
                pk[i >> 1] = pack2(p0, p1);
            }
            l_run = l_run * factor + (rs0 + rs1);
            // the previous P V product has read the P tile and settled O
            if (ok && j > 0 && !mbar_wait(o_full(0), (j - 1) & 1, a.err, abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (__any_sync(0xffffffffu, factor != 1.f) && ok) {
                float v[32];
                tmem_ld32(t_o, v);
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] *= factor;
                tmem_st32(t_o, v);
            }
            if (ok) {
                uint8_t *prow = gen + OFF_P + (qt >> 1) * HALF_TILE + row * 128;
#pragma unroll
                for (int q = 0; q < 4; ++q) // 16-byte chunk (qt & 1) * 4 + q of the row's 64-key block, swizzled by row
                    *(uint4 *)(prow + ((((qt & 1) * 4 + q) ^ (row & 7)) << 4)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(p_ready(s)) : "memory");
        }
        float o_acc[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) o_acc[i] = 0.f;
        if (ok && n_tiles > 0) {
            if (!mbar_wait(o_full(0), (n_tiles - 1) & 1, a.err, abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (ok) tmem_ld32(t_o, o_acc);
        }
        // the row's sum is the sum over its four threads (all ran on the same maxima)
        if (!ok) l_run = 0.f;
        asm volatile("bar.sync 1, 512;" ::: "memory");
        red[qt * 128 + row] = l_run;
        asm volatile("bar.sync 1, 512;" ::: "memory");
        const float l_tot = (red[row] + red[128 + row]) + (red[256 + row] + red[384 + row]);
        if (ok && row < q_rows) {
            const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
            bf16 *dst = (bf16 *)a.out + ((long)(bi * ns + q0 + row) * a.n_q_heads + hq) * FD + qt * 32;
#pragma unroll
            for (int i = 0; i < 32; i += 8)
                *(uint4 *)(dst + i) = make_uint4(pack2(o_acc[i] * inv, o_acc[i + 1] * inv), pack2(o_acc[i + 2] * inv, o_acc[i + 3] * inv),
                                                 pack2(o_acc[i + 4] * inv, o_acc[i + 5] * inv), pack2(o_acc[i + 6] * inv, o_acc[i + 7] * inv));
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) stamp_exit(a.stamp);
    if (warp == 18) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

} // namespace

// Tensor maps: q as [tokens][n_q_heads * 128] with a 64 x 128 box; K / V pages as
// [n_pages * n_kv_heads * 16 rows][128] with a 64 x 16 box (128-byte swizzle).
cudaError_t launch_prefill_attention_umma(const AttnArgs &a, cudaStream_t st)
{
    if (a.head_dim != FD || a.pt.block != 16 || !a.q_map || !a.k_map || !a.v_map || a.tm.decode || a.tm.ns <= 0 || a.M % a.tm.ns)
        return cudaErrorInvalidValue;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(prefill_attention_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    dim3 grid((a.tm.ns + FQ - 1) / FQ, a.n_q_heads, a.M / a.tm.ns);
    return launch_kernel(prefill_attention_umma_kernel, grid, dim3(F_THREADS), F_SMEM, st, 0, *(const CUtensorMap *)a.q_map,
                         *(const CUtensorMap *)a.k_map, *(const CUtensorMap *)a.v_map, a);
}

} // namespace spd
