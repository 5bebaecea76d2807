// bf16 projection GEMM on the 5th-generation tensor cores: TMA (cp.async.bulk.tensor, no
// multicast) -> 128B-swizzled shared-memory ring -> tcgen05.mma (cta_group::1, kind::f16)
// with the fp32 accumulator in tensor memory -> tcgen05.ld epilogue.
//
// One launch computes, for every batch z (an emulated TP shard, or a single batch) and K-split s,
//     C[z, s][m][col0(z) + n] = sum_{k in split s} A_z[m][k] * W_z[n][k]
// Both operands are K-major ([rows, K] row-major), so no transposes are needed for
// activations x torch.nn.Linear weights.  Batching over z is how the shard structure of the
// SPD block (Sec. 4.1.1) is expressed: per-shard K-slices of the row-split o_proj whose
// planes Y_z are kept apart, and per-shard MLP inputs for the column-split gate/up.
//
// SWAP = true  (decode, few tokens): the 128-row MMA "M" side holds WEIGHT rows and the tokens
//               sit on the N side (BN = 16..64), so a CTA streams a 128 x K weight slab.
// SWAP = false (prefill): tokens on the M side, BN weight rows on the N side.
#include "common.cuh"
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace spd {

namespace {

using namespace tc;

template <int BN> struct Cfg {
    static constexpr int STAGES = (BN <= 64) ? 5 : 3;
    static constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int TMEM_COLS = BN < 32 ? 32 : BN;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN, bool SWAP>
__global__ void __launch_bounds__(128) gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_w0, const __grid_constant__ CUtensorMap tm_w1,
                                                      const __grid_constant__ CUtensorMap tm_w2,
                                                      const __grid_constant__ CUtensorMap tm_t, TcGemmArgs g)
{
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + C::STAGES * C::STAGE_BYTES; // full[S], empty[S], tmem_full
    uint32_t *tmem_slot = (uint32_t *)(gen_base + C::STAGES * C::STAGE_BYTES + 8 * (2 * C::STAGES + 1));
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (C::STAGES + s); };
    const uint32_t tmem_full_bar = bars + 8u * (2 * C::STAGES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // tile coordinates: x -> (batch z, weight tile), y -> token tile, z -> split
    // (a launch may cover up to three weight matrices that share the token operand: Q|K|V, gate|up)
    const int z = blockIdx.x / g.w_tiles_per_batch;
    const int wt = blockIdx.x % g.w_tiles_per_batch;
    const int wi = (wt >= g.tile_start[2]) ? 2 : ((wt >= g.tile_start[1]) ? 1 : 0);
    const CUtensorMap *tm_w = wi == 0 ? &tm_w0 : (wi == 1 ? &tm_w1 : &tm_w2);
    const int w_rows = g.w_rows[wi];
    const int w_row0 = (wt - g.tile_start[wi]) * (SWAP ? BM : BN);
    const int t_row0 = blockIdx.y * (SWAP ? BN : BM);
    const int split = blockIdx.z;
    const int kb_begin = (int)((long)g.num_kb * split / g.splits);
    const int kb_end = (int)((long)g.num_kb * (split + 1) / g.splits);
    const int n_kb = kb_end - kb_begin;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(tm_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_t) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = *tmem_slot;

    // A side = 128-row operand, B side = BN-row operand
    const int a_row0 = SWAP ? w_row0 : t_row0, b_row0 = SWAP ? t_row0 : w_row0;
    const int a_z = SWAP ? (g.w_batched ? z : 0) : (g.t_batched ? z : 0);
    const int b_z = SWAP ? (g.t_batched ? z : 0) : (g.w_batched ? z : 0);

    if (warp == 0 && lane == 0) {
        // TMA producer.  The weight tiles do not depend on the preceding kernel, so the first
        // ring of them is requested before waiting for it (programmatic dependent launch): the
        // weight stream of this GEMM overlaps the tail of whatever ran before.
        const int pre = n_kb < C::STAGES ? n_kb : C::STAGES;
        for (int i = 0; i < pre; ++i) {
            mbar_expect_tx(full_bar(i), C::STAGE_BYTES);
            const uint32_t sa = base + i * C::STAGE_BYTES, sb = sa + C::A_BYTES;
            const int kx = (kb_begin + i) * BK;
            if (SWAP) tma_load_3d(sa, tm_w, kx, a_row0, a_z, full_bar(i));
            else tma_load_3d(sb, tm_w, kx, b_row0, b_z, full_bar(i));
        }
        pdl_wait();
        for (int i = 0; i < n_kb; ++i) {
            const int s = i % C::STAGES;
            const uint32_t sa = base + s * C::STAGE_BYTES, sb = sa + C::A_BYTES;
            const int kx = (kb_begin + i) * BK;
            if (i >= pre) {
                if (!mbar_wait(empty_bar(s), ((i / C::STAGES) & 1) ^ 1, g.err, abort_flag)) break;
                mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
                if (SWAP) tma_load_3d(sa, tm_w, kx, a_row0, a_z, full_bar(s));
                else tma_load_3d(sb, tm_w, kx, b_row0, b_z, full_bar(s));
            }
            if (SWAP) tma_load_3d(sb, &tm_t, kx, b_row0, b_z, full_bar(s));
            else tma_load_3d(sa, &tm_t, kx, a_row0, a_z, full_bar(s));
        }
    } else if (warp == 1 && lane == 0) {
        // MMA issuer
        constexpr uint32_t idesc = make_idesc(BN);
        bool ok = true;
        for (int i = 0; i < n_kb && ok; ++i) {
            const int s = i % C::STAGES;
            ok = mbar_wait(full_bar(s), (i / C::STAGES) & 1, g.err, abort_flag);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa = base + s * C::STAGE_BYTES, sb = sa + C::A_BYTES;
            const uint64_t da = make_desc(sa), db = make_desc(sb);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
                umma(tmem_acc, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                     (i > 0 || k > 0) ? 1u : 0u);
            umma_commit(empty_bar(s)); // frees the stage once these MMAs have read it
        }
        umma_commit(tmem_full_bar);    // arrives when every MMA above has completed
    }
    __syncwarp();
    pdl_wait(); // the output buffer may still be read by an earlier kernel until this returns

    // epilogue: warp w owns TMEM lanes [32w, 32w+32)
    const bool acc_ok = (n_kb > 0) && mbar_wait(tmem_full_bar, 0, g.err, abort_flag);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    __syncwarp();
    float *Cz = g.C + g.c_off[wi] + (long)z * g.c_batch_stride + (long)split * g.c_split_stride;
    const int row = warp * 32 + lane; // accumulator row = TMEM lane
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 16) {
        float v[16];
        if (acc_ok) tmem_ld16(tmem_acc + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
        else {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
        }
        if (SWAP) {
            // row = weight row n, columns = tokens m
            const int n = w_row0 + row;
            if (n < w_rows) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int m = t_row0 + c0 + j;
                    if (m < g.t_rows) Cz[(long)m * g.ldc + n] = v[j];
                }
            }
        } else {
            // row = token m, columns = weight rows n
            const int m = t_row0 + row;
            if (m < g.t_rows) {
                float *dst = Cz + (long)m * g.ldc + w_row0 + c0;
                if (w_row0 + c0 + 16 <= w_rows && ((((uintptr_t)dst) & 15) == 0)) {
#pragma unroll
                    for (int j = 0; j < 16; j += 4) *(float4 *)(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (w_row0 + c0 + j < w_rows) dst[j] = v[j];
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(C::TMEM_COLS) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

template <int BN, bool SWAP>
cudaError_t launch_cfg(const CUtensorMap *const *tw, const CUtensorMap &tt, const TcGemmArgs &g, dim3 grid, cudaStream_t st)
{
    using C = Cfg<BN>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, SWAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    return launch_kernel(gemm_tc_kernel<BN, SWAP>, grid, dim3(128), C::SMEM_BYTES, st, 0, *tw[0], *tw[1], *tw[2], tt, g);
}

} // namespace

// rows x K bf16 matrix (row stride ld elements), optionally `batches` of them, as a 3-D map
// {K, rows, batches} with a {64, box_rows, 1} box and the 128-byte swizzle.
int make_operand_map(TcMap *out, const void *ptr, long k_inner, long rows, long batches, long ld_elems,
                     long batch_stride_elems, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return -1;
    if (((uintptr_t)ptr & 15) || (ld_elems * 2) % 16 || (batches > 1 && (batch_stride_elems * 2) % 16)) return -2;
    cuuint64_t dims[3] = {(cuuint64_t)k_inner, (cuuint64_t)rows, (cuuint64_t)(batches < 1 ? 1 : batches)};
    cuuint64_t strides[2] = {(cuuint64_t)ld_elems * 2, (cuuint64_t)(batches > 1 ? batch_stride_elems : ld_elems * rows) * 2};
    cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn((CUtensorMap *)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -3;
}

// A paged K or V cache ([pages][kv heads][16 tokens][128 dims] bf16, `rows` token rows in all) as a 3-D map {64 dims,
// rows, 2 halves of the head dimension} with a {64, 16, 2} box: one copy brings a (page, head)'s 4 KB in as two
// 16 x 64 tiles in the 128-byte swizzle, low half of the head dimension first.
int make_page_map(TcMap *out, const void *ptr, long rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return -1;
    if ((uintptr_t)ptr & 15) return -2;
    cuuint64_t dims[3] = {64, (cuuint64_t)rows, 2};
    cuuint64_t strides[2] = {256, 128};
    cuuint32_t box[3] = {64, 16, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn((CUtensorMap *)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -3;
}

int tc_token_box(bool swap, int tokens)
{
    if (!swap) return BM;
    return tokens <= 16 ? 16 : (tokens <= 32 ? 32 : 64);
}
int tc_weight_box(bool swap) { return BM; }

cudaError_t launch_gemm_tc(const TcMap *const *weights, int n_weights, const TcMap &tokens, const TcGemmArgs &g,
                           bool swap, cudaStream_t st)
{
    if (n_weights < 1 || n_weights > 3) return cudaErrorInvalidValue;
    if (g.t_rows <= 0) return cudaSuccess;
    if (g.splits < 1 || g.splits > g.num_kb) return cudaErrorInvalidValue;
    const CUtensorMap *tw[3];
    for (int i = 0; i < 3; ++i) tw[i] = (const CUtensorMap *)weights[i < n_weights ? i : 0];
    const CUtensorMap &tt = *(const CUtensorMap *)&tokens;
    const int w_tile = swap ? BM : 128;
    TcGemmArgs a = g;
    int tiles = 0;
    for (int i = 0; i < 3; ++i) {
        a.tile_start[i] = tiles;
        if (i < n_weights) {
            if (g.w_rows[i] <= 0) return cudaErrorInvalidValue;
            tiles += (g.w_rows[i] + w_tile - 1) / w_tile;
        } else {
            a.tile_start[i] = 1 << 30; // never selected
            a.w_rows[i] = 0;
            a.c_off[i] = 0;
        }
    }
    a.w_tiles_per_batch = tiles;
    if (swap) {
        const int bn = tc_token_box(true, g.t_rows);
        dim3 grid(tiles * g.batches, (g.t_rows + bn - 1) / bn, g.splits);
        switch (bn) {
        case 16: return launch_cfg<16, true>(tw, tt, a, grid, st);
        case 32: return launch_cfg<32, true>(tw, tt, a, grid, st);
        default: return launch_cfg<64, true>(tw, tt, a, grid, st);
        }
    }
    dim3 grid(tiles * g.batches, (g.t_rows + BM - 1) / BM, g.splits);
    return launch_cfg<128, false>(tw, tt, a, grid, st);
}

} // namespace spd
