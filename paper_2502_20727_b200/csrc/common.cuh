// Shared device helpers and host-side launch declarations of the SPD block library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spd {

typedef __nv_bfloat16 bf16;

// Bits of the device error flag (read back by spd_device_error / the next call).
enum : int {
    ERR_PAGE_RANGE = 1,   // block-table entry outside [0, n_pages)
    ERR_CAPACITY = 2,     // position beyond the block-table row / max_context
    ERR_WAIT_TIMEOUT = 4, // a bounded mbarrier wait gave up
    ERR_PEER_TIMEOUT = 8, // a bounded wait for another rank's partial sums gave up
};

// Remember a failing CUDA call for spd_last_cuda_error() (per thread); used by every file that returns SPD_ECUDA.
void note_cuda_error(cudaError_t e);
// Streaming multiprocessors of the current device (queried once per device; 148, the B200's count, when there is
// no device to ask, as in host-only calls).  Launch shapes and split counts are sized from it.
int sm_count();

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// Programmatic dependent launch.  Every kernel of the library signals at its very top that the
// next kernel in the stream may be scheduled, and waits for the completion (and memory
// visibility) of the previous one before it touches anything a predecessor wrote or may still
// read.  Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch stamps (optional; spd_timeline_*).  A launch may be handed a slot of two 64-bit words preset to all
// ones.  One thread of every block lowers word 0 to the global nanosecond timer when the block starts and word 1
// to the timer's complement when it ends, so that afterwards word 0 is the launch's earliest block start and
// ~word 1 its latest block end - taken inside a replayed graph, with nothing inserted between the launches.
__device__ __forceinline__ void stamp_entry(unsigned long long *slot)
{
    if (!slot) return;
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    atomicMin(slot, t);
}
__device__ __forceinline__ void stamp_exit(unsigned long long *slot)
{
    if (!slot) return;
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    atomicMin(slot + 1, ~t);
}

// Launch with the programmatic-stream-serialization attribute (and an optional cluster size).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 int cluster_x, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    int n = 0;
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = (unsigned)cluster_x;
        at[n].val.clusterDim.y = 1;
        at[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The same with a thread-block cluster along grid z.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_z(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                   int cluster_z, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = 1;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = (unsigned)(cluster_z > 1 ? cluster_z : 1);
    cfg.attrs = at;
    cfg.numAttrs = cluster_z > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Where the tokens of a launch sit in their sequences.
//   prefill chunk: token m = bi * ns + si is position s0 + si of sequence b0 + bi
//   decode       : token m is position seq_lens[m] of sequence m
struct TokMap {
    int decode;
    int b0, ns, s0;
    const int32_t *seq_lens;
    __device__ __forceinline__ void locate(int m, int &b, int &pos) const
    {
        if (decode) { b = m; pos = seq_lens[m]; }
        else { b = b0 + m / ns; pos = s0 + m % ns; }
    }
};

struct PageTable {
    const int32_t *block_table; // [B, max_pages]
    int max_pages, n_pages, block, n_kv_heads;
};

// ---- host-side launchers (defined in the .cu files) ----------------------------------

// C[z][m][n] (+)= sum_k A_s[m][k] * W[s*n_per_shard + n][k] over split z's K range.
struct GemmProblem {
    const void *A;          // [M, K] row-major, leading dimension lda (elements)
    long lda;
    long a_shard_stride;    // elements between the A operands of consecutive shards (0: shared)
    const void *W;          // [n_shards * n_per_shard, K] row-major, leading dimension ldw
    long ldw;
    float *C;               // fp32 [splits][M][ldc]; column = s * n_per_shard + n
    long ldc;
    long c_split_stride;    // elements between split planes
    int M, n_per_shard, n_shards, K;
    int splits;             // K is cut into `splits` equal ranges of k_per_split
    int k_per_split;
};
template <typename T> cudaError_t launch_gemm_simt(const GemmProblem &p, cudaStream_t st);

struct NormArgs {
    const void *x_in;     // storage dtype [M,H] (first layer) or null
    const float *res_in;  // fp32 [M,H] or null
    const float *part;    // fp32 [n_groups * per_group][M][H] partial sums, or null
    long part_stride;     // elements between partial planes
    int n_groups;         // 1: everything is summed; T: SPD, one group per shard
    int per_group;        // partial planes per group
    float *res_out;       // fp32 [M,H]: res + all partials (may alias res_in)
    void *h_out;          // storage [n_groups][M][H] (plane stride h_stride): norm(res + group)*g ; or null
    long h_stride;
    const void *gain;     // storage [H] or null (then no norm output)
    void *final_out;      // storage [M,H] copy of res_out, or null
    int M, H;
    float eps;
    // block with bias (Sec. 4.1.2): `bias` (storage [H], the unsplittable bias of the row-split layer whose
    // partials these are) is added to every group's residual and once to res_out; `shift` non-null turns the
    // RMSNorm into a LayerNorm with that shift
    const void *bias, *shift;
};
template <typename T> cudaError_t launch_residual_norm(const NormArgs &a, cudaStream_t st);

// wg[n] = sum_k g[k] W[n][k], wb[n] = sum_k beta[k] W[n][k] + b[n] (b may be null); W bf16 [N][K] (block with bias, Sec. 4.1.2)
cudaError_t launch_ln_fold(const void *W, int N, int K, const void *g, const void *beta, const void *b, float *wg, float *wb, cudaStream_t st);

cudaError_t launch_rope_table(float2 *table, TokMap tm, int M, int head_dim, float base, cudaStream_t st,
                              unsigned long long *stamp = nullptr);

struct RopeKvArgs {
    const float *qkv;     // fp32 [splits][M][ldq]: columns [q | k | v]
    long ldq, split_stride;
    int splits;
    const float2 *table;  // [M][d/2] cos,sin
    void *q_out;          // storage [M, nq*d]
    void *k_pages, *v_pages;
    PageTable pt;
    TokMap tm;
    int M, n_q_heads, head_dim;
    int use_rope;
    int *err;
    const void *bq, *bk, *bv; // storage [nq*d], [nkv*d], [nkv*d] or null: biases of the column-split projections
};
template <typename T> cudaError_t launch_rope_kv(const RopeKvArgs &a, cudaStream_t st);

struct SiluMulArgs {
    const float *gate, *up; // fp32 [splits][M][ld]
    long ld, split_stride;
    int splits;
    void *act;              // storage [M,F]
    int M, F;
    const void *bias;       // storage [F] or null
    int relu;               // 1: act = relu(gate + bias) (fc1 of the block with bias; `up` is not read)
};
template <typename T> cudaError_t launch_silu_mul(const SiluMulArgs &a, cudaStream_t st);

struct AttnArgs {
    const void *q;          // storage [M, nq*d]
    const void *k_pages, *v_pages;
    PageTable pt;
    TokMap tm;
    void *out;              // storage [M, nq*d]
    int M, n_q_heads, head_dim;
    // decode only
    int B, splits, max_context;
    float *part_o;          // fp32 [B][nq][splits][d]
    float *part_ml;         // fp32 [B][nq][splits][2]
    int *counters;          // [B][nq] zero-initialised arrival counters (split merge)
    int *err;
    // optional (decode, bf16, head_dim 128, 16-token pages): tensor maps over the K and V pages seen as
    // [n_pages * n_kv_heads * 16 rows][head_dim], box 64 x 16, 128-byte swizzle (host pointers to CUtensorMap)
    const void *k_map, *v_map;
    // optional (prefill, same conditions): tensor map over q as [tokens][n_q_heads * head_dim], box 64 x 128
    const void *q_map;
    // ... and how far (in powers of two) the running row maximum may grow before the accumulated output is rescaled
    float rescale_log2;
    int cluster_merge;      // set by the launcher: the splits of a (sequence, head tile) are one thread-block cluster
    unsigned long long *stamp; // launch stamp slot or null
};
// Paged decode attention with 16-token pages: query heads per thread block for a GQA group
// size, and the most pages one block may be given (the host picks splits accordingly).
constexpr int DECODE_MAX_PAGES_PER_BLOCK = 512;
inline int decode_heads_per_block(int group) { return group % 4 == 0 ? 4 : (group % 2 == 0 ? 2 : 1); }
// ... and of the tensor-core variant, which serves grouped-query attention with group sizes 4, 8, ...
inline bool decode_uses_mma(int group, int head_dim, int dtype_bf16, int kv_block) { return dtype_bf16 && head_dim == 128 && kv_block == 16 && group % 4 == 0; }
inline int decode_heads_per_block_mma(int group) { return group % 8 == 0 ? 8 : 4; }
template <typename T> cudaError_t launch_prefill_attention(const AttnArgs &a, cudaStream_t st);
cudaError_t launch_prefill_attention_umma(const AttnArgs &a, cudaStream_t st); // attention_prefill_tc.cu
template <typename T> cudaError_t launch_decode_attention(const AttnArgs &a, cudaStream_t st);

// head grouping measurements (head_grouping.cu)
template <typename T>
cudaError_t launch_head_scores(const void *q, const void *k_pages, PageTable pt, int b0, int S, int n_seq, int n_q_heads, int d,
                               float *sigma, int *err, cudaStream_t st);
cudaError_t launch_head_distance(const float *sigma, long len, int n_heads, float *dist, cudaStream_t st);

// part[b] = sum over block b's slice of (a - r)^2, fixed order (strategy.cu)
cudaError_t launch_sq_diff(const void *a, const void *r, long n, int dtype_bf16, float *part, int n_blocks, cudaStream_t st);

} // namespace spd
