// Host interface of the fused decode projections (gemm_decode.cu): the weight-streaming
// tcgen05 GEMM of a decode step with the step that follows it folded into its tail.
#pragma once
#include "common.cuh"
#include "gemm_tc.cuh"

namespace spd {

// The step folded into the tail of each projection.  The K ranges of one output tile (splits,
// times the shards for the row-split o_proj) form one thread-block cluster: at most 8.
enum DecEpilogue {
    EPI_QKV = 0,   // a2 + a3: rstd of the attention RMSNorm, rotary embedding, q store, K/V page append
    EPI_OPROJ = 1, // a5-a7: Y_i, residual add(s), gain-scaled MLP inputs and their row sums of squares
    EPI_GATEUP = 2,// a8: rstd of the MLP RMSNorm, SwiGLU
    EPI_DOWN = 3,  // a9 + a10: shard sum (the K accumulation), output residual, next block's norm input
};

// RMSNorm is split in two: the producer of a residual stream stores x * gain (bf16, the
// next GEMM's input) and per-128-column partial sums of x^2; the consumer GEMM multiplies its
// fp32 result by rstd = rsqrt(sum / H + eps), a per-token (and per-shard) scalar that commutes
// with the projection.
struct SumSq {
    const float *part; // [tiles][groups][Mcap]
    int tiles, groups;
    long Mcap;
    int H;
    float eps;
};

struct DecGemmArgs {
    // ---- tiling --------------------------------------------------------------------
    int t_rows;            // tokens
    int num_kb, splits;    // 64-wide K blocks per batch; K splits
    int batches;           // emulated shards covered by grid x (1 when the weights are not batched)
    int w_batched, t_batched;
    int w_rows[3];         // valid rows per batch of weight i
    int n_weights;
    int z_is_plane;        // o_proj: batch z is a K range of the same output tile (the K slice of shard z)
    int l2_prefetch_kb;    // K blocks of weights per thread block pulled into L2 before the dependency wait
    int *err;
    // ---- epilogue operands -----------------------------------------------------------
    SumSq ss_in;           // QKV, GATEUP: sums of squares of the GEMM input's rows
    int rstd_per_shard;    // GATEUP in an SPD block: shard z reads group z
    // QKV
    const float2 *rope;    // [tokens][d/2] cos,sin or null
    void *q_out;           // bf16 [tokens][nq*d]
    void *k_pages, *v_pages;
    PageTable pt;
    TokMap tm;
    int n_q_heads, head_dim;
    // OPROJ, DOWN
    const float *res_in;   // fp32 [tokens][H]
    float *res_out;        // fp32 [tokens][H]
    const void *gain;      // bf16 [H] gain of the norm that follows, or null
    void *hg;              // bf16 [groups][Mcap][H]: (residual) * gain
    long hg_stride;
    float *ss_out;         // [tiles][groups][Mcap]
    long Mcap;
    int n_groups;          // OPROJ: T (SPD) or 1 (sync); DOWN: 1
    void *final_out;       // DOWN of the last block: bf16 [tokens][H], or null
    int H;
    // GATEUP
    void *act;             // bf16 [tokens][F]
    int F, Fs;
};

// Tensor maps: weights with 128-row boxes (64-row boxes for EPI_GATEUP: gate and up rows of the
// same FFN columns share a tile), tokens with a tc_token_box(true, tokens)-row box.
cudaError_t launch_gemm_decode(DecEpilogue epi, const TcMap *const *weights, const TcMap &tokens, const DecGemmArgs &g,
                               cudaStream_t st);

// Output tiles per batch of a launch.
int decode_tiles_per_batch(DecEpilogue epi, const int *w_rows, int n_weights);

// Block input -> fp32 residual stream, x * gain and its partial sums of squares (a1 of the first block).
struct PrologueArgs {
    const void *x;     // bf16 [tokens][H]
    float *res_out;    // fp32 [tokens][H]
    const void *gain;  // bf16 [H]
    void *hg;          // bf16 [tokens][H]
    float *ss_out;     // [tiles][1][Mcap]
    long Mcap;
    int M, H;
    // decode: the same launch also fills the rotary table of the step (cos, sin of pos * base^(-2j/d))
    float2 *rope_table; // [M][head_dim/2] or null
    TokMap tm;
    int head_dim;
    float rope_base;
};
cudaError_t launch_decode_prologue(const PrologueArgs &a, cudaStream_t st);

} // namespace spd
