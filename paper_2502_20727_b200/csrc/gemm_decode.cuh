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
    EPI_RESID_TP = 4, // o_proj / down of a rank that holds one shard: the shard sum is an exchange with the other ranks
};

constexpr int TP_MAX_RANKS = 8;
constexpr int TP_FLAG_RANGES = 8; // flag words per (tile, source rank): one per K range of the source's cluster

// Tensor-parallel execution proper (Sec. 3): every rank of the group holds one shard and owns a
// region of device memory that its peers can write.  Batch z of a launch is local rank z (one per
// launch on a real group; all T when one GPU executes every rank), and every rank-private pointer
// of the launch is that of local rank 0, rank z's lying z_stride bytes further on.
//
// A shard sum (sync-point) is a one-shot exchange folded into the tail of the projection whose
// output it adds up: each rank writes its fp32 partial rows into every rank's receive planes
// (plane = source rank), publishes the step number in one flag word per (tile, source, K range)
// on every rank, waits - with a time limit - until its own flags show this step for all sources,
// and adds the T planes in rank order, so that all ranks hold bit-identical sums.  Two receive
// buffers alternate between consecutive exchanges; kernel boundaries order their reuse.
struct TpArgs {
    int on;                // 0: not a rank-mode launch
    int T, rank_base;      // group size; group rank of local rank 0
    long z_stride;         // bytes between the regions of consecutive local ranks
    long out_stride;       // bytes between the final outputs of consecutive local ranks
    int exchange;          // 1: the partial rows are summed over the group; 0: they stay local (SPD o_proj)
    int buf;               // receive buffer (0 / 1) of this exchange; consecutive exchanges alternate
    long buf_bytes, src_bytes; // one receive buffer ([T][Mcap][H] fp32); one source plane of it
    char *rx[TP_MAX_RANKS];        // rank j's receive buffers (buffer 0 first)
    unsigned *flags[TP_MAX_RANKS]; // rank j's flag words of this exchange: [tile][token tile][source][TP_FLAG_RANGES]
    const unsigned *step;  // step number (> 0, same on all ranks)
    unsigned long long wait_ns; // how long a rank waits for its peers' rows before it gives up (error bit 8)
    const float *addend;   // fp32 [Mcap][H] added to the partial before the exchange (Y_i of an SPD block), or null
    float *ysave;          // fp32 [Mcap][H]: the partial is kept here (Y_i), or null
};

// RMSNorm is split in two: the producer of a residual stream stores x * gain (bf16, the
// next GEMM's input) and per-128-column partial sums of x^2; the consumer GEMM multiplies its
// fp32 result by rstd = rsqrt(sum / H + eps), a per-token (and per-shard) scalar that commutes
// with the projection.
// For the block with bias (Sec. 4.1.2) the norm is a LayerNorm, u = (x - mean) * rstd * g + beta, and commutes the same
// way once two vectors per projection are known: u W^T + b = rstd * ((x * g) W^T - mean * wg) + wb with
// wg[n] = sum_k g[k] W[n][k] and wb[n] = sum_k beta[k] W[n][k] + b[n] (computed once, when the context is created).
// The producer then also stores partial row sums of x (`sum`, same layout as `part`).
struct SumSq {
    const float *part; // [tiles][groups][Mcap]
    int tiles, groups;
    long Mcap;
    int H;
    float eps;
    const float *sum;  // partial row sums, same layout, or null (RMSNorm)
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
    int ring_stages;       // stages of the operand ring (3, 4; 5 at 16-token tiles); 0 = chosen per launch
    int planes_per_block;  // z_is_plane with splits == 1: shard slices one block computes one after the other, each into
                           // its own accumulator columns (1 or 2; 0 = two where one per block would not be resident at once)
    int *err;
    unsigned long long *stamp; // launch stamp slot or null
    // ---- epilogue operands -----------------------------------------------------------
    SumSq ss_in;           // QKV, GATEUP: sums of squares of the GEMM input's rows
    int rstd_per_shard;    // GATEUP in an SPD block: shard z reads group z
    // block with bias: LayerNorm folded into the tail (see SumSq): fp32 vectors over the launch's weight rows (QKV: q, k, v
    // rows one after the other; GATEUP: the rows of fc1), or null
    const float *ln_wg, *ln_wb;
    int fc1_only;          // GATEUP: one weight (fc1), 128 consecutive rows per tile, ReLU instead of SwiGLU
    const void *bias;      // OPROJ, DOWN: bf16 [H] bias of the row-split layer, added once to the residual stream (and so to every device's X + P_i)
    float *sum_out;        // OPROJ, DOWN: partial row sums of the new residual, same layout as ss_out, or null
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
    TpArgs tp;
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
    // rank mode: n_z local ranks, whose res_out / hg / ss_out / step lie z_stride bytes apart; step (or null) is advanced by one
    int n_z;
    long z_stride;
    unsigned *step;
    unsigned long long *stamp; // launch stamp slot or null
    float *sum_out;    // block with bias: partial row sums of x, same layout as ss_out, or null
};
cudaError_t launch_decode_prologue(const PrologueArgs &a, cudaStream_t st);

} // namespace spd
