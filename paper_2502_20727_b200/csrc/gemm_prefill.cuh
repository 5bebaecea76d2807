// Host interface of the fused prefill projections (gemm_prefill.cu): persistent tcgen05 GEMMs
// with many tokens on the 128-row MMA side and the step that follows each projection applied
// straight from tensor memory.
#pragma once
#include "common.cuh"
#include "gemm_decode.cuh"
#include "gemm_tc.cuh"

namespace spd {

enum PreEpilogue {
    PRE_QKV = 0,       // a2 + a3: rstd, rotary embedding, q store, K/V page append
    PRE_RESID = 1,     // sync o_proj (a5-a7) and down (a9, a10): residual add, next norm's input and sums of squares
    PRE_GATEUP = 2,    // a8: rstd (per emulated device in an SPD block), SwiGLU
    PRE_OPROJ_SPD = 3, // a5-a7 of an SPD block: the T K-slices of one output tile in turn, R_i = X + Y_i kept apart
    PRE_SCATTER = 4,   // rank mode: the rank's partial rows of a row-split projection go to the ranks that own them
};

// Rank mode (one shard per rank, Sec. 3), prompts: the shard sums a block keeps are two-shot exchanges.  Shot one
// (PRE_SCATTER, the tail of the projection that produces the partial): the 128-token tiles of a launch are dealt
// round-robin to the ranks (tile i belongs to rank i % T); a block stores its fp32 partial rows of tile i into the
// owner's receive plane [source = own rank][slot = i / T][128 rows][H] with plain peer stores and then publishes the
// step number in the owner's flag word [slot][column tile][source].  Shot two is the finishing kernel of tp_prefill.cu.
struct TpScatter {
    int T, me;                     // group size; this rank
    int n_tiles;                   // column tiles of the launch (flag words per slot and source)
    long src_stride;               // bytes between the source planes of a receive buffer
    char *rx[TP_MAX_RANKS];        // rank j's receive buffer of this exchange
    unsigned *flags[TP_MAX_RANKS]; // rank j's scatter flags of this exchange: [slot][column tile][source]
    const float *addend;           // fp32 [tokens][H] added to the partial before it leaves (Y_r of an SPD block), or null
    const unsigned *step;          // this rank's step number (> 0, the same on all ranks)
};

struct PreGemmArgs {
    int t_rows;          // tokens of this launch
    int num_kb;          // 64-wide K blocks (per shard slice where the operands are batched)
    int batches;         // emulated devices: column blocks for GATEUP, K slices for OPROJ_SPD
    int t_batched;       // GATEUP in an SPD block: device z reads token-operand plane z
    int w_rows[3];       // valid rows (per device for GATEUP) of weight i
    int n_weights;
    int *err;
    unsigned long long *stamp; // launch stamp slot or null
    SumSq ss_in;         // QKV, GATEUP
    int rstd_per_shard;
    // block with bias (Sec. 4.1.2): LayerNorm folded into the tail (see SumSq): fp32 vectors over the launch's weight rows
    // (QKV: q, k, v rows one after the other; GATEUP: the rows of fc1), or null
    const float *ln_wg, *ln_wb;
    int fc1_only;        // GATEUP: one weight (fc1), 256 consecutive rows per tile, ReLU instead of SwiGLU
    const void *bias;    // RESID, OPROJ_SPD: bf16 [H] bias of the row-split layer, added once to the residual stream
    float *sum_out;      // RESID, OPROJ_SPD: partial row sums of the new residual, same layout as ss_out, or null
    // QKV
    const float2 *rope;  // [tokens][d/2] cos,sin or null
    void *q_out;         // bf16 [tokens][nq*d]
    void *k_pages, *v_pages;
    PageTable pt;
    TokMap tm;
    int n_q_heads, head_dim;
    // RESID, OPROJ_SPD
    const float *res_in; // fp32 [tokens][H]
    float *res_out;      // fp32 [tokens][H]
    const void *gain;    // bf16 [H] or null
    void *hg;            // bf16 [groups][Mcap][H]
    long hg_stride;
    float *ss_out;       // [tiles][groups][Mcap]; tiles = pre_ss_tiles(epilogue, H)
    long Mcap;
    void *final_out;     // bf16 [tokens][H] or null
    int H;
    // GATEUP
    void *act;           // bf16 [tokens][F]
    int F, Fs;
    // Head grouping (Sec. 4.2.4, MLP matching): GATEUP with w_rot = r applies MLP partition (z + r) % T to the
    // input of device z (output in the partition's column block); OPROJ_SPD with norm_only != 0 only writes, per
    // K slice and token, the sum of squares of the slice's output to ss_out (no residual, no operand planes).
    int w_rot;
    int norm_only;
    // CTA pairs: two CTAs of a cluster share one tile of 256 tokens (one M = 256 MMA over both), each loading half
    // of the tile's weight rows.  The weight maps must then have boxes of HALF the tile's rows: 128 (QKV, RESID,
    // GATEUP: gate rows in one CTA, up rows in the other), 64 (OPROJ_SPD).  Not with norm_only.
    int pair;
    // rank mode: fixed batch coordinate of the weight and of the token map (the rank's shard / the rank's plane)
    int w_z, t_z;
    int q_head0, kv_head0; // QKV: first query / KV head of the rank in q_out and in the pages
    int act_col0;          // GATEUP: first column of the rank's slice in act
    float *ysave;          // RESID: fp32 [tokens][H] copy of the projection's output (Y_r of an SPD block), or null
    TpScatter sc;          // SCATTER
    int group_m;         // token tiles per group of the tile order; 0 = default (8 pair tiles / 16 single tiles = 2048 tokens)
};

// Weight maps: 256-row boxes (QKV, RESID), 128-row boxes (GATEUP: gate and up; OPROJ_SPD: the
// shard-sliced W_O); with g.pair, boxes of half as many rows (see PreGemmArgs::pair).  Token map: 128-row box.
cudaError_t launch_gemm_prefill(PreEpilogue epi, const TcMap *const *weights, const TcMap &tokens, const PreGemmArgs &g,
                                cudaStream_t st);

// Column tiles (= partial sums of squares per token) the residual epilogues write.
int pre_ss_tiles(PreEpilogue epi, int H);

// Block input -> fp32 residual stream, x * gain, whole-row sum of squares (one tile).
cudaError_t launch_prefill_prologue(const PrologueArgs &a, cudaStream_t st);

} // namespace spd
