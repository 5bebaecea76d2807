// Host interface of the rank-mode prompt exchange (tp_prefill.cu): the finishing kernel of a two-shot shard sum
// and the wait that lets the next projection start.
#pragma once
#include "common.cuh"
#include "gemm_decode.cuh"

namespace spd {

struct TpFinishArgs {
    int T, me;             // group size; this rank (owner of the 128-token tiles me, me + T, ...)
    int M, H;              // tokens of the launch; hidden size
    int n_tiles;           // column tiles per 128-token tile (flag words per slot and source)
    const char *rx;        // this rank's receive buffer of the exchange: [source][slot][128][H] fp32
    long src_stride;       // bytes between its source planes
    const unsigned *sflags; // this rank's scatter flags of the exchange: [slot][column tile][source]
    const unsigned *step;  // step number (> 0, the same on all ranks)
    const float *res_in;   // this rank's residual stream, fp32 [tokens][H]: what the summed update joins
    const void *gain;      // bf16 [H] gain of the norm that follows, or null (then the bf16 copy is the plain sum)
    // all-gather: every rank's region, and where in it the finished rows go
    char *region[TP_MAX_RANKS];
    long off_res_out;      // fp32 [tokens][H]
    long off_hg;           // bf16 [tokens][H]
    long off_ss;           // fp32 [tokens]: row sums of squares of the new residual (one tile)
    long off_gflags;       // gather flags of the exchange: [128-token tile][blocks per tile]
    unsigned long long wait_ns;
    int *err;
    unsigned long long *stamp;
};
cudaError_t launch_tp_finish(const TpFinishArgs &a, cudaStream_t st);
int tp_finish_blocks_per_tile();

// One warp waits (bounded) until the gather flags of all 128-token tiles of a launch of M tokens show the step.
cudaError_t launch_tp_gather_wait(const unsigned *gflags, int M, const unsigned *step, unsigned long long wait_ns, int *err, cudaStream_t st);

} // namespace spd
