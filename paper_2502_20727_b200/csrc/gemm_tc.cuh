// Host interface of the tcgen05 projection GEMM (gemm_tc.cu).
#pragma once
#include <cuda_runtime.h>

namespace spd {

// A CUtensorMap kept opaque so that callers need not include the driver header.
struct alignas(64) TcMap { unsigned long long opaque[16]; };

// One launch covers up to three weight matrices that share the token operand (Q|K|V, gate|up).
struct TcGemmArgs {
    float *C;             // fp32 output
    long c_off[3];        // element offset of weight i's output inside C (column or plane offset)
    long ldc;             // elements between token rows of C
    long c_batch_stride;  // elements added per batch z (a column offset or a plane offset)
    long c_split_stride;  // elements between K-split planes
    int t_rows;           // valid token rows
    int w_rows[3];        // valid rows per batch of weight i
    int batches;          // z extent
    int w_batched;        // weight operands have a batch dimension
    int t_batched;        // token operand has a batch dimension
    int num_kb;           // 64-wide K blocks per batch (ceil)
    int splits;           // K splits, <= num_kb
    int *err;             // device error flag
    // filled by the launcher
    int w_tiles_per_batch;
    int tile_start[3];
};

// Encode rows x k_inner bf16 (row stride ld_elems), `batches` of them batch_stride_elems apart.
// Returns 0, or <0 when the driver entry point is missing / alignment is violated / encode fails.
int make_operand_map(TcMap *out, const void *ptr, long k_inner, long rows, long batches, long ld_elems,
                     long batch_stride_elems, int box_rows);
// A paged K / V cache (16-token pages, head_dim 128) as a map whose {64, 16, 2} box is one (page, head): see gemm_tc.cu.
int make_page_map(TcMap *out, const void *ptr, long rows);

// Box rows of the token-side operand for a given token count (swap: 16/32/64, else 128).
int tc_token_box(bool swap, int tokens);
int tc_weight_box(bool swap);

// swap = weights on the 128-row MMA side (decode); otherwise tokens on it (prefill).
cudaError_t launch_gemm_tc(const TcMap *const *weights, int n_weights, const TcMap &tokens, const TcGemmArgs &g,
                           bool swap, cudaStream_t st);

} // namespace spd
