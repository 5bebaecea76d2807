/*
 * spd.h - C ABI of the B200 (sm_100a) Sync-Point Drop block library.
 *
 * The library runs the forward pass of a stack of tensor-parallel (TP) LLaMA-style
 * decoder blocks whose T devices ("shards") are emulated on ONE GPU.  Each block is
 * either a fully synchronous TP block (Sec. 3, Fig. 1(a)) or an SPD block (Sec. 4.1.1,
 * Fig. 1(b), Fig. 3(a)), chosen per block by a mask - the block list that Algorithm 1
 * produces.  Both kinds use the same parameters (Sec. 4.2.3).
 *
 * Conventions common to every call
 *   - All tensor pointers are DEVICE pointers unless marked "host".  Nothing passed in is
 *     ever freed or retained beyond what is stated; the library allocates no device memory.
 *   - dtype 0: float32 storage and arithmetic.  dtype 1: bfloat16 storage (weights,
 *     activations in/out, KV pages), float32 accumulation, float32 residual stream.
 *   - Linear weights use the torch.nn.Linear layout [out_features, in_features], row-major,
 *     contiguous.  Shard i of a column-split matrix (wq, wk, wv, w_gate, w_up) is its rows
 *     [i*n/T, (i+1)*n/T); shard i of a row-split matrix (wo, w_down) is its columns
 *     [i*k/T, (i+1)*k/T) (Sec. 4.1.2).  Head grouping (Sec. 4.2.4) is a permutation the
 *     caller applies to the weights beforehand.
 *   - KV pages of one layer: [n_pages, n_kv_heads, kv_block_size, head_dim] in the storage
 *     dtype, separately for K and V.  block_table[b, j] (int32) is the page holding tokens
 *     [j*kv_block_size, (j+1)*kv_block_size) of sequence b.
 *   - Every call returns SPD_OK (0) or a negative SPD_E* code and never throws, aborts or
 *     traps.  Work is enqueued on `stream` (a cudaStream_t passed as void*) and is
 *     asynchronous; a CUDA error of an earlier launch may be reported by a later call.
 */
#ifndef SPD_H
#define SPD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPD_OK 0
#define SPD_EINVAL (-1)     /* bad dimension, divisibility (nq % T, nkv % T, ffn % T), batch > max ... */
#define SPD_ENULL (-2)      /* a required pointer is null                                            */
#define SPD_EWORKSPACE (-3) /* workspace too small or misaligned (256 bytes)                          */
#define SPD_ECAPACITY (-4)  /* sequence would outgrow max_seq_len or the block table                  */
#define SPD_ECUDA (-5)      /* a CUDA call failed; see spd_last_cuda_error()                          */
#define SPD_EDEVICE (-6)    /* a kernel recorded a bounds / bounded-wait failure in its error flag   */
#define SPD_ECALLBACK (-7)  /* the all-reduce callback of spd_tp_baseline_* returned non-zero          */

typedef struct spd_ctx spd_ctx; /* opaque; owned by the library, freed by spd_destroy */

typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn;
    int32_t T;            /* emulated tensor-parallel devices                                   */
    int32_t dtype;        /* 0 = float32, 1 = bfloat16                                          */
    float rms_eps;
    float rope_base;      /* <= 0 disables the rotary embedding                                 */
    int32_t kv_block_size;      /* tokens per KV page (16)                                      */
    int32_t max_batch;          /* largest B of spd_decode_step / spd_prefill                   */
    int32_t max_seq_len;        /* largest context (cached + new tokens) of one sequence        */
    int32_t max_prefill_tokens; /* tokens processed per internal prefill chunk (bounds workspace)*/
    int32_t block_kind;         /* 0: block without bias (Sec. 4.1.1; RMSNorm, rotary, SwiGLU);
                                   1: block with bias (Sec. 4.1.2; LayerNorm, biased projections, ReLU,
                                      no rotary embedding; rms_eps is the LayerNorm eps)               */
} spd_dims;

typedef struct {
    const void *attn_norm; /* [hidden]                      RMSNorm gain before attention        */
    const void *wq;        /* [n_q_heads*head_dim, hidden]                                       */
    const void *wk;        /* [n_kv_heads*head_dim, hidden]                                      */
    const void *wv;        /* [n_kv_heads*head_dim, hidden]                                      */
    const void *wo;        /* [hidden, n_q_heads*head_dim]                                       */
    const void *mlp_norm;  /* [hidden]                      RMSNorm gain before the MLP          */
    const void *w_gate;    /* [ffn, hidden]                                                      */
    const void *w_up;      /* [ffn, hidden]                                                      */
    const void *w_down;    /* [hidden, ffn]                                                      */
    void *k_pages;         /* [n_pages, n_kv_heads, kv_block_size, head_dim]  written by the lib */
    void *v_pages;         /* same shape                                                         */
    /* block_kind 1 only (ignored, may be null, for kind 0).  There w_gate is fc1 [ffn, hidden], w_down is
     * fc2 [hidden, ffn] and w_up is not read.  Biases of column-split layers are split with them; the biases
     * of the row-split layers (bo, b_fc2) cannot be split: each is added once, after the shard sum - in an
     * SPD block bo also enters every device's MLP input X + P_i + b (Sec. 4.1.2). */
    const void *attn_norm_b; /* [hidden]  LayerNorm shift before attention                       */
    const void *bq;          /* [n_q_heads*head_dim]                                             */
    const void *bk, *bv;     /* [n_kv_heads*head_dim]                                            */
    const void *bo;          /* [hidden]  the b of Y_i = P_i + b                                 */
    const void *mlp_norm_b;  /* [hidden]  LayerNorm shift before the MLP                         */
    const void *b_fc1;       /* [ffn]                                                            */
    const void *b_fc2;       /* [hidden]                                                         */
} spd_layer;               /* device pointers, BORROWED: the caller keeps the tensors alive      */

/* Bytes of device workspace spd_create needs for these dims and mask (host call, no GPU
 * work).  sync_mask: host array [n_layers], 1 = synchronous TP block, 0 = SPD block.
 * Errors: SPD_ENULL, SPD_EINVAL. */
int spd_workspace_bytes(const spd_dims *dims, const uint8_t *sync_mask, size_t *out_bytes);

/* Build a context for a stack of blocks: Algorithm 1's block list, entry l being a TP block
 * when sync_mask[l] != 0 and an SPD block otherwise (Sec. 4.2; the block designs are those
 * of Sec. 3 and Sec. 4.1.1).
 *   layers    : host array [n_layers] of device pointers (copied; the tensors are borrowed)
 *   n_pages   : pages in every k_pages / v_pages tensor (block-table entries are checked
 *               against it on the device)
 *   workspace : device memory, 256-byte aligned, >= spd_workspace_bytes(); borrowed until
 *               spd_destroy; must not be shared by contexts running concurrently.  spd_create
 *               zeroes it (error flag, arrival counters, pad rows) between two device-wide
 *               synchronisations and returns only when that has completed, so the first call
 *               may use any stream.  A set-up call: not to be made during a stream capture.
 * Requires a CUDA device of compute capability 10.x as the current device.
 * Errors: SPD_ENULL, SPD_EINVAL, SPD_EWORKSPACE, SPD_ECUDA. */
int spd_create(const spd_dims *dims, const uint8_t *sync_mask, const spd_layer *layers,
               int32_t n_pages, void *workspace, size_t workspace_bytes, spd_ctx **out);

/* Prefill: run B prompts of S tokens each through the stack, writing their K/V into the
 * pages named by block_table (positions 0..S-1) and the last block's output to `out`.
 *   x, out      : [B, S, hidden] storage dtype; must not alias
 *   block_table : [B, max_pages] int32, max_pages*kv_block_size >= S
 * Attention is causal within each prompt (Sec. 3: each shard attends over its own heads).
 * Errors: SPD_ENULL, SPD_EINVAL (B > max_batch), SPD_ECAPACITY, SPD_ECUDA. */
int spd_prefill(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table,
                int32_t max_pages, void *out, void *stream);

/* One decode step: one new token per sequence.  Appends the token's K/V at position
 * seq_lens[b] and attends over seq_lens[b] + 1 tokens; the caller advances seq_lens.
 *   x, out       : [B, hidden] storage dtype; must not alias
 *   seq_lens     : [B] int32 device, tokens already cached per sequence
 *   max_context  : host-side upper bound of seq_lens[b] + 1 over the batch (sizes the
 *                  split of the KV range over thread blocks; <= max_seq_len)
 * A sequence whose seq_lens[b] + 1 exceeds max_context or its block-table row is skipped and
 * the device error flag is set (see spd_device_error).
 * Errors: SPD_ENULL, SPD_EINVAL, SPD_ECAPACITY, SPD_ECUDA. */
int spd_decode_step(spd_ctx *ctx, const void *x, int32_t B, const int32_t *seq_lens,
                    const int32_t *block_table, int32_t max_pages, int32_t max_context,
                    void *out, void *stream);

/* Decode steps are replayed from CUDA graphs (on by default): the first call with a given
 * (x, seq_lens, block_table, out, B, max_pages, max_context rounded up to 256) captures the
 * step's kernels on `stream` and later calls with the same values launch the captured graph;
 * tensor CONTENTS (inputs, seq_lens, block table) may change freely between calls.  Up to 8
 * graphs are kept per context.  A growing context changes bucket every 256 steps; the graph of the
 * next bucket is captured (not run) once max_context is within 32 of the edge, so the step that
 * crosses over finds its graph ready and the capture overlaps the steps still queued on the device.  A caller that passes fresh pointers every step should turn
 * this off (each new pointer set costs a capture).  Calls on the legacy default stream (which
 * cannot be captured), calls made while `stream` is itself being captured, and calls made
 * while profiling launch the kernels directly. */
int spd_set_graphs(spd_ctx *ctx, int32_t enabled);

/* Tuning knobs of the bf16 decode step (results stay deterministic for a given setting; every
 * change drops the captured decode graphs).  value 0 restores the automatic choice of a split key.
 *   "qkv_splits", "o_proj_splits", "gate_up_splits", "down_splits"
 *       how many ranges the K dimension of that weight-streaming projection is cut into (more
 *       ranges = more thread blocks pulling weights at once; the ranges of one output tile form
 *       a thread-block cluster that adds up its partials through shared memory).  Automatic:
 *       about three resident thread blocks per SM.  Clamped to at least four 64-wide K blocks
 *       per range and to 8 ranges per tile (8 / T for o_proj, whose T shard slices are ranges).
 *   "attention_splits"
 *       ranges the cached context of a sequence is cut into for the paged decode attention
 *       (clamped to 32 and to four pages per range).
 *   "l2_prefetch_blocks"
 *       64-wide K blocks of weights each thread block of a projection pulls into L2 before it
 *       waits for the preceding kernel (default 0 = off, at most 64; measured neutral to harmful).
 *   "decode_ring_stages"
 *       stages of the shared-memory ring the weight tiles of a decode projection stream through:
 *       3, 4 or (16-token tiles) 5; 0 = chosen per launch (four stages; at 16-token tiles five for
 *       launches of at most two thread blocks per SM and three where a launch only then stays
 *       resident at once).
 *   "o_proj_planes"
 *       decode o_proj: shard slices one thread block computes one after the other, each into its own accumulator
 *       columns (1 or 2; 0 = chosen per launch: two where one slice per block would not be resident at once - T * H/128
 *       blocks against two resident blocks per SM at 32- and 64-token tiles, three at 16).  Same sums in the same order.
 *   "prefill_rescale_log2"
 *       prefill attention on the tensor cores keeps its output accumulator relative to a row
 *       maximum that follows the true running maximum lazily: the accumulator is rescaled only
 *       when the maximum has grown by more than 2^value since the last rescale (default 8, at
 *       most 16; 0 = follow the maximum exactly, every growth rescales).  The result is the same
 *       softmax either way; only the rounding of the bf16 probabilities differs.
 *   "prefill_pairs"
 *       prompt projections on pairs of thread blocks (one 256-token tile and one tensor-core instruction over
 *       two SMs, each block loading half of the tile's weight rows): 1 (default) wherever a launch has more
 *       than 128 tokens, 0 = always one block per 128-token tile.  Same results bit for bit.
 *   "prefill_group_m"
 *       tile order of the prompt projections: token tiles are taken in groups of this many, and inside a group
 *       the token tile runs fastest, then the weight tile, so that a group's token panels stay in L2 while the
 *       weight tiles sweep past (0 = default: 2048 tokens per group; a value >= the number of token tiles gives
 *       the plain order with all token tiles fastest).  A schedule only: same results.
 *   "bias_fused"
 *       block with bias (Sec. 4.1.2) in bf16: 1 (default) = the same five fused projections per block as the
 *       block without bias - LayerNorm enters the QKV and fc1 tails through two vectors per layer folded from
 *       the weights at spd_create (sum_k g_k W_nk and sum_k beta_k W_nk + b_n) and the row mean and variance
 *       the preceding tail left; out_proj / fc2 biases and ReLU in the tails; 0 = K-split GEMMs with separate
 *       LayerNorm, bias and activation kernels.  The two differ in rounding only.  The fold subtracts
 *       mean * sum_k g_k W_nk from the accumulator: rows whose mean dwarfs their spread lose that much precision.
 *   "peer_wait_ms"
 *       rank mode (spd_tp_*): milliseconds a rank waits for the other ranks' partial sums before
 *       it gives up with error bit 8 (default and value 0: 1000; at most 60000).  Always bounded.
 *       Raise it where the ranks' hosts can be skewed by more than a second (a rank that is still
 *       instantiating its graph), lower it to fail fast.
 * Errors: SPD_ENULL, SPD_EINVAL (unknown key, negative value). */
int spd_set_tuning(spd_ctx *ctx, const char *key, int32_t value);

/* The projection building block on its own (exposed for kernel-level tests): the bf16
 * tensor-core GEMM every projection of the block uses, with the batching that expresses the
 * shard structure of Sec. 4.1.1 - per-shard weight row blocks (column split) and, when
 * a_batched != 0, a separate input per shard (the SPD block's per-device MLP input).
 *   a : bf16 [a_batched ? batches : 1][M][K]      w : bf16 [batches][N][K]
 *   c : fp32 [splits][M][batches*N];  c[s][m][z*N + n] = sum over K-range s of a_z[m][:] . w_z[n][:]
 *   swap != 0 puts the weight rows on the 128-row MMA side (the decode configuration)
 *   err_flag : device int32, bit 4 is set if a bounded wait inside the kernel gave up
 * K must be a multiple of 8; 1 <= splits <= ceil(K/64).  Errors: SPD_ENULL, SPD_EINVAL, SPD_ECUDA. */
int spd_gemm_bf16(const void *a, const void *w, float *c, int32_t M, int32_t N, int32_t K, int32_t batches,
                  int32_t a_batched, int32_t splits, int32_t swap, int32_t *err_flag, void *stream);

/* The same split-K projection GEMM for callers that cannot obtain device memory at the time of
 * the call: code running inside a serving engine whose allocator owns the whole GPU, a plugin
 * invoked under a "no cudaMalloc / no allocator call" rule (the driver call synchronises the
 * device and can fail once other tenants have filled it), or a process that must stay within a
 * fixed memory budget.  (The paper has no counterpart; this is a library convenience.)
 *   c : fp32 [M][batches*N] = the SUM over the K splits (same operands and meaning as
 *       spd_gemm_bf16, whose split planes this call adds up in split order)
 * The split planes are kept in an array that is part of the library image,
 * SPD_STATIC_SCRATCH_BYTES per GPU that loads the library, held until the process exits.  The
 * call allocates and frees no device memory itself and uses no allocating library routine;
 * inputs, output and err_flag are still the caller's.
 *   - splits * M * batches * N * 4 bytes must fit in the array, else SPD_EWORKSPACE is
 *     returned and nothing is launched.
 *   - The first call on a device looks up the array's device address (the device must be
 *     current); make that first call outside any stream capture.
 *   - All calls share the one array, and it keeps whatever the previous call left there.
 *     Each call overwrites every element it later reads, so nothing needs clearing, but two
 *     calls whose kernels may overlap on the GPU (different streams) race: serialise them.
 * Errors: SPD_ENULL, SPD_EINVAL, SPD_EWORKSPACE (too large for the array), SPD_ECUDA. */
#define SPD_STATIC_SCRATCH_BYTES (4u << 20)
int spd_gemm_bf16_sum_static(const void *a, const void *w, float *c, int32_t M, int32_t N, int32_t K, int32_t batches,
                             int32_t a_batched, int32_t splits, int32_t swap, int32_t *err_flag, void *stream);

/* Replace the per-block mask of a context (same meaning as in spd_create).  A mask with an SPD
 * block needs the larger workspace of such a stack: SPD_EWORKSPACE if the context was created
 * from an all-sync mask.  Drops the captured decode graphs.  Errors: SPD_ENULL, SPD_EWORKSPACE. */
int spd_set_mask(spd_ctx *ctx, const uint8_t *sync_mask);

/* Block-wise sync-sensitivity identification (Sec. 4.2.1) on this stack, with the mean squared
 * difference from the all-TP output as the quality metric in place of perplexity (this path
 * has no LM head).  For i = L-1 .. 0 the prompt batch x is run with blocks i .. L-1 as SPD blocks
 * and blocks 0 .. i-1 as TP blocks; metric[i] is that output's mean squared difference from the
 * all-TP output (metric[L] = 0), and sensitivity[i] = metric[i] - metric[i+1]: what turning
 * block i into an SPD block adds when every later block already is one.
 *   x, block_table, B, S : as for spd_prefill (the caches of those rows are overwritten by each pass)
 *   ref_out, tmp_out     : device scratch, [B, S, hidden] storage dtype each (ref_out returns the all-TP output)
 *   sensitivity          : host [n_layers];  metric : host [n_layers + 1] or null
 * Runs n_layers + 1 prefills, synchronises `stream`, restores the context's mask.
 * Errors: those of spd_prefill and spd_set_mask. */
int spd_sensitivity_scan(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table, int32_t max_pages,
                         void *ref_out, void *tmp_out, double *sensitivity, double *metric, void *stream);

/* Algorithm 1: rank the blocks by sensitivity (ascending, ties by index), turn the first n_spd
 * into SPD blocks and label each by tier: sensitivity <= tau1 in-sensitive (zero-shot dropping,
 * Sec. 4.2.2), <= tau2 sensitive (wants block-to-block distillation first, Sec. 4.2.3), else
 * extremely sensitive (wants head grouping and distillation, Sec. 4.2.4).  The library only
 * runs blocks; distillation and head grouping produce different weights for the same kernels.
 *   sync_mask : host out [n_blocks], 1 = stays a TP block, 0 = SPD block;  tier : host out [n_blocks]
 * Pure host function.  Errors: SPD_ENULL, SPD_EINVAL (n_spd outside [0, n_blocks], tau1 > tau2). */
#define SPD_TIER_TP 0
#define SPD_TIER_ISB 1
#define SPD_TIER_SB 2
#define SPD_TIER_ESB 3
int spd_alg1_plan(const double *sensitivity, int32_t n_blocks, int32_t n_spd, double tau1, double tau2, uint8_t *sync_mask,
                  uint8_t *tier);

/* SPD-aware attention head grouping (Sec. 4.2.4), measurements.  The prompt batch x runs through
 * blocks 0 .. layer-1 as TP blocks (Sec. 4.2.3) and through block `layer` as an SPD block with the weights as
 * they are now (device i = head rows [i*nq/T, (i+1)*nq/T), MLP partition m = FFN rows [m*F/T, (m+1)*F/T)):
 *   dist  : host out [nq][nq], Euclidean distance between the attention-score vectors of two heads over all
 *           prompts (softmax probabilities, causal, zeros above the diagonal) - the d(sigma, sigma) of Eq. 2
 *   norms : host out [T][T], norms[i][m] = Frobenius norm over all tokens of MLP_m(rmsnorm(X + Y_i)), the
 *           output of MLP partition m (its slice of gate/up/down, before any sum) on device i's input - Eq. 3
 *   sigma_scratch : device, nq * B * S * S floats;  dist_dev : device, nq * nq floats
 * bf16 stacks only; B * S <= max_prefill_tokens; overwrites the caches of those rows for blocks 0 .. layer;
 * synchronises `stream`.  Errors: SPD_ENULL, SPD_EINVAL, SPD_ECAPACITY, SPD_EWORKSPACE (context created from
 * an all-sync mask), SPD_ECUDA. */
int spd_head_grouping_stats(spd_ctx *ctx, int32_t layer, const void *x, int32_t B, int32_t S, const int32_t *block_table,
                            int32_t max_pages, float *sigma_scratch, float *dist_dev, float *dist, double *norms, void *stream);

/* Head scattering, Eq. 2: split the heads into T equal sets so that the sum, over the sets, of the pairwise
 * distances inside a set is largest (similar heads end up on different devices).  The query heads of one KV head
 * stay together: a unit is heads_per_unit consecutive heads, the distance of two units the sum over their head
 * pairs.  Exhaustive for up to 12 units, else a greedy start improved by pairwise swaps until none helps.
 *   dist : host [n_heads][n_heads];  device_of_unit : host out [n_heads / heads_per_unit]
 * Pure host function.  Errors: SPD_ENULL, SPD_EINVAL (units not divisible by T, ...). */
int spd_head_scatter(const float *dist, int32_t n_heads, int32_t heads_per_unit, int32_t T, int32_t *device_of_unit, double *objective);

/* MLP matching, Eq. 3: the assignment of MLP partitions to devices with the largest sum of output norms, over
 * all T! matchings.  norms : host [T][T] as from spd_head_grouping_stats;  mlp_of_device : host out [T].
 * Pure host function.  Errors: SPD_ENULL, SPD_EINVAL (T > 8). */
int spd_mlp_match(const double *norms, int32_t T, int32_t *mlp_of_device, double *objective);

/* ---- Tensor parallelism across GPUs (Sec. 3: one shard per device; Sec. 4.1.1: what an SPD block
 * still exchanges) --------------------------------------------------------------------------------
 *
 * A context created from the dims of ONE shard (T = 1; n_q_heads, n_kv_heads, ffn and the weight
 * matrices those of the shard: rows [r*n/T, (r+1)*n/T) of wq / wk / wv / w_gate / w_up, columns
 * [r*k/T, (r+1)*k/T) of wo / w_down stored as a contiguous matrix) becomes rank r of a group of T
 * ranks once it is attached to the group's regions.  A region is spd_tp_region_bytes() of device
 * memory owned by one rank and WRITABLE BY EVERY RANK (peer-mapped: CUDA IPC, the driver's
 * virtual-memory mappings or a symmetric-memory allocator; plain stores and loads only, no
 * multicast).  It holds the rank's receive planes and arrival flags and the rank's private copy
 * of the residual stream.  `regions` is a host array of T device pointers as mapped in the
 * calling process; entry j is rank j's region; 1024-byte aligned.
 *
 * A context created with T > 1 shards (the emulation all other entry points use) can be attached
 * with rank_base = 0 and group size T = dims.T: then ONE GPU executes all T ranks, every launch
 * covering all ranks' data, through exactly the same kernels and exchange protocol; its T regions
 * must lie at equal distances (regions[j] = regions[0] + j * stride).  All thread blocks of such
 * a launch have to be resident at once (they wait on one another): a launch that does not fit is
 * refused with SPD_ECUDA (cudaErrorCooperativeLaunchTooLarge) before anything runs.
 *
 * Attaching zeroes the local regions on `stream`.  It is collective: every rank attaches, then
 * the group synchronises on the host (stream synchronize + barrier) before anyone's first step.
 * bf16 LLaMA-style stacks only (dtype 1, block_kind 0, hidden % 16 == 0).
 * Errors: SPD_ENULL, SPD_EINVAL, SPD_EWORKSPACE (region too small / misaligned), SPD_ECUDA. */
int spd_tp_region_bytes(const spd_ctx *ctx, int32_t T, size_t *out_bytes);
int spd_tp_attach(spd_ctx *ctx, int32_t T, int32_t rank_base, void *const *regions, size_t region_bytes,
                  void *stream);
int spd_tp_detach(spd_ctx *ctx);

/* One decode step of an attached context (same arguments as spd_decode_step; every rank of the
 * group calls it with the same x, seq_lens and block-table contents, and the same number of
 * times).  Per block and rank: QKV on the rank's heads, attention, o_proj, gate/up, down - and
 * the shard sums the block keeps as one-shot exchanges inside the tail of the projection that
 * produces the partial: each rank stores its fp32 partial rows into every rank's receive planes,
 * publishes the step number in the peers' flags and adds the T planes in rank order, so all
 * ranks hold bit-identical residual streams.  A TP block exchanges twice (Y_i after o_proj,
 * Z_i after down: Sec. 3), an SPD block once (Y_i + Z_i after down: Sec. 4.1.1).
 *   out : [ranks held by the context][B][hidden] bf16 - every rank's copy of the output
 * A wait for a peer gives up after about one second ("peer_wait_ms" of spd_set_tuning): the kernels then return normally, the
 * step's output is undefined and spd_device_error reports bit 8; the context stays usable.
 * Errors: SPD_ENULL, SPD_EINVAL (not attached, B > max_batch), SPD_ECAPACITY, SPD_ECUDA. */
int spd_tp_decode_step(spd_ctx *ctx, const void *x, int32_t B, const int32_t *seq_lens,
                       const int32_t *block_table, int32_t max_pages, int32_t max_context, void *out,
                       void *stream);

/* Prompt processing of an attached context (same arguments as spd_prefill, same collective rules as
 * spd_tp_decode_step), at tensor-core speed: every rank runs the prompt projections on its own shard, and every
 * shard sum the block keeps is a two-shot exchange.  Shot one is the tail of the projection that produces the
 * partial: the 128-token tiles of a launch are dealt round-robin to the ranks, and each rank stores its fp32
 * partial rows of a tile into the owner's receive plane (plain peer stores) and publishes the step number in the
 * owner's flags.  Shot two: the owner adds the T planes in rank order (all ranks end up with the same bits), adds
 * the residual and writes the finished rows - residual stream, operand of the next projection, sums of squares -
 * into every rank's planes; a small kernel on each rank waits for all owners before the next projection starts.
 * A TP block exchanges Y_r and Z_r (Sec. 3), an SPD block only Y_r + Z_r (Sec. 4.1.1).  Prompts go in chunks of
 * at most min(max_prefill_tokens, 2048) tokens, every chunk attending to the cached positions before it.
 *   out : [ranks held by the context][B][S][hidden] bf16
 * Waits for peers are bounded as in spd_tp_decode_step (error bit 8, "peer_wait_ms").
 * Errors: SPD_ENULL, SPD_EINVAL (not attached, B > max_batch), SPD_ECAPACITY, SPD_ECUDA. */
int spd_tp_prefill(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table,
                   int32_t max_pages, void *out, void *stream);

/* Baseline of the rank mode: the same shard-per-rank execution with the shard sums done by a library collective
 * BETWEEN kernels - how tensor parallelism is normally run (Sec. 3: two all-reduces per TP block, NCCL in the
 * paper's measurements) - instead of the exchange fused into the projection's tail.  The context is ONE shard's
 * stack (created with T = 1 from the shard's dims and weights, exactly as for spd_tp_attach; not attached).  The
 * step runs the projections as K-split GEMMs with separate residual / norm kernels and calls `all_reduce` on
 * `stream`'s behalf at every sync-point the block keeps: a TP block twice (Y_r after o_proj, Z_r after down),
 * an SPD block once (Y_r + Z_r after down; R_r = X + Y_r feeds the rank's own MLP, X joins after the sum:
 * Sec. 4.1.1).
 *   all_reduce(user, buf, count, stream) : must leave in buf (device, fp32, `count` = tokens of the launch x hidden
 *       elements) the element-wise SUM of all ranks' buf, ordered on `stream` after the work enqueued so far and
 *       before what is enqueued next (e.g. ncclAllReduce on that stream); returns 0, anything else aborts the
 *       call with SPD_ECALLBACK.  Every rank makes the same calls in the same order.
 *   scratch : device, fp32, at least 2 x (tokens per launch) x hidden floats; tokens per launch = B for a decode
 *       step, min(B * S, max_prefill_tokens) for prompts
 * Launched directly (no graph replay: the collective is the caller's).  bf16 LLaMA-style stacks only.
 * Errors: SPD_ENULL, SPD_EINVAL (context holds more than one shard, ...), SPD_ECAPACITY, SPD_EWORKSPACE (scratch too
 * small), SPD_ECALLBACK, SPD_ECUDA. */
typedef int (*spd_allreduce_fn)(void *user, float *buf, size_t count, void *stream);
int spd_tp_baseline_decode_step(spd_ctx *ctx, const void *x, int32_t B, const int32_t *seq_lens,
                                const int32_t *block_table, int32_t max_pages, int32_t max_context, void *out,
                                float *scratch, size_t scratch_floats, spd_allreduce_fn all_reduce, void *user,
                                void *stream);
int spd_tp_baseline_prefill(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table,
                            int32_t max_pages, void *out, float *scratch, size_t scratch_floats,
                            spd_allreduce_fn all_reduce, void *user, void *stream);

/* Number of shard sums ("sync-points", Sec. 3) one forward pass of this stack executes:
 * 2 per TP block, 1 per SPD block. */
int spd_sync_points(const spd_ctx *ctx);

/* Number of kernels one spd_decode_step / one spd_prefill chunk launches (bookkeeping). */
int spd_launches_per_decode_step(const spd_ctx *ctx);

/* Read and clear the device error flag (synchronises `stream`).  0 = clean; otherwise a bit
 * set: 1 block-table entry out of range, 2 position beyond capacity, 4 bounded wait gave up,
 * 8 a wait for another rank's partial sums gave up.
 * Kernels that meet such a condition skip the access, set the flag and return normally. */
int spd_device_error(spd_ctx *ctx, void *stream, int32_t *out_flag);

/* Per-kernel-kind timing for benchmarks.  Between spd_profile_begin and spd_profile_end every
 * kernel launch of spd_prefill / spd_decode_step is bracketed by CUDA events on the call's
 * stream (the launches are not fused or reordered, only time-stamped).  spd_profile_end
 * synchronises `stream` and fills ms_by_kind / launches_by_kind (host arrays of
 * spd_profile_kinds() entries; a "launch" here is one bracketed call site, which for decode
 * attention covers its split and merge kernels).  Not to be used under stream capture. */
int spd_profile_begin(spd_ctx *ctx);
int spd_profile_end(spd_ctx *ctx, void *stream, float *ms_by_kind, int32_t *launches_by_kind);
int spd_profile_kinds(void);
const char *spd_profile_kind_name(int kind);

/* Launch timeline for benchmarks: how much of a call's duration every kernel accounts for INSIDE the call as it
 * is normally issued - decode steps replayed from their graph, back to back, launches overlapping through
 * programmatic dependent launch - with nothing inserted between the launches and no host round trip between
 * the calls (spd_profile_* brackets every launch with events, which serialises them).  After spd_timeline_begin
 * every kernel of the bf16 prompt and decode paths (block_kind 0; the kernels of the other paths carry no stamps
 * and are left out) gets a slot in the workspace: one thread of each of its blocks records the GPU's global
 * nanosecond timer at block start and end, the slot keeps the earliest start and the latest end.  A small
 * kernel at the end of each spd_prefill / spd_decode_step / spd_tp_decode_step call (part of the captured
 * step) folds the stamps into running totals: launch i's own share of the call = end[i] minus the later of
 * start[i] and the latest end before it (consecutive launches overlap: the next kernel's blocks start, and
 * request their first weights, under the tail of the one before), and the call's span = latest end - earliest
 * start; the shares add up to at most the span.
 *   spd_timeline_begin : presets slots and totals on `stream`; the first begin drops the captured decode graphs (a
 *                        step is captured again, with slots), a further begin only clears the totals
 *   spd_timeline_read  : synchronises `stream`; totals since spd_timeline_begin over *n_calls calls, for the first
 *                        min(launches of the last call, max_launches) launches in launch order: kinds[i] (index
 *                        of spd_profile_kind_name) and own_ns[i]; *span_ns = sum of the calls' spans.  Meaningful
 *                        when all calls since begin had the same launch sequence (same call, B, mask).  A call
 *                        with more than 6 * n_layers + 16 launches (chunked prompts) accounts for the first ones.
 *   spd_timeline_end   : stops stamping, drops the captured graphs
 * Errors: SPD_ENULL, SPD_EINVAL (read without begin), SPD_ECUDA. */
int spd_timeline_begin(spd_ctx *ctx, void *stream);
int spd_timeline_read(spd_ctx *ctx, void *stream, int32_t max_launches, int32_t *kinds, uint64_t *own_ns,
                      int32_t *n_launches, uint64_t *span_ns, uint64_t *n_calls);
int spd_timeline_end(spd_ctx *ctx);

/* Free the context (host state, descriptors, graphs).  Never touches caller tensors. */
void spd_destroy(spd_ctx *ctx);

const char *spd_status_string(int status);
/* cudaError_t value of the most recent failing CUDA call seen by this thread (0 = none). */
int spd_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SPD_H */
