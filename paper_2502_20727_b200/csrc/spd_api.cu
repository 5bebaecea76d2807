// C ABI of the SPD block library: validation, workspace layout and the per-layer launch
// sequence of the synchronous TP block (Sec. 3) and the SPD block (Sec. 4.1.1).
#include "../../include/spd.h"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "gemm_decode.cuh"
#include "gemm_prefill.cuh"
#include "tp_prefill.cuh"

#include <math.h>
#include <new>
#include <string.h>
#include <vector>

using namespace spd;

static thread_local int g_last_cuda_error = 0;

void spd::note_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

int spd::sm_count()
{
    static int cached[64] = {};
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    if (cached[dev]) return cached[dev];
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { cudaGetLastError(); return 148; }
    return cached[dev] = n;
}

#define CU_TRY(expr)                                                   \
    do {                                                               \
        cudaError_t e__ = (expr);                                      \
        if (e__ != cudaSuccess) { g_last_cuda_error = (int)e__; return SPD_ECUDA; } \
    } while (0)

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int cdiv(int a, int b) { return (a + b - 1) / b; }

// How one launch sequence cuts its GEMMs along K (per-call-site split counts).
struct Plan {
    int qkv_splits, o_per_group, gu_splits, down_splits, attn_splits;
    // float32 (CUDA-core) path only: elements of K per split
    int qkv_kps, o_kps, gu_kps, down_kps;
};

// Largest s <= want such that K splits into s ranges that are multiples of `align`.
int fit_splits(int K, int want, int align)
{
    for (int s = want; s > 1; --s)
        if (K % s == 0 && (K / s) % align == 0) return s;
    return 1;
}

int want_splits(long tiles, int cap)
{
    long s = (2 * sm_count() + tiles - 1) / tiles;
    if (s > cap) s = cap;
    return (int)(s < 1 ? 1 : s);
}

enum ActBuf { AB_H = 0, AB_ATTN, AB_ATTN_SHARD, AB_ACT, AB_ACT_SHARD, AB_Q, AB_COUNT };
enum Kind { K_NORM = 0, K_QKV, K_ROPE_KV, K_ATTN, K_OPROJ, K_GATE_UP, K_SILU_MUL, K_DOWN, K_ROPE_TABLE, K_COUNT };
enum Site { SITE_QKV = 0, SITE_O, SITE_GU, SITE_DOWN, SITE_ATTN, SITE_COUNT };
const char *const kind_names[K_COUNT] = {"residual_rmsnorm", "gemm_qkv", "rope_kv_append", "attention", "gemm_o_proj",
                                         "gemm_gate_up", "silu_mul", "gemm_down", "rope_table"};

struct LayerMaps { TcMap wq, wk, wv, wo_full, wo_shard, wo_shard64, w_gate, w_up, w_down, w_gate64, w_up64, wq256, wk256, wv256, wo256, wd256, wd_shard, kpages, vpages, kpage_whole, vpage_whole; };

// A captured decode step is valid for exactly these arguments.
struct GraphKey {
    const void *x;
    const int32_t *seq_lens, *block_table;
    void *out;
    int B, max_pages, ctx_bucket;
    int mode; // 0: spd_decode_step; rank mode: 1 + receive buffer of the step's first exchange
    bool operator==(const GraphKey &o) const
    {
        return x == o.x && seq_lens == o.seq_lens && block_table == o.block_table && out == o.out && B == o.B &&
               max_pages == o.max_pages && ctx_bucket == o.ctx_bucket && mode == o.mode;
    }
};
struct GraphEntry { GraphKey key; cudaGraphExec_t exec; unsigned long long last_use; int launches; std::vector<int> tl_kind; };

// One rank's region of a tensor-parallel group (offsets in bytes; every rank uses the same layout).
struct TpLayout {
    size_t flags, rx, res0, res1, ysave, hg, ss_attn, ss_mlp, step, total;
    size_t site_flags; // flag words of one (layer, exchange site) of the decode step's one-shot exchange
    size_t buf_bytes, src_bytes;
    long Mb;           // token capacity of the residual / operand / sums planes: a decode batch or a prompt chunk
    long Md;           // token capacity of the decode step's receive planes (max_batch)
    int tok_tiles;
    // prompts: two-shot exchange over 128-token tiles dealt round-robin to the ranks
    size_t rs_rx, sflags, gflags;       // receive buffers (two), scatter flags, gather flags
    size_t rs_src_stride, rs_buf_bytes; // one source plane ([slot][128][H] fp32); one receive buffer (T source planes)
    size_t sflag_words, gflag_words;    // flag words of one (layer, exchange site)
    int slots_cap, n_tiles;             // 128-token tiles a rank can own per launch; 256-column tiles of H
};

struct TpState {
    bool on;
    int T, rank_base;
    long z_stride;
    unsigned long long exchanges; // exchanges launched since the attach (the same number on every rank)
    TpLayout L;
    char *regions[TP_MAX_RANKS];
    std::vector<TcMap> qkv_maps; // per layer: wq, wk, wv with one batch per local shard
    TcMap h_maps[4];             // the local ranks' gain-scaled inputs, token boxes 16 / 32 / 64 / 128
};

struct Ctx {
    spd_dims d;
    bool use_graphs;
    std::vector<GraphEntry> graphs;
    unsigned long long graph_clock;
    std::vector<uint8_t> mask;
    std::vector<spd_layer> layers;
    std::vector<LayerMaps> maps; // bf16 only
    int n_pages;
    bool any_spd;
    long Mcap; // token capacity of every activation buffer (plane stride = Mcap * width)
    char *ws;
    size_t ws_bytes;
    float *res[2];
    void *h, *q, *attn, *act;
    float *qkv32, *proj32, *gu32, *part_o, *part_ml;
    float2 *rope;
    int *err, *attn_cnt;
    float *ss_attn, *ss_mlp;     // partial row sums of squares (fused decode path)
    float *sm_attn, *sm_mlp;     // block with bias: partial row sums (LayerNorm means)
    float *lnvec;                // block with bias: per layer wg_qkv[nqkv], wb_qkv[nqkv], wg_fc1[F], wb_fc1[F]
    int bias_fused;              // block with bias on the fused projections (1) or on the K-split GEMMs with separate row kernels (0)
    int split_override[SITE_COUNT];
    int l2_prefetch_kb;          // K blocks per thread block prefetched into L2 by the decode GEMMs
    int ring_stages;             // decode GEMMs: stages of the operand ring (0 = per launch)
    int oproj_planes;            // decode o_proj: shard slices per thread block (0 = per launch, 1, 2)
    int prefill_rescale_log2;    // tcgen05 prefill attention: growth of the row maximum (log2) that triggers a rescale
    int peer_wait_ms;            // rank mode: how long a rank waits for its peers' partial sums
    int prefill_group_m;         // prompt projections: token tiles per group of the tile order (0 = default)
    int prefill_pairs;           // prompt projections: CTA pairs (256-token tiles) where a launch has more than 128 tokens
    int launches_last;
    TpState tp;
    // activation tensor maps, by buffer and token box (16, 32, 64, 128), built on first use
    TcMap act_maps[AB_COUNT][4];
    bool act_map_ready[AB_COUNT][4];

    // optional launch stamps (spd_timeline_*): slot i = earliest block start / latest block end of the call's i-th launch
    bool timeline;
    unsigned long long *stamps;
    int stamps_cap, tl_next;
    std::vector<int> tl_kind;

    // optional per-kernel-kind timing (spd_profile_begin / spd_profile_end)
    bool profiling;
    std::vector<cudaEvent_t> ev_pool;
    std::vector<int> ev_kind; // kind of the launch bracketed by events 2i, 2i+1
    size_t ev_used;
};

cudaError_t prof_mark(Ctx *c, int kind, cudaStream_t st)
{
    if (!c->profiling) return cudaSuccess;
    if (c->ev_used == c->ev_pool.size()) {
        cudaEvent_t e;
        cudaError_t rc = cudaEventCreate(&e);
        if (rc != cudaSuccess) return rc;
        c->ev_pool.push_back(e);
    }
    if (kind >= 0) c->ev_kind.push_back(kind);
    return cudaEventRecord(c->ev_pool[c->ev_used++], st);
}

// The stamp slot of the call's next launch (null when no timeline is being taken or the slots are used up).
unsigned long long *next_stamp(Ctx *c, int kind)
{
    if (!c->timeline || c->tl_next >= c->stamps_cap) return nullptr;
    c->tl_kind.push_back(kind);
    return c->stamps + 2 * (size_t)c->tl_next++;
}

// A call starts its timeline afresh (the slots were preset by spd_timeline_begin or by the fold of the call before).
cudaError_t timeline_restart(Ctx *c, cudaStream_t)
{
    if (!c->timeline) return cudaSuccess;
    c->tl_next = 0;
    c->tl_kind.clear();
    return cudaSuccess;
}

// Last launch of a stamped call.  Turns the stamps into every launch's own share of the call - its end minus the
// later of its start and the latest end of the launches before it, so overlapping launches are not counted twice
// and the shares add up to at most the call's span -, adds shares and span to running totals and presets the
// slots for the next call: stamped steps can then run back to back, replayed from their graph, with no host
// round trip in between.  acc: [cap] shares, then span, then number of calls (all in ns / counts, 64-bit).
__global__ void __launch_bounds__(256) timeline_fold_kernel(unsigned long long *slots, int n, unsigned long long *acc, int cap)
{
    pdl_launch_dependents();
    pdl_wait(); // every launch of the call has completed: each waited for the one before it
    __shared__ unsigned long long sm_end[256];
    __shared__ unsigned long long sm_carry, sm_first;
    const int t = threadIdx.x;
    if (t == 0) { sm_carry = 0; sm_first = ~0ull; }
    __syncthreads();
    for (int base = 0; base < n; base += 256) {
        const int i = base + t;
        unsigned long long s = 0, e = 0;
        bool ok = false;
        if (i < n) {
            const unsigned long long a = slots[2 * i], b = slots[2 * i + 1];
            ok = a != ~0ull && b != ~0ull;
            s = a; e = ok ? ~b : 0;
            slots[2 * i] = ~0ull; slots[2 * i + 1] = ~0ull;
        }
        // inclusive running maximum of the ends (launches that did not run count as 0)
        sm_end[t] = e;
        __syncthreads();
        for (int d = 1; d < 256; d <<= 1) {
            const unsigned long long o = t >= d ? sm_end[t - d] : 0;
            __syncthreads();
            if (o > sm_end[t]) sm_end[t] = o;
            __syncthreads();
        }
        const unsigned long long carry = sm_carry;
        unsigned long long before = t > 0 ? sm_end[t - 1] : 0;
        if (carry > before) before = carry;
        if (ok) {
            const unsigned long long begin = s > before ? s : before;
            if (e > begin) acc[i] += e - begin;
            atomicMin(&sm_first, s);
        }
        __syncthreads();
        if (t == 255) sm_carry = sm_end[255] > carry ? sm_end[255] : carry;
        __syncthreads();
    }
    if (t == 0) {
        if (sm_first != ~0ull && sm_carry > sm_first) acc[cap] += sm_carry - sm_first;
        acc[cap + 1] += 1;
    }
}

cudaError_t timeline_fold(Ctx *c, cudaStream_t st)
{
    if (!c->timeline || c->tl_next == 0) return cudaSuccess;
    return launch_kernel(timeline_fold_kernel, dim3(1), dim3(256), 0, st, 0, c->stamps, c->tl_next,
                         c->stamps + 2 * (size_t)c->stamps_cap, c->stamps_cap);
}

#define LAUNCH(kind, expr)                   \
    do {                                     \
        CU_TRY(prof_mark(c, (kind), st));    \
        CU_TRY(expr);                        \
        CU_TRY(prof_mark(c, -1, st));        \
        ++launches;                          \
    } while (0)

// ... for a launch whose argument struct carries a stamp slot
#define LAUNCH_S(kind, args, expr)                \
    do {                                          \
        (args).stamp = next_stamp(c, (kind));     \
        LAUNCH(kind, expr);                       \
    } while (0)

size_t esize(const spd_dims &d) { return d.dtype == 0 ? 4 : 2; }

int stamp_slots(const spd_dims &d) { return 6 * d.n_layers + 16; }

// M = tokens of the launch.  decode: few tokens, the weight-streaming GEMMs are cut along K so
// that about two CTAs per SM are in flight; prefill: no K splits.
Plan make_plan(const spd_dims &d, int M, bool decode, int max_context, int attn_override = 0)
{
    Plan p{};
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn, T = d.T;
    p.qkv_splits = p.gu_splits = p.down_splits = p.o_per_group = 1;
    if (decode && d.dtype == 1) {
        // tcgen05 path: 128-row weight tiles, 64-wide K blocks, uneven splits allowed, >= 4 blocks each
        const int tok_tiles = cdiv(M, 64);
        auto cap = [](int kb) { int c = kb / 4; return c < 1 ? 1 : (c > 16 ? 16 : c); };
        p.qkv_splits = want_splits((long)(cdiv(qd, 128) + 2 * cdiv(kd, 128)) * tok_tiles, cap(cdiv(H, 64)));
        p.gu_splits = want_splits((long)cdiv(F / T, 128) * T * 2 * tok_tiles, cap(cdiv(H, 64)));
        p.down_splits = want_splits((long)cdiv(H, 128) * tok_tiles, cap(cdiv(F, 64)));
        p.o_per_group = want_splits((long)cdiv(H, 128) * T * tok_tiles, cap(cdiv(qd / T, 64)));
    } else if (decode) {
        const long mt = cdiv(M, 64);
        p.qkv_splits = fit_splits(H, want_splits(mt * cdiv(qd, 64), 16), 16);
        p.gu_splits = fit_splits(H, want_splits(mt * cdiv(F, 64), 16), 16);
        p.down_splits = fit_splits(F, want_splits(mt * cdiv(H, 64), 16), 16);
        p.o_per_group = fit_splits(qd / T, cdiv(want_splits(mt * cdiv(H, 64), 16), T), 16);
    }
    p.qkv_kps = H / p.qkv_splits;
    p.gu_kps = H / p.gu_splits;
    p.down_kps = F / p.down_splits;
    p.o_kps = qd / (T * p.o_per_group);
    p.attn_splits = 1;
    if (decode) {
        // decode attention: up to four thread blocks per SM, at least four 16-token pages each
        const int group = d.n_q_heads / d.n_kv_heads;
        const int gt = decode_uses_mma(group, d.head_dim, d.dtype == 1, d.kv_block_size) ? decode_heads_per_block_mma(group)
                                                                                           : decode_heads_per_block(group);
        const long ctas = (long)M * (d.n_q_heads / gt);
        const int pages = cdiv(max_context, 16);
        int s = attn_override > 0 ? attn_override : (int)((4L * sm_count()) / ctas);
        if (s < 1) s = 1;
        if (s > pages / 4) s = pages / 4;
        if (s > 32) s = 32;
        // Up to 8 ranges merge through cluster shared memory; more go through global partial results and a
        // last-arriver merge, which only pays when a range is still long (measured at 70B dims, one sequence of
        // 2k tokens: 8 ranges 17 us per block, 16 ranges 21 us, 32 ranges 27 us).
        if (attn_override <= 0 && s > 8 && pages / 8 <= 64) s = 8;
        if (s < cdiv(pages, DECODE_MAX_PAGES_PER_BLOCK)) s = cdiv(pages, DECODE_MAX_PAGES_PER_BLOCK);
        p.attn_splits = s < 1 ? 1 : s;
    }
    return p;
}

// K ranges of a fused decode GEMM: as many as keep the launch within the thread blocks that are resident
// at once (three per SM at 16-token tiles, two at 32 and 64 tokens: the operand ring is 72-98 KB), each at
// least four K blocks long, at most `max_ranges` (the ranges of one output tile form a thread-block
// cluster of at most 8 blocks).
int decode_splits(long tiles, int num_kb, int override_, int max_ranges, int blocks_per_sm = 3)
{
    long s = override_ > 0 ? override_ : ((long)blocks_per_sm * sm_count()) / (tiles < 1 ? 1 : tiles);
    const long cap = num_kb / 4 < 1 ? 1 : num_kb / 4;
    if (s > cap) s = cap;
    if (s > max_ranges) s = max_ranges;
    return (int)(s < 1 ? 1 : s);
}

// Shape of the four fused decode GEMMs: output tiles per token tile, K blocks per range unit and
// how many ranges the shard structure already contributes (T for the row-split o_proj).
struct SiteGeom { long tiles; int num_kb; int shard_ranges; };
SiteGeom site_geom(const spd_dims &d, int site)
{
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn, T = d.T;
    switch (site) {
    case SITE_QKV: return {cdiv(qd, 128) + 2L * cdiv(kd, 128), cdiv(H, 64), 1};
    case SITE_O: return {(long)cdiv(H, 128) * T, cdiv(qd / T, 64), T};
    case SITE_GU: return {(long)cdiv(F / T, 64) * T, cdiv(H, 64), 1};
    default: return {cdiv(H, 128), cdiv(F, 64), 1};
    }
}

struct Layout {
    size_t res[2], h, q, attn, act, qkv32, proj32, gu32, part_o, part_ml, attn_cnt, rope, err, ss_attn, ss_mlp, stamps, total;
    size_t sm_attn, sm_mlp, lnvec; // block with bias: partial row sums beside the sums of squares; folded-LayerNorm vectors
    size_t Mcap;
};

// Sizes every region for the worse of the two regimes (prefill chunk, decode batch).
Layout make_layout(const spd_dims &d, bool any_spd)
{
    const size_t es = esize(d);
    const size_t H = d.hidden, qd = (size_t)d.n_q_heads * d.head_dim, kd = (size_t)d.n_kv_heads * d.head_dim;
    const size_t F = d.ffn, T = d.T, nqkv = qd + 2 * kd;
    size_t Mp = d.max_prefill_tokens, Md = d.max_batch;
    size_t Mmax = Mp > Md ? Mp : Md;
    Plan pp = make_plan(d, (int)Mp, false, d.max_seq_len);
    Plan pd = make_plan(d, 1, true, d.max_seq_len); // one token gives the largest split counts
    auto mx = [](size_t a, size_t b) { return a > b ? a : b; };
    Layout L;
    L.Mcap = Mmax;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
    L.err = take(256);
    L.res[0] = take(Mmax * H * 4);
    L.res[1] = take(Mmax * H * 4);
    L.h = take((any_spd ? T : 1) * Mmax * H * es);
    L.q = take(Mmax * qd * es);
    L.attn = take(Mmax * qd * es);
    L.act = take(Mmax * F * es);
    L.rope = take(Mmax * (d.head_dim / 2) * sizeof(float2));
    L.qkv32 = take(mx(pp.qkv_splits * Mp, pd.qkv_splits * Md) * nqkv * 4);
    L.proj32 = take(mx(mx(T * pp.o_per_group, (size_t)pp.down_splits) * Mp, mx(T * pd.o_per_group, (size_t)pd.down_splits) * Md) * H * 4);
    L.gu32 = take(mx(pp.gu_splits * Mp, pd.gu_splits * Md) * 2 * F * 4);
    L.part_o = take(Md * d.n_q_heads * 32 * d.head_dim * 4);
    L.part_ml = take(Md * d.n_q_heads * 32 * 2 * 4);
    L.attn_cnt = take(Md * d.n_q_heads * 4);
    // fused decode path: partial sums of squares per 128-column tile
    const size_t h_tiles = (H + 127) / 128;
    L.ss_attn = take(h_tiles * Mmax * 4);
    L.ss_mlp = take(2 * h_tiles * T * Mmax * 4); // the SPD o_proj of the prefill path leaves two partials per tile
    L.stamps = take((size_t)stamp_slots(d) * 16 + ((size_t)stamp_slots(d) + 2) * 8); // slots, then the running totals
    const bool bias_block = d.block_kind == 1 && d.dtype == 1;
    L.sm_attn = take(bias_block ? h_tiles * Mmax * 4 : 0);
    L.sm_mlp = take(bias_block ? 2 * h_tiles * T * Mmax * 4 : 0);
    L.lnvec = take(bias_block ? (size_t)d.n_layers * 2 * (nqkv + F) * 4 : 0); // per layer: wg_qkv, wb_qkv, wg_fc1, wb_fc1
    L.total = off;
    return L;
}

TpLayout tp_layout(const spd_dims &d, int T)
{
    TpLayout L{};
    const size_t H = d.hidden, h_tiles = (H + 127) / 128;
    // rows: a decode batch, or a prompt chunk of up to 2048 tokens
    const long chunk = d.max_prefill_tokens < 2048 ? d.max_prefill_tokens : 2048;
    L.Mb = d.max_batch > chunk ? d.max_batch : chunk;
    L.Md = d.max_batch;
    L.tok_tiles = (int)((L.Md + 15) / 16); // an upper bound for every token box
    L.site_flags = h_tiles * L.tok_tiles * T * TP_FLAG_RANGES;
    L.src_bytes = (size_t)L.Md * H * 4;
    L.buf_bytes = L.src_bytes * T;
    const size_t plane = (size_t)L.Mb * H * 4;
    const int m128_cap = (int)((L.Mb + 127) / 128);
    L.slots_cap = (m128_cap + T - 1) / T;
    L.n_tiles = (int)((H + 255) / 256);
    L.rs_src_stride = (size_t)L.slots_cap * 128 * H * 4;
    L.rs_buf_bytes = L.rs_src_stride * T;
    L.sflag_words = (size_t)L.slots_cap * L.n_tiles * T;
    L.gflag_words = (size_t)m128_cap * tp_finish_blocks_per_tile();
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
    L.step = take(256);
    L.flags = take((size_t)d.n_layers * 2 * L.site_flags * 4);
    L.sflags = take((size_t)d.n_layers * 2 * L.sflag_words * 4);
    L.gflags = take((size_t)d.n_layers * 2 * L.gflag_words * 4);
    L.rx = take(2 * L.buf_bytes);
    L.rs_rx = take(2 * L.rs_buf_bytes);
    L.res0 = take(plane);
    L.res1 = take(plane);
    L.ysave = take(plane);
    L.hg = take((size_t)L.Mb * H * 2);
    L.ss_attn = take(h_tiles * L.Mb * 4);
    L.ss_mlp = take(h_tiles * L.Mb * 4);
    L.total = off;
    return L;
}

int check_dims(const spd_dims *d, const uint8_t *mask)
{
    if (!d || !mask) return SPD_ENULL;
    if (d->n_layers < 1 || d->hidden < 8 || d->n_q_heads < 1 || d->n_kv_heads < 1 || d->ffn < 1) return SPD_EINVAL;
    if (d->T < 1 || d->T > 8) return SPD_EINVAL;
    if (d->dtype != 0 && d->dtype != 1) return SPD_EINVAL;
    if (d->head_dim != 32 && d->head_dim != 64 && d->head_dim != 128) return SPD_EINVAL;
    if (d->n_q_heads % d->n_kv_heads) return SPD_EINVAL;
    if (d->n_q_heads % d->T || d->n_kv_heads % d->T || d->ffn % d->T) return SPD_EINVAL;
    if (d->hidden % 4 || d->hidden > 65536) return SPD_EINVAL;
    if (d->dtype == 1 && (d->hidden % 8 || (d->ffn / d->T) % 8)) return SPD_EINVAL; // 16-byte rows for bf16 tiles
    if (d->kv_block_size < 1 || d->max_batch < 1 || d->max_seq_len < 1 || d->max_prefill_tokens < 1) return SPD_EINVAL;
    if (!(d->rms_eps > 0.f)) return SPD_EINVAL;
    if (d->block_kind != 0 && d->block_kind != 1) return SPD_EINVAL;
    return SPD_OK;
}

int box_index(int box) { return box == 16 ? 0 : (box == 32 ? 1 : (box == 64 ? 2 : 3)); }

// Tensor map of an activation buffer for a token box, built once.
const TcMap *act_map(Ctx *c, ActBuf buf, int box)
{
    const int bi = box_index(box);
    if (c->act_map_ready[buf][bi]) return &c->act_maps[buf][bi];
    const spd_dims &d = c->d;
    const long H = d.hidden, qd = (long)d.n_q_heads * d.head_dim, F = d.ffn, T = d.T, Mc = c->Mcap;
    int rc = -1;
    switch (buf) {
    case AB_H: rc = make_operand_map(&c->act_maps[buf][bi], c->h, H, Mc, c->any_spd ? T : 1, H, Mc * H, box); break;
    case AB_ATTN: rc = make_operand_map(&c->act_maps[buf][bi], c->attn, qd, Mc, 1, qd, 0, box); break;
    case AB_ATTN_SHARD: rc = make_operand_map(&c->act_maps[buf][bi], c->attn, qd / T, Mc, T, qd, qd / T, box); break;
    case AB_ACT: rc = make_operand_map(&c->act_maps[buf][bi], c->act, F, Mc, 1, F, 0, box); break;
    case AB_ACT_SHARD: rc = make_operand_map(&c->act_maps[buf][bi], c->act, F / T, Mc, T, F, F / T, box); break;
    case AB_Q: rc = make_operand_map(&c->act_maps[buf][bi], c->q, qd, Mc, 1, qd, 0, box); break;
    default: break;
    }
    if (rc) return nullptr;
    c->act_map_ready[buf][bi] = true;
    return &c->act_maps[buf][bi];
}

#define MAP_OR_FAIL(var, expr)                     \
    const TcMap *var = (expr);                     \
    if (!var) { g_last_cuda_error = (int)cudaErrorInvalidValue; return SPD_ECUDA; }

template <typename T>
int run_tokens(Ctx *c, const void *x, void *out, int M, TokMap tm, const int32_t *bt, int max_pages,
               bool decode, int max_context, cudaStream_t st)
{
    constexpr bool TC = sizeof(T) == 2; // bf16 -> tcgen05 GEMMs; float32 -> CUDA-core GEMMs
    const spd_dims &d = c->d;
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn, Tn = d.T;
    const int nqkv = qd + 2 * kd;
    const long Mc = c->Mcap;
    const Plan p = make_plan(d, M, decode, max_context);
    PageTable pt{bt, max_pages, c->n_pages, d.kv_block_size, d.n_kv_heads};
    const bool swap = decode;
    const int tbox = TC ? tc_token_box(swap, M) : 0;
    int launches = 0;
    const bool opt = d.block_kind == 1;              // block with bias (Sec. 4.1.2): LayerNorm, biases, ReLU, no rotary
    const bool rope_on = d.rope_base > 0.f && !opt;

    if (rope_on) LAUNCH(K_ROPE_TABLE, launch_rope_table(c->rope, tm, M, d.head_dim, d.rope_base, st));

    // block input -> fp32 residual stream and its attention RMSNorm
    {
        NormArgs a{};
        a.x_in = x; a.res_out = c->res[0]; a.h_out = c->h; a.h_stride = Mc * H;
        a.gain = c->layers[0].attn_norm; a.n_groups = 1; a.per_group = 0; a.M = M; a.H = H; a.eps = d.rms_eps;
        if (opt) a.shift = c->layers[0].attn_norm_b;
        LAUNCH(K_NORM, launch_residual_norm<T>(a, st));
    }
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c->layers[l];
        const bool sync = c->mask[l] != 0;
        // a2: column-split Q/K/V projections of all shards = the full matrices
        {
            const void *wm[3] = {w.wq, w.wk, w.wv};
            const int wn[3] = {qd, kd, kd}, wcol[3] = {0, qd, qd + kd};
            if (TC) {
                // one launch over the three matrices
                const TcMap *wmaps[3] = {&c->maps[l].wq, &c->maps[l].wk, &c->maps[l].wv};
                MAP_OR_FAIL(am, act_map(c, AB_H, tbox));
                TcGemmArgs g{};
                g.C = c->qkv32; g.ldc = nqkv; g.c_batch_stride = 0; g.c_split_stride = (long)M * nqkv;
                for (int i = 0; i < 3; ++i) { g.w_rows[i] = wn[i]; g.c_off[i] = wcol[i]; }
                g.t_rows = M; g.batches = 1; g.w_batched = 0; g.t_batched = 0;
                g.num_kb = cdiv(H, 64); g.splits = p.qkv_splits; g.err = c->err;
                LAUNCH(K_QKV, launch_gemm_tc(wmaps, 3, *am, g, swap, st));
            }
            for (int i = 0; i < 3 && !TC; ++i) {
                {
                    GemmProblem g{};
                    g.A = c->h; g.lda = H; g.a_shard_stride = 0; g.W = wm[i]; g.ldw = H;
                    g.C = c->qkv32 + wcol[i]; g.ldc = nqkv; g.c_split_stride = (long)M * nqkv;
                    g.M = M; g.n_per_shard = wn[i]; g.n_shards = 1; g.K = H; g.splits = p.qkv_splits; g.k_per_split = p.qkv_kps;
                    LAUNCH(K_QKV, launch_gemm_simt<T>(g, st));
                }
            }
        }
        // a3: rotary embedding, KV-page append
        {
            RopeKvArgs a{};
            a.qkv = c->qkv32; a.ldq = nqkv; a.split_stride = (long)M * nqkv; a.splits = p.qkv_splits;
            a.table = c->rope; a.q_out = c->q; a.k_pages = w.k_pages; a.v_pages = w.v_pages; a.pt = pt; a.tm = tm;
            a.M = M; a.n_q_heads = d.n_q_heads; a.head_dim = d.head_dim; a.use_rope = rope_on; a.err = c->err;
            if (opt) { a.bq = w.bq; a.bk = w.bk; a.bv = w.bv; }
            LAUNCH(K_ROPE_KV, launch_rope_kv<T>(a, st));
        }
        // a4: attention, each shard over its own heads
        {
            AttnArgs a{};
            a.q = c->q; a.k_pages = w.k_pages; a.v_pages = w.v_pages; a.pt = pt; a.tm = tm; a.out = c->attn;
            a.M = M; a.n_q_heads = d.n_q_heads; a.head_dim = d.head_dim; a.B = M; a.splits = p.attn_splits;
            a.max_context = max_context; a.part_o = c->part_o; a.part_ml = c->part_ml; a.counters = c->attn_cnt; a.err = c->err;
            if (!decode && d.dtype == 1 && d.head_dim == 128 && d.kv_block_size == 16) {
                MAP_OR_FAIL(qm, act_map(c, AB_Q, 128));
                a.q_map = qm; a.k_map = &c->maps[l].kpages; a.v_map = &c->maps[l].vpages; a.rescale_log2 = (float)c->prefill_rescale_log2;
            }
            if (decode) LAUNCH(K_ATTN, launch_decode_attention<T>(a, st));
            else LAUNCH(K_ATTN, launch_prefill_attention<T>(a, st));
        }
        // a5: row-split output projection.  Plane (i, j) holds the part of Y_i that comes from
        // sub-range j of shard i's K slice.  A synchronous block in prefill needs only the sum:
        // one plane over all of K.
        const bool o_single = sync && !decode;
        const int o_planes = o_single ? 1 : Tn * p.o_per_group;
        if (TC) {
            MAP_OR_FAIL(am, act_map(c, o_single ? AB_ATTN : AB_ATTN_SHARD, tbox));
            TcGemmArgs g{};
            g.C = c->proj32; g.ldc = H; g.c_batch_stride = (long)p.o_per_group * M * H; g.c_split_stride = (long)M * H;
            g.t_rows = M; g.w_rows[0] = H; g.batches = o_single ? 1 : Tn; g.w_batched = !o_single; g.t_batched = !o_single;
            g.num_kb = cdiv(o_single ? qd : qd / Tn, 64); g.splits = o_single ? 1 : p.o_per_group; g.err = c->err;
            const TcMap *wmaps[1] = {o_single ? &c->maps[l].wo_full : &c->maps[l].wo_shard};
            LAUNCH(K_OPROJ, launch_gemm_tc(wmaps, 1, *am, g, swap, st));
        } else {
            GemmProblem g{};
            g.A = c->attn; g.lda = qd; g.W = w.wo; g.ldw = qd; g.C = c->proj32; g.ldc = H; g.c_split_stride = (long)M * H;
            g.M = M; g.n_per_shard = H; g.n_shards = 1; g.K = qd; g.splits = o_planes; g.k_per_split = o_single ? qd : p.o_kps;
            LAUNCH(K_OPROJ, launch_gemm_simt<T>(g, st));
        }
        // a6 + a7: sync-point #1 (sync) or its drop (SPD), residual add, MLP RMSNorm
        {
            NormArgs a{};
            a.res_in = c->res[0]; a.part = c->proj32; a.part_stride = (long)M * H;
            a.n_groups = sync ? 1 : Tn; a.per_group = sync ? o_planes : p.o_per_group;
            a.res_out = c->res[1]; a.h_out = c->h; a.h_stride = Mc * H; a.gain = w.mlp_norm;
            a.M = M; a.H = H; a.eps = d.rms_eps;
            // Y_i = P_i + b: b enters every device's MLP input and, once, the carried residual
            if (opt) { a.bias = w.bo; a.shift = w.mlp_norm_b; }
            LAUNCH(K_NORM, launch_residual_norm<T>(a, st));
        }
        // a8: column-split gate / up; in an SPD block shard i reads its own MLP input plane
        {
            const void *gm[2] = {w.w_gate, w.w_up};
            if (TC) {
                // gate and up in one launch: same token operand, two weight matrices
                const TcMap *wmaps[2] = {&c->maps[l].w_gate, &c->maps[l].w_up};
                MAP_OR_FAIL(am, act_map(c, AB_H, tbox));
                TcGemmArgs g{};
                g.C = c->gu32; g.ldc = F; g.c_batch_stride = F / Tn; g.c_split_stride = (long)M * F;
                g.c_off[0] = 0; g.c_off[1] = (long)p.gu_splits * M * F;
                g.t_rows = M; g.w_rows[0] = g.w_rows[1] = F / Tn; g.batches = Tn; g.w_batched = 1; g.t_batched = sync ? 0 : 1;
                g.num_kb = cdiv(H, 64); g.splits = p.gu_splits; g.err = c->err;
                LAUNCH(K_GATE_UP, launch_gemm_tc(wmaps, opt ? 1 : 2, *am, g, swap, st));
            }
            for (int i = 0; i < (opt ? 1 : 2) && !TC; ++i) {
                float *Cg = c->gu32 + (long)i * p.gu_splits * M * F;
                {
                    GemmProblem g{};
                    g.A = c->h; g.lda = H; g.a_shard_stride = sync ? 0 : Mc * H; g.W = gm[i]; g.ldw = H;
                    g.C = Cg; g.ldc = F; g.c_split_stride = (long)M * F;
                    g.M = M; g.n_per_shard = F / Tn; g.n_shards = Tn; g.K = H; g.splits = p.gu_splits; g.k_per_split = p.gu_kps;
                    LAUNCH(K_GATE_UP, launch_gemm_simt<T>(g, st));
                }
            }
        }
        {
            SiluMulArgs a{};
            a.gate = c->gu32; a.up = c->gu32 + (long)p.gu_splits * M * F; a.ld = F; a.split_stride = (long)M * F;
            a.splits = p.gu_splits; a.act = c->act; a.M = M; a.F = F;
            if (opt) { a.relu = 1; a.bias = w.b_fc1; }
            LAUNCH(K_SILU_MUL, launch_silu_mul<T>(a, st));
        }
        // a9: row-split down projection; summing over all of K = F IS the kept sync-point
        if (TC) {
            MAP_OR_FAIL(am, act_map(c, AB_ACT, tbox));
            TcGemmArgs g{};
            g.C = c->proj32; g.ldc = H; g.c_batch_stride = 0; g.c_split_stride = (long)M * H;
            g.t_rows = M; g.w_rows[0] = H; g.batches = 1; g.w_batched = 0; g.t_batched = 0;
            g.num_kb = cdiv(F, 64); g.splits = p.down_splits; g.err = c->err;
            const TcMap *wmaps[1] = {&c->maps[l].w_down};
            LAUNCH(K_DOWN, launch_gemm_tc(wmaps, 1, *am, g, swap, st));
        } else {
            GemmProblem g{};
            g.A = c->act; g.lda = F; g.W = w.w_down; g.ldw = F; g.C = c->proj32; g.ldc = H; g.c_split_stride = (long)M * H;
            g.M = M; g.n_per_shard = H; g.n_shards = 1; g.K = F; g.splits = p.down_splits; g.k_per_split = p.down_kps;
            LAUNCH(K_DOWN, launch_gemm_simt<T>(g, st));
        }
        // a10: output residual.  res[1] already holds X + sum_i Y_i in both modes
        // (sync: R; SPD: Y_i before the sum, X after it), so out = res[1] + sum_i Z_i.
        {
            NormArgs a{};
            a.res_in = c->res[1]; a.part = c->proj32; a.part_stride = (long)M * H; a.n_groups = 1; a.per_group = p.down_splits;
            a.res_out = c->res[0]; a.M = M; a.H = H; a.eps = d.rms_eps;
            if (opt) a.bias = w.b_fc2;
            if (l + 1 < d.n_layers) {
                a.h_out = c->h; a.h_stride = Mc * H; a.gain = c->layers[l + 1].attn_norm;
                if (opt) a.shift = c->layers[l + 1].attn_norm_b;
            } else a.final_out = out;
            LAUNCH(K_NORM, launch_residual_norm<T>(a, st));
        }
    }
    c->launches_last = launches;
    return SPD_OK;
}

// Baseline of the rank mode (Sec. 3): ONE shard's stack (a context created with T = 1 from the shard's dims and
// weights, as for spd_tp_attach) run through the unfused kernels, with every shard sum the block keeps handed to
// a caller-supplied all-reduce - a library collective (NCCL) between kernels instead of the exchange inside the
// projection's tail.  A TP block calls it twice (Y_r after o_proj, Z_r after down), an SPD block once
// (Y_r + Z_r after down; R_r = X + Y_r stays on the rank, X joins after the sum: Sec. 4.1.1).
// scratch: 2 * M * H floats.  cur / other: the two residual-stream buffers.
int run_tp_baseline(Ctx *c, const void *x, void *out, int M, TokMap tm, const int32_t *bt, int max_pages, bool decode,
                    int max_context, float *scratch, spd_allreduce_fn fn, void *user, cudaStream_t st)
{
    const spd_dims &d = c->d;
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn;
    const int nqkv = qd + 2 * kd;
    const long Mc = c->Mcap;
    const Plan p = make_plan(d, M, decode, max_context);
    PageTable pt{bt, max_pages, c->n_pages, d.kv_block_size, d.n_kv_heads};
    const bool swap = decode;
    const int tbox = tc_token_box(swap, M);
    const bool rope_on = d.rope_base > 0.f;
    const long MH = (long)M * H;
    float *ybuf = scratch, *zbuf = scratch + MH;
    float *cur = c->res[0], *other = c->res[1];
    int launches = 0;
    // dst = base + sum of n planes (fp32 [M][H] each); base may be null (then plane 0 serves as base)
    auto add_planes = [&](float *dst, const float *base, const float *planes, int n) -> cudaError_t {
        NormArgs a{};
        a.res_in = base ? base : planes;
        a.part = base ? planes : (n > 1 ? planes + MH : nullptr);
        a.part_stride = MH; a.n_groups = 1; a.per_group = base ? n : n - 1;
        a.res_out = dst; a.M = M; a.H = H; a.eps = d.rms_eps;
        return launch_residual_norm<bf16>(a, st);
    };
    auto all_reduce = [&](float *buf) -> int {
        if (fn(user, buf, (size_t)MH, (void *)st) != 0) return SPD_ECALLBACK;
        return SPD_OK;
    };
    auto gemm = [&](Kind kind, const TcMap *const *wmaps, int nw, ActBuf ab, float *C, long ldc, const int *w_rows, const long *c_off,
                    int K, int splits) -> int {
        MAP_OR_FAIL(am, act_map(c, ab, tbox));
        TcGemmArgs g{};
        g.C = C; g.ldc = ldc; g.c_batch_stride = 0; g.c_split_stride = (long)M * ldc;
        for (int i = 0; i < nw; ++i) { g.w_rows[i] = w_rows[i]; g.c_off[i] = c_off[i]; }
        g.t_rows = M; g.batches = 1; g.w_batched = 0; g.t_batched = 0;
        g.num_kb = cdiv(K, 64); g.splits = splits; g.err = c->err;
        LAUNCH(kind, launch_gemm_tc(wmaps, nw, *am, g, swap, st));
        return SPD_OK;
    };

    if (rope_on) LAUNCH(K_ROPE_TABLE, launch_rope_table(c->rope, tm, M, d.head_dim, d.rope_base, st));
    {
        NormArgs a{};
        a.x_in = x; a.res_out = cur; a.h_out = c->h; a.h_stride = Mc * H;
        a.gain = c->layers[0].attn_norm; a.n_groups = 1; a.per_group = 0; a.M = M; a.H = H; a.eps = d.rms_eps;
        LAUNCH(K_NORM, launch_residual_norm<bf16>(a, st));
    }
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c->layers[l];
        const LayerMaps &lm = c->maps[l];
        const bool sync = c->mask[l] != 0;
        int rc;
        {   // a2 - a4 on the rank's own heads
            const TcMap *wmaps[3] = {&lm.wq, &lm.wk, &lm.wv};
            const int wn[3] = {qd, kd, kd};
            const long wcol[3] = {0, qd, (long)qd + kd};
            if ((rc = gemm(K_QKV, wmaps, 3, AB_H, c->qkv32, nqkv, wn, wcol, H, p.qkv_splits)) != SPD_OK) return rc;
            RopeKvArgs a{};
            a.qkv = c->qkv32; a.ldq = nqkv; a.split_stride = (long)M * nqkv; a.splits = p.qkv_splits;
            a.table = c->rope; a.q_out = c->q; a.k_pages = w.k_pages; a.v_pages = w.v_pages; a.pt = pt; a.tm = tm;
            a.M = M; a.n_q_heads = d.n_q_heads; a.head_dim = d.head_dim; a.use_rope = rope_on; a.err = c->err;
            LAUNCH(K_ROPE_KV, launch_rope_kv<bf16>(a, st));
            AttnArgs t{};
            t.q = c->q; t.k_pages = w.k_pages; t.v_pages = w.v_pages; t.pt = pt; t.tm = tm; t.out = c->attn;
            t.M = M; t.n_q_heads = d.n_q_heads; t.head_dim = d.head_dim; t.B = M; t.splits = p.attn_splits;
            t.max_context = max_context; t.part_o = c->part_o; t.part_ml = c->part_ml; t.counters = c->attn_cnt; t.err = c->err;
            if (!decode && d.head_dim == 128 && d.kv_block_size == 16) {
                MAP_OR_FAIL(qm, act_map(c, AB_Q, 128));
                t.q_map = qm; t.k_map = &lm.kpages; t.v_map = &lm.vpages; t.rescale_log2 = (float)c->prefill_rescale_log2;
            }
            if (decode) LAUNCH(K_ATTN, launch_decode_attention<bf16>(t, st));
            else LAUNCH(K_ATTN, launch_prefill_attention<bf16>(t, st));
        }
        {   // a5: the rank's partial attention output Y_r, in K-range planes, then as one [M][H] buffer
            const TcMap *wmaps[1] = {&lm.wo_full};
            const int wn[1] = {H};
            const long wcol[1] = {0};
            if ((rc = gemm(K_OPROJ, wmaps, 1, AB_ATTN, c->proj32, H, wn, wcol, qd, p.o_per_group)) != SPD_OK) return rc;
            LAUNCH(K_NORM, add_planes(ybuf, nullptr, c->proj32, p.o_per_group));
        }
        // a6: sync-point 1 is an all-reduce of Y_r in a TP block and is dropped in an SPD block (R_r = X + Y_r)
        if (sync && (rc = all_reduce(ybuf)) != SPD_OK) return rc;
        {   // a7
            NormArgs a{};
            a.res_in = cur; a.part = ybuf; a.part_stride = MH; a.n_groups = 1; a.per_group = 1;
            a.res_out = other; a.h_out = c->h; a.h_stride = Mc * H; a.gain = w.mlp_norm; a.M = M; a.H = H; a.eps = d.rms_eps;
            LAUNCH(K_NORM, launch_residual_norm<bf16>(a, st));
        }
        {   // a8, a9 on the rank's MLP slice
            const TcMap *wmaps[2] = {&lm.w_gate, &lm.w_up};
            const int wn[2] = {F, F};
            const long wcol[2] = {0, (long)p.gu_splits * M * F};
            if ((rc = gemm(K_GATE_UP, wmaps, 2, AB_H, c->gu32, F, wn, wcol, H, p.gu_splits)) != SPD_OK) return rc;
            SiluMulArgs a{};
            a.gate = c->gu32; a.up = c->gu32 + (long)p.gu_splits * M * F; a.ld = F; a.split_stride = (long)M * F;
            a.splits = p.gu_splits; a.act = c->act; a.M = M; a.F = F;
            LAUNCH(K_SILU_MUL, launch_silu_mul<bf16>(a, st));
            const TcMap *dmaps[1] = {&lm.w_down};
            const int dn[1] = {H};
            const long dcol[1] = {0};
            if ((rc = gemm(K_DOWN, dmaps, 1, AB_ACT, c->proj32, H, dn, dcol, F, p.down_splits)) != SPD_OK) return rc;
        }
        // the kept sync-point: Z_r in a TP block, Y_r + Z_r in an SPD block
        LAUNCH(K_NORM, add_planes(zbuf, sync ? nullptr : ybuf, c->proj32, p.down_splits));
        if ((rc = all_reduce(zbuf)) != SPD_OK) return rc;
        {   // a10: TP block out = R + sum Z; SPD block out = X + sum (Y + Z)
            // TP block: R (in other) + sum Z goes back into the block's input buffer.  SPD block: X (still in cur) + the
            // sum goes over R_r, which is no longer needed, and the two buffers change roles.
            NormArgs a{};
            a.res_in = sync ? other : cur; a.part = zbuf; a.part_stride = MH; a.n_groups = 1; a.per_group = 1;
            a.res_out = sync ? cur : other; a.M = M; a.H = H; a.eps = d.rms_eps;
            if (l + 1 < d.n_layers) { a.h_out = c->h; a.h_stride = Mc * H; a.gain = c->layers[l + 1].attn_norm; }
            else a.final_out = out;
            LAUNCH(K_NORM, launch_residual_norm<bf16>(a, st));
            if (!sync) { float *t2 = cur; cur = other; other = t2; }
        }
    }
    c->launches_last = launches;
    return SPD_OK;
}

// One decode step of the bf16 stack with the fused projections: per block QKV(+rotary, KV append),
// paged attention, o_proj(+residuals, MLP norm input), gate/up(+SwiGLU), down(+shard sum, residual).
int run_decode_fused(Ctx *c, const void *x, void *out, int M, TokMap tm, const int32_t *bt, int max_pages,
                     int max_context, cudaStream_t st)
{
    const spd_dims &d = c->d;
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn, Tn = d.T;
    const int Fs = F / Tn;
    const long Mc = c->Mcap;
    const Plan p = make_plan(d, M, true, max_context, c->split_override[SITE_ATTN]);
    PageTable pt{bt, max_pages, c->n_pages, d.kv_block_size, d.n_kv_heads};
    const int tbox = tc_token_box(true, M);
    const int tok_tiles = cdiv(M, tbox), h_tiles = cdiv(H, 128);
    int launches = 0;
    // block with bias (Sec. 4.1.2): LayerNorm folded into the QKV / fc1 tails, biases in the tails, ReLU, no rotary embedding
    const bool opt = d.block_kind == 1;
    const bool rope = d.rope_base > 0.f && !opt;
    const int nqkv = qd + 2 * kd;
    auto lnvec = [&](int l) { return c->lnvec + (size_t)l * 2 * (nqkv + F); }; // wg_qkv, wb_qkv, wg_fc1, wb_fc1
    // K ranges of a site: automatic or overridden; a tile's ranges (times the shards for o_proj) fit a cluster of 8
    auto splits_of = [&](int site) {
        const SiteGeom sg = site_geom(d, site);
        return decode_splits(sg.tiles * tok_tiles, sg.num_kb, c->split_override[site], 8 / sg.shard_ranges, tbox == 16 ? 3 : 2);
    };
    {
        PrologueArgs a{};
        a.x = x; a.res_out = c->res[0]; a.gain = c->layers[0].attn_norm; a.hg = c->h; a.ss_out = c->ss_attn;
        a.Mcap = Mc; a.M = M; a.H = H;
        if (rope) { a.rope_table = c->rope; a.tm = tm; a.head_dim = d.head_dim; a.rope_base = d.rope_base; }
        if (opt) a.sum_out = c->sm_attn;
        LAUNCH_S(K_NORM, a, launch_decode_prologue(a, st));
    }
    auto base_args = [&]() {
        DecGemmArgs g{};
        g.t_rows = M; g.err = c->err; g.H = H; g.Mcap = Mc; g.batches = 1; g.n_weights = 1; g.n_groups = 1;
        g.l2_prefetch_kb = c->l2_prefetch_kb;
        g.ring_stages = c->ring_stages;
        g.planes_per_block = c->oproj_planes;
        return g;
    };
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c->layers[l];
        const bool sync = c->mask[l] != 0;
        {   // a2 + a3
            DecGemmArgs g = base_args();
            const TcMap *wmaps[3] = {&c->maps[l].wq, &c->maps[l].wk, &c->maps[l].wv};
            MAP_OR_FAIL(am, act_map(c, AB_H, tbox));
            g.n_weights = 3; g.w_rows[0] = qd; g.w_rows[1] = g.w_rows[2] = kd;
            g.num_kb = cdiv(H, 64);
            g.splits = splits_of(SITE_QKV);
            g.ss_in = SumSq{c->ss_attn, h_tiles, 1, Mc, H, d.rms_eps, opt ? c->sm_attn : nullptr};
            if (opt) { g.ln_wg = lnvec(l); g.ln_wb = lnvec(l) + nqkv; }
            g.rope = rope ? c->rope : nullptr; g.q_out = c->q; g.k_pages = w.k_pages; g.v_pages = w.v_pages; g.pt = pt; g.tm = tm;
            g.n_q_heads = d.n_q_heads; g.head_dim = d.head_dim;
            LAUNCH_S(K_QKV, g, launch_gemm_decode(EPI_QKV, wmaps, *am, g, st));
        }
        {   // a4
            AttnArgs a{};
            a.q = c->q; a.k_pages = w.k_pages; a.v_pages = w.v_pages; a.pt = pt; a.tm = tm; a.out = c->attn;
            a.M = M; a.n_q_heads = d.n_q_heads; a.head_dim = d.head_dim; a.B = M; a.splits = p.attn_splits;
            a.max_context = max_context; a.part_o = c->part_o; a.part_ml = c->part_ml; a.counters = c->attn_cnt; a.err = c->err;
            if (d.head_dim == 128 && d.kv_block_size == 16) { a.k_map = &c->maps[l].kpage_whole; a.v_map = &c->maps[l].vpage_whole; }
            LAUNCH_S(K_ATTN, a, launch_decode_attention<bf16>(a, st));
        }
        {   // a5 - a7: shard i's K slice gives the plane group Y_i
            DecGemmArgs g = base_args();
            const TcMap *wmaps[1] = {&c->maps[l].wo_shard};
            MAP_OR_FAIL(am, act_map(c, AB_ATTN_SHARD, tbox));
            g.w_rows[0] = H; g.batches = Tn; g.w_batched = 1; g.t_batched = 1; g.z_is_plane = 1;
            g.num_kb = cdiv(qd / Tn, 64);
            g.splits = splits_of(SITE_O);
            g.res_in = c->res[0]; g.res_out = c->res[1]; g.gain = w.mlp_norm; g.hg = c->h; g.hg_stride = Mc * H;
            g.ss_out = c->ss_mlp;
            g.n_groups = sync ? 1 : Tn;
            if (opt) { g.bias = w.bo; g.sum_out = c->sm_mlp; } // Y_i = P_i + b: b once in the stream, and in every device's MLP input
            LAUNCH_S(K_OPROJ, g, launch_gemm_decode(EPI_OPROJ, wmaps, *am, g, st));
        }
        {   // a8: 64 gate rows and the 64 up rows of the same FFN columns per tile
            DecGemmArgs g = base_args();
            const TcMap *wmaps[2] = {&c->maps[l].w_gate64, &c->maps[l].w_up64};
            MAP_OR_FAIL(am, act_map(c, AB_H, tbox));
            g.n_weights = 2; g.w_rows[0] = g.w_rows[1] = Fs; g.batches = Tn; g.w_batched = 1; g.t_batched = sync ? 0 : 1;
            g.num_kb = cdiv(H, 64);
            g.splits = splits_of(SITE_GU);
            g.ss_in = SumSq{c->ss_mlp, h_tiles, sync ? 1 : Tn, Mc, H, d.rms_eps, opt ? c->sm_mlp : nullptr};
            if (opt) {   // fc1 alone: 128 of its rows per tile, bias and ReLU in the tail
                g.n_weights = 1; g.fc1_only = 1; g.ln_wg = lnvec(l) + 2 * nqkv; g.ln_wb = lnvec(l) + 2 * nqkv + F;
                g.splits = decode_splits((long)cdiv(Fs, 128) * Tn * tok_tiles, g.num_kb, c->split_override[SITE_GU], 8, tbox == 16 ? 3 : 2);
            }
            g.rstd_per_shard = sync ? 0 : 1;
            g.act = c->act; g.F = F; g.Fs = Fs;
            LAUNCH_S(K_GATE_UP, g, launch_gemm_decode(EPI_GATEUP, wmaps, *am, g, st));
        }
        {   // a9 + a10: res[1] holds X + sum_i Y_i in both modes, so out = res[1] + sum_i Z_i
            DecGemmArgs g = base_args();
            const TcMap *wmaps[1] = {&c->maps[l].w_down};
            MAP_OR_FAIL(am, act_map(c, AB_ACT, tbox));
            g.w_rows[0] = H;
            g.num_kb = cdiv(F, 64);
            g.splits = splits_of(SITE_DOWN);
            g.res_in = c->res[1]; g.res_out = c->res[0];
            if (l + 1 < d.n_layers) { g.gain = c->layers[l + 1].attn_norm; g.hg = c->h; g.hg_stride = Mc * H; g.ss_out = c->ss_attn; }
            else g.final_out = out;
            if (opt) { g.bias = w.b_fc2; if (l + 1 < d.n_layers) g.sum_out = c->sm_attn; }
            LAUNCH_S(K_DOWN, g, launch_gemm_decode(EPI_DOWN, wmaps, *am, g, st));
        }
    }
    c->launches_last = launches;
    return SPD_OK;
}

// One decode step of M tokens in rank mode (tensor parallelism across GPUs, Sec. 3): every local rank runs
// the block on its own shard and its own copy of the residual stream; the shard sums that the block keeps
// (o_proj of a TP block, down of every block; Sec. 4.1.1) are one-shot exchanges with the other ranks of the
// group inside the projection's tail.  out: rank z's [M][H] rows lie out_stride bytes after rank z-1's.
int run_tp(Ctx *c, const void *x, void *out, long out_stride, int M, TokMap tm, const int32_t *bt, int max_pages,
           int max_context, cudaStream_t st)
{
    constexpr bool decode = true;
    const spd_dims &d = c->d;
    TpState &tp = c->tp;
    const TpLayout &TL = tp.L;
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn, nl = d.T;
    const int Fs = F / nl;
    const long Mb = TL.Mb;
    const Plan p = make_plan(d, M, decode, max_context, c->split_override[SITE_ATTN]);
    PageTable pt{bt, max_pages, c->n_pages, d.kv_block_size, d.n_kv_heads};
    const int tbox = tc_token_box(true, M);
    const int tok_tiles = cdiv(M, tbox), h_tiles = cdiv(H, 128);
    if (tok_tiles > TL.tok_tiles || M > TL.Md) return SPD_EINVAL;
    const TcMap *hmap = &tp.h_maps[box_index(tbox)];
    int launches = 0;
    const bool rope = d.rope_base > 0.f;
    char *r0 = tp.regions[tp.rank_base];
    {   // a1 of the first block for every local rank; the ranks' step numbers advance
        PrologueArgs a{};
        a.x = x; a.res_out = (float *)(r0 + TL.res0); a.gain = c->layers[0].attn_norm; a.hg = r0 + TL.hg;
        a.ss_out = (float *)(r0 + TL.ss_attn); a.Mcap = Mb; a.M = M; a.H = H;
        a.n_z = nl; a.z_stride = tp.z_stride; a.step = (unsigned *)(r0 + TL.step);
        if (rope) { a.rope_table = c->rope; a.tm = tm; a.head_dim = d.head_dim; a.rope_base = d.rope_base; }
        LAUNCH_S(K_NORM, a, launch_decode_prologue(a, st));
    }
    auto base_args = [&]() {
        DecGemmArgs g{};
        g.t_rows = M; g.err = c->err; g.H = H; g.Mcap = Mb; g.batches = nl; g.w_batched = 1; g.t_batched = 1;
        g.n_weights = 1; g.n_groups = 1;
        g.ring_stages = c->ring_stages;
        g.planes_per_block = c->oproj_planes;
        g.tp.on = 1; g.tp.T = tp.T; g.tp.rank_base = tp.rank_base; g.tp.z_stride = tp.z_stride;
        g.tp.step = (const unsigned *)(r0 + TL.step);
        g.tp.wait_ns = (unsigned long long)c->peer_wait_ms * 1000000ull;
        return g;
    };
    int exchange = 0;
    // the exchange of block l at site s (0: o_proj, 1: down)
    auto with_exchange = [&](DecGemmArgs &g, int l, int s) {
        g.tp.exchange = 1;
        g.tp.buf = (int)((tp.exchanges + exchange++) & 1);
        g.tp.buf_bytes = (long)TL.buf_bytes; g.tp.src_bytes = (long)TL.src_bytes;
        for (int j = 0; j < tp.T; ++j) {
            g.tp.rx[j] = tp.regions[j] + TL.rx;
            g.tp.flags[j] = (unsigned *)(tp.regions[j] + TL.flags) + ((size_t)l * 2 + s) * TL.site_flags;
        }
    };
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c->layers[l];
        const bool sync = c->mask[l] != 0;
        {   // a2 + a3: rank z projects its own heads from its own copy of the normalised input
            DecGemmArgs g = base_args();
            const TcMap *wmaps[3] = {&tp.qkv_maps[3 * l], &tp.qkv_maps[3 * l + 1], &tp.qkv_maps[3 * l + 2]};
            g.n_weights = 3; g.w_rows[0] = qd / nl; g.w_rows[1] = g.w_rows[2] = kd / nl;
            g.num_kb = cdiv(H, 64);
            g.splits = decode_splits((long)decode_tiles_per_batch(EPI_QKV, g.w_rows, 3) * nl * tok_tiles, g.num_kb,
                                     c->split_override[SITE_QKV], 8, tbox == 16 ? 3 : 2);
            g.ss_in = SumSq{(const float *)(r0 + TL.ss_attn), h_tiles, 1, Mb, H, d.rms_eps};
            g.rope = rope ? c->rope : nullptr; g.q_out = c->q; g.k_pages = w.k_pages; g.v_pages = w.v_pages; g.pt = pt; g.tm = tm;
            g.n_q_heads = d.n_q_heads; g.head_dim = d.head_dim;
            LAUNCH_S(K_QKV, g, launch_gemm_decode(EPI_QKV, wmaps, *hmap, g, st));
        }
        {   // a4: heads are rank-local by construction
            AttnArgs a{};
            a.q = c->q; a.k_pages = w.k_pages; a.v_pages = w.v_pages; a.pt = pt; a.tm = tm; a.out = c->attn;
            a.M = M; a.n_q_heads = d.n_q_heads; a.head_dim = d.head_dim; a.B = M; a.splits = p.attn_splits;
            a.max_context = max_context; a.part_o = c->part_o; a.part_ml = c->part_ml; a.counters = c->attn_cnt; a.err = c->err;
            if (d.head_dim == 128 && d.kv_block_size == 16) { a.k_map = &c->maps[l].kpage_whole; a.v_map = &c->maps[l].vpage_whole; }
            LAUNCH_S(K_ATTN, a, launch_decode_attention<bf16>(a, st));
        }
        {   // a5 - a7: Y_z from the rank's own heads.  TP block: R = X + sum over ranks (sync-point 1);
            // SPD block: the sync-point is dropped, R_z = X + Y_z feeds the rank's MLP and Y_z is kept for a10
            DecGemmArgs g = base_args();
            const TcMap *wmaps[1] = {&c->maps[l].wo_shard};
            MAP_OR_FAIL(am, act_map(c, AB_ATTN_SHARD, tbox));
            g.w_rows[0] = H;
            g.num_kb = cdiv(qd / nl, 64);
            g.splits = decode_splits((long)h_tiles * nl * tok_tiles, g.num_kb, c->split_override[SITE_O], 8, tbox == 16 ? 3 : 2);
            g.res_in = (const float *)(r0 + TL.res0); g.gain = w.mlp_norm; g.hg = r0 + TL.hg; g.ss_out = (float *)(r0 + TL.ss_mlp);
            if (sync) { with_exchange(g, l, 0); g.res_out = (float *)(r0 + TL.res1); }
            else g.tp.ysave = (float *)(r0 + TL.ysave);
            LAUNCH_S(K_OPROJ, g, launch_gemm_decode(EPI_RESID_TP, wmaps, *am, g, st));
        }
        {   // a8
            DecGemmArgs g = base_args();
            const TcMap *wmaps[2] = {&c->maps[l].w_gate64, &c->maps[l].w_up64};
            g.n_weights = 2; g.w_rows[0] = g.w_rows[1] = Fs;
            g.num_kb = cdiv(H, 64);
            g.splits = decode_splits((long)decode_tiles_per_batch(EPI_GATEUP, g.w_rows, 2) * nl * tok_tiles, g.num_kb,
                                     c->split_override[SITE_GU], 8, tbox == 16 ? 3 : 2);
            g.ss_in = SumSq{(const float *)(r0 + TL.ss_mlp), h_tiles, 1, Mb, H, d.rms_eps};
            g.act = c->act; g.F = F; g.Fs = Fs;
            LAUNCH_S(K_GATE_UP, g, launch_gemm_decode(EPI_GATEUP, wmaps, *hmap, g, st));
        }
        {   // a9 + a10, the kept sync-point.  TP block: out = R + sum_z Z_z;  SPD block: out = X + sum_z (Y_z + Z_z)
            DecGemmArgs g = base_args();
            const TcMap *wmaps[1] = {&c->maps[l].wd_shard};
            MAP_OR_FAIL(am, act_map(c, AB_ACT_SHARD, tbox));
            g.w_rows[0] = H;
            g.num_kb = cdiv(Fs, 64);
            g.splits = decode_splits((long)h_tiles * nl * tok_tiles, g.num_kb, c->split_override[SITE_DOWN], 8, tbox == 16 ? 3 : 2);
            with_exchange(g, l, 1);
            g.res_in = (const float *)(r0 + (sync ? TL.res1 : TL.res0));
            if (!sync) g.tp.addend = (const float *)(r0 + TL.ysave);
            g.res_out = (float *)(r0 + TL.res0);
            if (l + 1 < d.n_layers) { g.gain = c->layers[l + 1].attn_norm; g.hg = r0 + TL.hg; g.ss_out = (float *)(r0 + TL.ss_attn); }
            else { g.final_out = out; g.tp.out_stride = out_stride; }
            LAUNCH_S(K_DOWN, g, launch_gemm_decode(EPI_RESID_TP, wmaps, *am, g, st));
        }
    }
    c->launches_last = launches;
    return SPD_OK;
}

// A prompt chunk of M tokens in rank mode at tensor-core speed: every local rank runs the prompt projections
// (gemm_prefill.cu, CTA pairs) on its own shard and its own copy of the residual stream; the shard sums the
// block keeps are two-shot exchanges - the projection's tail scatters the rank's partial rows to the ranks that
// own them (128-token tiles dealt round-robin), the owner adds the T planes in rank order, applies the residual
// and writes the finished rows into every rank's planes, and a small kernel waits for all owners before the next
// projection starts (tp_prefill.cu).  A TP block exchanges Y_r after o_proj and Z_r after down (Sec. 3), an SPD
// block keeps R_r = X + Y_r on the rank and exchanges Y_r + Z_r after down (Sec. 4.1.1).  With several local
// ranks (all ranks on one GPU) every kernel is launched once per rank, all scatters before any finish: no
// kernel then waits for one launched after it.
int run_tp_prefill(Ctx *c, const void *x, void *out, long out_stride, int M, TokMap tm, const int32_t *bt, int max_pages,
                   int max_context, cudaStream_t st)
{
    const spd_dims &d = c->d;
    TpState &tp = c->tp;
    const TpLayout &TL = tp.L;
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn, nl = d.T;
    const int qd_r = qd / nl, kd_r = kd / nl, Fs = F / nl;
    const long Mb = TL.Mb;
    if (M > Mb) return SPD_EINVAL;
    PageTable pt{bt, max_pages, c->n_pages, d.kv_block_size, d.n_kv_heads};
    int launches = 0;
    const bool rope = d.rope_base > 0.f;
    const TcMap *hmap = &tp.h_maps[3]; // 128-token boxes
    auto reg = [&](int z) { return tp.regions[tp.rank_base + z]; };
    const unsigned long long wait_ns = (unsigned long long)c->peer_wait_ms * 1000000ull;
    if (rope) LAUNCH(K_ROPE_TABLE, launch_rope_table(c->rope, tm, M, d.head_dim, d.rope_base, st, next_stamp(c, K_ROPE_TABLE)));
    for (int z = 0; z < nl; ++z) {   // a1 of the first block; the rank's step number advances
        PrologueArgs a{};
        a.x = x; a.res_out = (float *)(reg(z) + TL.res0); a.gain = c->layers[0].attn_norm; a.hg = reg(z) + TL.hg;
        a.ss_out = (float *)(reg(z) + TL.ss_attn); a.Mcap = Mb; a.M = M; a.H = H; a.step = (unsigned *)(reg(z) + TL.step);
        LAUNCH_S(K_NORM, a, launch_prefill_prologue(a, st));
    }
    auto base_args = [&](int z) {
        PreGemmArgs g{};
        g.t_rows = M; g.err = c->err; g.H = H; g.Mcap = Mb; g.batches = 1; g.n_weights = 1; g.pair = 1;
        g.group_m = c->prefill_group_m; g.w_z = z; g.t_z = z;
        return g;
    };
    int exchange = 0;
    // the exchange of block l at site s (0: o_proj, 1: down): scatter by every local rank, then finish, then wait
    auto scatter_args = [&](PreGemmArgs &g, int z, int l, int s, int buf, const float *addend) {
        g.sc.T = tp.T; g.sc.me = tp.rank_base + z; g.sc.n_tiles = TL.n_tiles; g.sc.src_stride = (long)TL.rs_src_stride;
        for (int j = 0; j < tp.T; ++j) {
            g.sc.rx[j] = tp.regions[j] + TL.rs_rx + (size_t)buf * TL.rs_buf_bytes;
            g.sc.flags[j] = (unsigned *)(tp.regions[j] + TL.sflags) + ((size_t)l * 2 + s) * TL.sflag_words;
        }
        g.sc.addend = addend;
        g.sc.step = (const unsigned *)(reg(z) + TL.step);
    };
    auto finish_and_wait = [&](int l, int s, int buf, size_t res_in_off, size_t res_out_off, const void *gain, size_t ss_off) -> int {
        const size_t goff = TL.gflags + (((size_t)l * 2 + s) * TL.gflag_words) * 4;
        for (int z = 0; z < nl; ++z) {
            TpFinishArgs a{};
            a.T = tp.T; a.me = tp.rank_base + z; a.M = M; a.H = H; a.n_tiles = TL.n_tiles;
            a.rx = reg(z) + TL.rs_rx + (size_t)buf * TL.rs_buf_bytes; a.src_stride = (long)TL.rs_src_stride;
            a.sflags = (const unsigned *)(reg(z) + TL.sflags) + ((size_t)l * 2 + s) * TL.sflag_words;
            a.step = (const unsigned *)(reg(z) + TL.step);
            a.res_in = (const float *)(reg(z) + res_in_off); a.gain = gain;
            for (int j = 0; j < tp.T; ++j) a.region[j] = tp.regions[j];
            a.off_res_out = (long)res_out_off; a.off_hg = (long)TL.hg; a.off_ss = (long)ss_off; a.off_gflags = (long)goff;
            a.wait_ns = wait_ns; a.err = c->err;
            LAUNCH_S(K_NORM, a, launch_tp_finish(a, st));
        }
        for (int z = 0; z < nl; ++z)
            LAUNCH(K_NORM, launch_tp_gather_wait((const unsigned *)(reg(z) + goff), M, (const unsigned *)(reg(z) + TL.step), wait_ns, c->err, st));
        return SPD_OK;
    };
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c->layers[l];
        const LayerMaps &lm = c->maps[l];
        const bool sync = c->mask[l] != 0;
        int rc;
        for (int z = 0; z < nl; ++z) {   // a2 + a3: rank z projects its own heads from its own copy of the normalised input
            PreGemmArgs g = base_args(z);
            const TcMap *wmaps[3] = {&tp.qkv_maps[3 * l], &tp.qkv_maps[3 * l + 1], &tp.qkv_maps[3 * l + 2]};
            g.n_weights = 3; g.w_rows[0] = qd_r; g.w_rows[1] = g.w_rows[2] = kd_r;
            g.num_kb = cdiv(H, 64);
            g.ss_in = SumSq{(const float *)(reg(z) + TL.ss_attn), 1, 1, Mb, H, d.rms_eps};
            g.rope = rope ? c->rope : nullptr; g.q_out = c->q; g.k_pages = w.k_pages; g.v_pages = w.v_pages; g.pt = pt; g.tm = tm;
            g.n_q_heads = d.n_q_heads; g.head_dim = d.head_dim;
            g.q_head0 = z * (d.n_q_heads / nl); g.kv_head0 = z * (d.n_kv_heads / nl);
            LAUNCH_S(K_QKV, g, launch_gemm_prefill(PRE_QKV, wmaps, *hmap, g, st));
        }
        {   // a4: heads are rank-local by construction
            AttnArgs a{};
            a.q = c->q; a.k_pages = w.k_pages; a.v_pages = w.v_pages; a.pt = pt; a.tm = tm; a.out = c->attn;
            a.M = M; a.n_q_heads = d.n_q_heads; a.head_dim = d.head_dim; a.B = M; a.splits = 1;
            a.max_context = max_context; a.part_o = c->part_o; a.part_ml = c->part_ml; a.counters = c->attn_cnt; a.err = c->err;
            if (d.head_dim == 128 && d.kv_block_size == 16) {
                MAP_OR_FAIL(qm, act_map(c, AB_Q, 128));
                a.q_map = qm; a.k_map = &lm.kpages; a.v_map = &lm.vpages; a.rescale_log2 = (float)c->prefill_rescale_log2;
            }
            LAUNCH_S(K_ATTN, a, launch_prefill_attention<bf16>(a, st));
        }
        int mlp_tiles = 1;
        MAP_OR_FAIL(attn_map, act_map(c, AB_ATTN_SHARD, 128));
        if (sync) {   // a5 - a7, TP block: sync-point 1 = exchange of Y_r; R = X + sum over ranks
            const int buf = (int)((tp.exchanges + exchange++) & 1);
            for (int z = 0; z < nl; ++z) {
                PreGemmArgs g = base_args(z);
                const TcMap *wmaps[1] = {&lm.wo_shard};
                g.w_rows[0] = H; g.num_kb = cdiv(qd_r, 64);
                scatter_args(g, z, l, 0, buf, nullptr);
                LAUNCH_S(K_OPROJ, g, launch_gemm_prefill(PRE_SCATTER, wmaps, *attn_map, g, st));
            }
            if ((rc = finish_and_wait(l, 0, buf, TL.res0, TL.res1, w.mlp_norm, TL.ss_mlp)) != SPD_OK) return rc;
        } else {      // SPD block: the sync-point is dropped, R_r = X + Y_r feeds the rank's MLP and Y_r is kept for a10
            for (int z = 0; z < nl; ++z) {
                PreGemmArgs g = base_args(z);
                const TcMap *wmaps[1] = {&lm.wo_shard};
                g.w_rows[0] = H; g.num_kb = cdiv(qd_r, 64);
                g.res_in = (const float *)(reg(z) + TL.res0); g.res_out = (float *)(reg(z) + TL.res1); g.gain = w.mlp_norm;
                g.hg = reg(z) + TL.hg; g.hg_stride = Mb * H; g.ss_out = (float *)(reg(z) + TL.ss_mlp);
                g.ysave = (float *)(reg(z) + TL.ysave);
                LAUNCH_S(K_OPROJ, g, launch_gemm_prefill(PRE_RESID, wmaps, *attn_map, g, st));
            }
            mlp_tiles = pre_ss_tiles(PRE_RESID, H);
        }
        for (int z = 0; z < nl; ++z) {   // a8 on the rank's MLP slice
            PreGemmArgs g = base_args(z);
            const TcMap *wmaps[2] = {&lm.w_gate, &lm.w_up};
            g.n_weights = 2; g.w_rows[0] = g.w_rows[1] = Fs;
            g.num_kb = cdiv(H, 64);
            g.ss_in = SumSq{(const float *)(reg(z) + TL.ss_mlp), mlp_tiles, 1, Mb, H, d.rms_eps};
            g.act = c->act; g.F = F; g.Fs = Fs; g.act_col0 = z * Fs;
            LAUNCH_S(K_GATE_UP, g, launch_gemm_prefill(PRE_GATEUP, wmaps, *hmap, g, st));
        }
        {   // a9 + a10, the kept sync-point.  TP block: out = R + sum_r Z_r;  SPD block: out = X + sum_r (Y_r + Z_r)
            MAP_OR_FAIL(act_shard, act_map(c, AB_ACT_SHARD, 128));
            const int buf = (int)((tp.exchanges + exchange++) & 1);
            for (int z = 0; z < nl; ++z) {
                PreGemmArgs g = base_args(z);
                const TcMap *wmaps[1] = {&lm.wd_shard};
                g.w_rows[0] = H; g.num_kb = cdiv(Fs, 64);
                scatter_args(g, z, l, 1, buf, sync ? nullptr : (const float *)(reg(z) + TL.ysave));
                LAUNCH_S(K_DOWN, g, launch_gemm_prefill(PRE_SCATTER, wmaps, *act_shard, g, st));
            }
            const void *gain = l + 1 < d.n_layers ? c->layers[l + 1].attn_norm : nullptr; // last block: the bf16 copy is the output
            if ((rc = finish_and_wait(l, 1, buf, sync ? TL.res1 : TL.res0, TL.res0, gain, TL.ss_attn)) != SPD_OK) return rc;
        }
    }
    // the last block's bf16 rows lie in every rank's operand plane: hand each local rank's copy to the caller
    for (int z = 0; z < nl; ++z)
        CU_TRY(cudaMemcpyAsync((char *)out + (long)z * out_stride, reg(z) + TL.hg, (size_t)M * H * 2, cudaMemcpyDeviceToDevice, st));
    c->launches_last = launches;
    return SPD_OK;
}

// Head-grouping measurements (Sec. 4.2.4) taken at one block while a prompt batch runs through the
// TP blocks before it: attention scores of every head and their pairwise distances (Eq. 2), and the
// sums of squares of MLP_m(norm(X + Y_i)) for every (device i, MLP partition m) (Eq. 3).
struct HeadProbe {
    int layer, n_seq, S;
    float *sigma;  // device [nq][n_seq][S][S]
    float *dist;   // device [nq][nq]
    double *norms; // host [T][T], sums of squares (the caller takes the root)
};

// One prefill chunk of the bf16 stack with the fused projections (same five kernels per block as
// a decode step, in their many-token form).
int run_prefill_fused(Ctx *c, const void *x, void *out, int M, TokMap tm, const int32_t *bt, int max_pages,
                      int max_context, cudaStream_t st, const HeadProbe *probe = nullptr)
{
    const spd_dims &d = c->d;
    const int H = d.hidden, qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim, F = d.ffn, Tn = d.T;
    const int Fs = F / Tn;
    const long Mc = c->Mcap;
    PageTable pt{bt, max_pages, c->n_pages, d.kv_block_size, d.n_kv_heads};
    int launches = 0;
    // block with bias (Sec. 4.1.2): LayerNorm folded into the QKV / fc1 tails, biases in the tails, ReLU, no rotary embedding
    const bool opt = d.block_kind == 1;
    const bool rope = d.rope_base > 0.f && !opt;
    const int nqkv = qd + 2 * kd;
    auto lnvec = [&](int l) { return c->lnvec + (size_t)l * 2 * (nqkv + F); }; // wg_qkv, wb_qkv, wg_fc1, wb_fc1
    if (rope) LAUNCH(K_ROPE_TABLE, launch_rope_table(c->rope, tm, M, d.head_dim, d.rope_base, st, next_stamp(c, K_ROPE_TABLE)));
    {
        PrologueArgs a{};
        a.x = x; a.res_out = c->res[0]; a.gain = c->layers[0].attn_norm; a.hg = c->h; a.ss_out = c->ss_attn;
        a.Mcap = Mc; a.M = M; a.H = H;
        if (opt) a.sum_out = c->sm_attn;
        LAUNCH_S(K_NORM, a, launch_prefill_prologue(a, st));
    }
    int attn_tiles = 1; // partial sums of squares per token in ss_attn
    // more than one 128-token tile: CTA pairs, 256 tokens per tile, weight maps with boxes of half a tile's rows
    const int pair = (M > 128 && c->prefill_pairs) ? 1 : 0;
    auto base_args = [&]() {
        PreGemmArgs g{};
        g.t_rows = M; g.err = c->err; g.H = H; g.Mcap = Mc; g.batches = 1; g.n_weights = 1; g.pair = pair;
        g.group_m = c->prefill_group_m;
        return g;
    };
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c->layers[l];
        const bool probing = probe && l == probe->layer;
        // while probing, the blocks before the probed one are TP blocks and the probed one is an SPD block
        const bool sync = probe ? !probing : c->mask[l] != 0;
        {   // a2 + a3
            PreGemmArgs g = base_args();
            const LayerMaps &lm = c->maps[l];
            const TcMap *wmaps[3] = {pair ? &lm.wq : &lm.wq256, pair ? &lm.wk : &lm.wk256, pair ? &lm.wv : &lm.wv256};
            MAP_OR_FAIL(am, act_map(c, AB_H, 128));
            g.n_weights = 3; g.w_rows[0] = qd; g.w_rows[1] = g.w_rows[2] = kd;
            g.num_kb = cdiv(H, 64);
            g.ss_in = SumSq{c->ss_attn, attn_tiles, 1, Mc, H, d.rms_eps, opt ? c->sm_attn : nullptr};
            if (opt) { g.ln_wg = lnvec(l); g.ln_wb = lnvec(l) + nqkv; }
            g.rope = rope ? c->rope : nullptr; g.q_out = c->q; g.k_pages = w.k_pages; g.v_pages = w.v_pages; g.pt = pt; g.tm = tm;
            g.n_q_heads = d.n_q_heads; g.head_dim = d.head_dim;
            LAUNCH_S(K_QKV, g, launch_gemm_prefill(PRE_QKV, wmaps, *am, g, st));
        }
        if (probing) {   // Eq. 2: attention score of every head as one long vector, pairwise Euclidean distances
            CU_TRY(launch_head_scores<bf16>(c->q, w.k_pages, pt, tm.b0, probe->S, probe->n_seq, d.n_q_heads, d.head_dim, probe->sigma,
                                            c->err, st));
            CU_TRY(launch_head_distance(probe->sigma, (long)probe->n_seq * probe->S * probe->S, d.n_q_heads, probe->dist, st));
        }
        {   // a4
            AttnArgs a{};
            a.q = c->q; a.k_pages = w.k_pages; a.v_pages = w.v_pages; a.pt = pt; a.tm = tm; a.out = c->attn;
            a.M = M; a.n_q_heads = d.n_q_heads; a.head_dim = d.head_dim; a.B = M; a.splits = 1;
            a.max_context = max_context; a.part_o = c->part_o; a.part_ml = c->part_ml; a.counters = c->attn_cnt; a.err = c->err;
            if (d.head_dim == 128 && d.kv_block_size == 16) {
                MAP_OR_FAIL(qm, act_map(c, AB_Q, 128));
                a.q_map = qm; a.k_map = &c->maps[l].kpages; a.v_map = &c->maps[l].vpages; a.rescale_log2 = (float)c->prefill_rescale_log2;
            }
            LAUNCH_S(K_ATTN, a, launch_prefill_attention<bf16>(a, st));
        }
        int mlp_tiles, mlp_groups;
        if (sync) {   // a5 - a7, sync block: sum_i Y_i is the K accumulation over all heads
            PreGemmArgs g = base_args();
            const TcMap *wmaps[1] = {pair ? &c->maps[l].wo_full : &c->maps[l].wo256};
            MAP_OR_FAIL(am, act_map(c, AB_ATTN, 128));
            g.w_rows[0] = H; g.num_kb = cdiv(qd, 64);
            g.res_in = c->res[0]; g.res_out = c->res[1]; g.gain = w.mlp_norm; g.hg = c->h; g.hg_stride = Mc * H; g.ss_out = c->ss_mlp;
            if (opt) { g.bias = w.bo; g.sum_out = c->sm_mlp; }
            LAUNCH_S(K_OPROJ, g, launch_gemm_prefill(PRE_RESID, wmaps, *am, g, st));
            mlp_tiles = pre_ss_tiles(PRE_RESID, H); mlp_groups = 1;
        } else {      // a5 - a7, SPD block: device i's K slice gives Y_i, kept apart
            PreGemmArgs g = base_args();
            const TcMap *wmaps[1] = {pair ? &c->maps[l].wo_shard64 : &c->maps[l].wo_shard};
            MAP_OR_FAIL(am, act_map(c, AB_ATTN_SHARD, 128));
            g.w_rows[0] = H; g.num_kb = cdiv(qd / Tn, 64); g.batches = Tn;
            g.res_in = c->res[0]; g.res_out = c->res[1]; g.gain = w.mlp_norm; g.hg = c->h; g.hg_stride = Mc * H; g.ss_out = c->ss_mlp;
            if (opt) { g.bias = w.bo; g.sum_out = c->sm_mlp; } // Y_i = P_i + b: b once in the carried sum, and in every device's MLP input
            LAUNCH_S(K_OPROJ, g, launch_gemm_prefill(PRE_OPROJ_SPD, wmaps, *am, g, st));
            mlp_tiles = pre_ss_tiles(PRE_OPROJ_SPD, H); mlp_groups = Tn;
        }
        if (probing) {
            // Eq. 3: for every rotation r, MLP partition (i + r) % T runs on device i's input X + Y_i; the
            // per-partition down projections only report the sums of squares of their outputs
            float *ssq = c->gu32; // [H tiles of 128][T][Mcap], idle in this path
            const int nt = pre_ss_tiles(PRE_OPROJ_SPD, H);
            std::vector<float> host((size_t)nt * Tn * M);
            for (int i = 0; i < Tn * Tn; ++i) probe->norms[i] = 0.0;
            for (int r = 0; r < Tn; ++r) {
                {
                    PreGemmArgs g = base_args();
                    const TcMap *wmaps[2] = {&c->maps[l].w_gate, &c->maps[l].w_up};
                    MAP_OR_FAIL(am, act_map(c, AB_H, 128));
                    g.n_weights = 2; g.w_rows[0] = g.w_rows[1] = Fs; g.batches = Tn; g.t_batched = 1; g.w_rot = r; g.pair = 0;
                    g.num_kb = cdiv(H, 64);
                    g.ss_in = SumSq{c->ss_mlp, mlp_tiles, mlp_groups, Mc, H, d.rms_eps};
                    g.rstd_per_shard = 1;
                    g.act = c->act; g.F = F; g.Fs = Fs;
                    LAUNCH(K_GATE_UP, launch_gemm_prefill(PRE_GATEUP, wmaps, *am, g, st));
                }
                {
                    PreGemmArgs g = base_args();
                    const TcMap *wmaps[1] = {&c->maps[l].wd_shard};
                    MAP_OR_FAIL(am, act_map(c, AB_ACT_SHARD, 128));
                    g.w_rows[0] = H; g.num_kb = cdiv(Fs, 64); g.batches = Tn; g.norm_only = 1; g.ss_out = ssq; g.pair = 0;
                    LAUNCH(K_DOWN, launch_gemm_prefill(PRE_OPROJ_SPD, wmaps, *am, g, st));
                }
                CU_TRY(cudaMemcpy2DAsync(host.data(), (size_t)M * 4, ssq, (size_t)Mc * 4, (size_t)M * 4, (size_t)nt * Tn,
                                         cudaMemcpyDeviceToHost, st));
                CU_TRY(cudaStreamSynchronize(st));
                for (int t = 0; t < nt; ++t)
                    for (int wz = 0; wz < Tn; ++wz) {
                        double acc = 0.0;
                        const float *row = host.data() + ((size_t)t * Tn + wz) * M;
                        for (int m = 0; m < M; ++m) acc += (double)row[m];
                        probe->norms[(size_t)((wz - r + Tn) % Tn) * Tn + wz] += acc; // device (wz - r), partition wz
                    }
            }
            c->launches_last = launches;
            return SPD_OK;
        }
        {   // a8
            PreGemmArgs g = base_args();
            const TcMap *wmaps[2] = {&c->maps[l].w_gate, &c->maps[l].w_up};
            MAP_OR_FAIL(am, act_map(c, AB_H, 128));
            g.n_weights = 2; g.w_rows[0] = g.w_rows[1] = Fs; g.batches = Tn; g.t_batched = sync ? 0 : 1;
            g.num_kb = cdiv(H, 64);
            g.ss_in = SumSq{c->ss_mlp, mlp_tiles, mlp_groups, Mc, H, d.rms_eps, opt ? c->sm_mlp : nullptr};
            g.rstd_per_shard = sync ? 0 : 1;
            g.act = c->act; g.F = F; g.Fs = Fs;
            if (opt) { g.n_weights = 1; g.fc1_only = 1; g.ln_wg = lnvec(l) + 2 * nqkv; g.ln_wb = lnvec(l) + 2 * nqkv + F; } // fc1 alone: bias, ReLU
            LAUNCH_S(K_GATE_UP, g, launch_gemm_prefill(PRE_GATEUP, wmaps, *am, g, st));
        }
        {   // a9 + a10: res[1] holds X + sum_i Y_i in both modes, so out = res[1] + sum_i Z_i
            PreGemmArgs g = base_args();
            const TcMap *wmaps[1] = {pair ? &c->maps[l].w_down : &c->maps[l].wd256};
            MAP_OR_FAIL(am, act_map(c, AB_ACT, 128));
            g.w_rows[0] = H; g.num_kb = cdiv(F, 64);
            g.res_in = c->res[1]; g.res_out = c->res[0];
            if (l + 1 < d.n_layers) { g.gain = c->layers[l + 1].attn_norm; g.hg = c->h; g.hg_stride = Mc * H; g.ss_out = c->ss_attn; }
            else g.final_out = out;
            if (opt) { g.bias = w.b_fc2; if (l + 1 < d.n_layers) g.sum_out = c->sm_attn; }
            LAUNCH_S(K_DOWN, g, launch_gemm_prefill(PRE_RESID, wmaps, *am, g, st));
            attn_tiles = pre_ss_tiles(PRE_RESID, H);
        }
    }
    c->launches_last = launches;
    return SPD_OK;
}

int read_err_flag(Ctx *c, cudaStream_t st, int *flag)
{
    CU_TRY(cudaMemcpyAsync(flag, c->err, sizeof(int), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    if (*flag) {
        // a kernel that gave up may have left arrival counters mid-count
        CU_TRY(cudaMemsetAsync(c->err, 0, sizeof(int), st));
        CU_TRY(cudaMemsetAsync(c->attn_cnt, 0, (size_t)c->d.max_batch * c->d.n_q_heads * 4, st));
    }
    return SPD_OK;
}

int build_weight_maps(Ctx &c)
{
    const spd_dims &d = c.d;
    const long H = d.hidden, qd = (long)d.n_q_heads * d.head_dim, kd = (long)d.n_kv_heads * d.head_dim, F = d.ffn, T = d.T;
    c.maps.resize(d.n_layers);
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c.layers[l];
        LayerMaps &m = c.maps[l];
        int rc = 0;
        rc |= make_operand_map(&m.wq, w.wq, H, qd, 1, H, 0, 128);
        rc |= make_operand_map(&m.wk, w.wk, H, kd, 1, H, 0, 128);
        rc |= make_operand_map(&m.wv, w.wv, H, kd, 1, H, 0, 128);
        rc |= make_operand_map(&m.wo_full, w.wo, qd, H, 1, qd, 0, 128);
        rc |= make_operand_map(&m.wo_shard, w.wo, qd / T, H, T, qd, qd / T, 128);
        rc |= make_operand_map(&m.wo_shard64, w.wo, qd / T, H, T, qd, qd / T, 64);
        rc |= make_operand_map(&m.w_gate, w.w_gate, H, F / T, T, H, (F / T) * H, 128);
        if (d.block_kind == 0) rc |= make_operand_map(&m.w_up, w.w_up, H, F / T, T, H, (F / T) * H, 128);
        rc |= make_operand_map(&m.w_down, w.w_down, F, H, 1, F, 0, 128);
        rc |= make_operand_map(&m.wq256, w.wq, H, qd, 1, H, 0, 256);
        rc |= make_operand_map(&m.wk256, w.wk, H, kd, 1, H, 0, 256);
        rc |= make_operand_map(&m.wv256, w.wv, H, kd, 1, H, 0, 256);
        rc |= make_operand_map(&m.wo256, w.wo, qd, H, 1, qd, 0, 256);
        rc |= make_operand_map(&m.wd256, w.w_down, F, H, 1, F, 0, 256);
        rc |= make_operand_map(&m.wd_shard, w.w_down, F / T, H, T, F, F / T, 128);
        if (d.head_dim == 128 && d.kv_block_size == 16) {
            // K / V pages as [n_pages * n_kv_heads * 16 token rows][head_dim]; one box = 64 dims of a page's 16 tokens
            const long rows = (long)c.n_pages * d.n_kv_heads * 16;
            rc |= make_operand_map(&m.kpages, w.k_pages, 128, rows, 1, 128, 0, 16);
            rc |= make_operand_map(&m.vpages, w.v_pages, 128, rows, 1, 128, 0, 16);
            rc |= make_page_map(&m.kpage_whole, w.k_pages, rows); // decode attention: one copy per (page, head)
            rc |= make_page_map(&m.vpage_whole, w.v_pages, rows);
        }
        rc |= make_operand_map(&m.w_gate64, w.w_gate, H, F / T, T, H, (F / T) * H, 64);
        if (d.block_kind == 0) rc |= make_operand_map(&m.w_up64, w.w_up, H, F / T, T, H, (F / T) * H, 64);
        if (rc) return SPD_EINVAL;
    }
    return SPD_OK;
}

// Captured decode steps.  A graph is valid for exactly one GraphKey; up to 8 are kept per context.
GraphEntry *find_graph(Ctx &c, const GraphKey &key)
{
    for (GraphEntry &e : c.graphs)
        if (e.key == key) return &e;
    return nullptr;
}

// Whether a call on `st` may use graphs at all: not while profiling, not inside somebody else's capture, not on
// the legacy default stream (which cannot be captured).
int graphs_usable(Ctx &c, cudaStream_t st, bool *ok)
{
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CU_TRY(cudaStreamIsCapturing(st, &cap));
    *ok = c.use_graphs && !c.profiling && cap == cudaStreamCaptureStatusNone && st != 0 && st != cudaStreamLegacy;
    return SPD_OK;
}

// Captures run() on `st` (nothing executes) and keeps the instantiated graph under `key`.
template <typename Run>
int capture_graph(Ctx &c, const GraphKey &key, Run run, cudaStream_t st, GraphEntry **out)
{
    CU_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    const int rc = run();
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(st, &graph);
    if (rc != SPD_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; return SPD_ECUDA; }
    cudaGraphExec_t exec = nullptr;
    e = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; return SPD_ECUDA; }
    if (c.graphs.size() >= 8) { // evict the least recently used
        size_t lru = 0;
        for (size_t i = 1; i < c.graphs.size(); ++i)
            if (c.graphs[i].last_use < c.graphs[lru].last_use) lru = i;
        cudaGraphExecDestroy(c.graphs[lru].exec);
        c.graphs.erase(c.graphs.begin() + lru);
    }
    c.graphs.push_back(GraphEntry{key, exec, ++c.graph_clock, c.launches_last, c.tl_kind});
    *out = &c.graphs.back();
    return SPD_OK;
}

// Runs a decode step from its captured graph, capturing it first when no graph matches `key`;
// directly when graphs cannot be used.
template <typename Run>
int replay_or_run(Ctx &c, const GraphKey &key, Run run, cudaStream_t st)
{
    bool usable = false;
    int rc = graphs_usable(c, st, &usable);
    if (rc != SPD_OK) return rc;
    if (!usable) return run();
    GraphEntry *hit = find_graph(c, key);
    if (!hit && (rc = capture_graph(c, key, run, st, &hit)) != SPD_OK) return rc;
    hit->last_use = ++c.graph_clock;
    c.launches_last = hit->launches;
    if (c.timeline) { c.tl_kind = hit->tl_kind; c.tl_next = (int)hit->tl_kind.size(); } // the replay stamps the slots of its capture
    CU_TRY(cudaGraphLaunch(hit->exec, st));
    return SPD_OK;
}

// The step's launch shape changes with the context bucket.  So that a growing context does not meet a capture at
// the very step that crosses into the next bucket, that bucket's graph is captured (not run) once the context is
// within GRAPH_AHEAD_STEPS of the edge - while the device is still busy with the steps already queued.
constexpr int GRAPH_AHEAD_STEPS = 32;
template <typename Run>
int capture_ahead(Ctx &c, const GraphKey &key, Run run, cudaStream_t st)
{
    bool usable = false;
    int rc = graphs_usable(c, st, &usable);
    if (rc != SPD_OK || !usable || find_graph(c, key)) return rc;
    const int launches = c.launches_last;
    const std::vector<int> kinds = c.tl_kind;
    const int next = c.tl_next;
    GraphEntry *e = nullptr;
    rc = capture_graph(c, key, run, st, &e);
    c.launches_last = launches; // bookkeeping stays that of the step that ran
    c.tl_kind = kinds;
    c.tl_next = next;
    return rc;
}

} // namespace

struct spd_ctx { Ctx c; };

extern "C" {

int spd_workspace_bytes(const spd_dims *dims, const uint8_t *sync_mask, size_t *out_bytes)
{
    if (!out_bytes) return SPD_ENULL;
    int rc = check_dims(dims, sync_mask);
    if (rc) return rc;
    bool any_spd = false;
    for (int l = 0; l < dims->n_layers; ++l) any_spd |= sync_mask[l] == 0;
    *out_bytes = make_layout(*dims, any_spd).total;
    return SPD_OK;
}

int spd_create(const spd_dims *dims, const uint8_t *sync_mask, const spd_layer *layers, int32_t n_pages,
               void *workspace, size_t workspace_bytes, spd_ctx **out)
{
    if (!out || !layers || !workspace) return SPD_ENULL;
    int rc = check_dims(dims, sync_mask);
    if (rc) return rc;
    if (n_pages < 1) return SPD_EINVAL;
    for (int l = 0; l < dims->n_layers; ++l) {
        const spd_layer &w = layers[l];
        if (!w.attn_norm || !w.wq || !w.wk || !w.wv || !w.wo || !w.mlp_norm || !w.w_gate || !w.w_down || !w.k_pages || !w.v_pages)
            return SPD_ENULL;
        if (dims->block_kind == 0 && !w.w_up) return SPD_ENULL;
        if (dims->block_kind == 1 && (!w.attn_norm_b || !w.bq || !w.bk || !w.bv || !w.bo || !w.mlp_norm_b || !w.b_fc1 || !w.b_fc2))
            return SPD_ENULL;
    }
    int dev = 0;
    cudaDeviceProp prop;
    CU_TRY(cudaGetDevice(&dev));
    CU_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return SPD_EINVAL;
    bool any_spd = false;
    for (int l = 0; l < dims->n_layers; ++l) any_spd |= sync_mask[l] == 0;
    Layout L = make_layout(*dims, any_spd);
    if (workspace_bytes < L.total || ((uintptr_t)workspace & 255)) return SPD_EWORKSPACE;
    spd_ctx *h = new (std::nothrow) spd_ctx();
    if (!h) return SPD_EINVAL;
    Ctx &c = h->c;
    c.d = *dims;
    c.mask.assign(sync_mask, sync_mask + dims->n_layers);
    c.layers.assign(layers, layers + dims->n_layers);
    c.n_pages = n_pages;
    c.any_spd = any_spd;
    c.Mcap = (long)L.Mcap;
    // regions are laid out from a 1024-byte aligned base inside the caller's buffer
    c.ws = (char *)workspace;
    c.ws_bytes = workspace_bytes;
    c.err = (int *)(c.ws + L.err);
    c.res[0] = (float *)(c.ws + L.res[0]);
    c.res[1] = (float *)(c.ws + L.res[1]);
    c.h = c.ws + L.h; c.q = c.ws + L.q; c.attn = c.ws + L.attn; c.act = c.ws + L.act;
    c.rope = (float2 *)(c.ws + L.rope);
    c.qkv32 = (float *)(c.ws + L.qkv32); c.proj32 = (float *)(c.ws + L.proj32); c.gu32 = (float *)(c.ws + L.gu32);
    c.part_o = (float *)(c.ws + L.part_o); c.part_ml = (float *)(c.ws + L.part_ml);
    c.attn_cnt = (int *)(c.ws + L.attn_cnt);
    c.ss_attn = (float *)(c.ws + L.ss_attn); c.ss_mlp = (float *)(c.ws + L.ss_mlp);
    c.sm_attn = (float *)(c.ws + L.sm_attn); c.sm_mlp = (float *)(c.ws + L.sm_mlp); c.lnvec = (float *)(c.ws + L.lnvec);
    c.bias_fused = 1;
    c.stamps = (unsigned long long *)(c.ws + L.stamps);
    c.stamps_cap = stamp_slots(*dims);
    c.timeline = false;
    c.tl_next = 0;
    for (int i = 0; i < SITE_COUNT; ++i) c.split_override[i] = 0;
    c.l2_prefetch_kb = 0;
    c.prefill_rescale_log2 = 8;
    c.peer_wait_ms = 1000;
    c.prefill_pairs = 1;
    c.prefill_group_m = 0;
    c.ring_stages = 0;
    c.oproj_planes = 0;
    c.launches_last = 0;
    c.tp.on = false;
    c.use_graphs = true;
    c.graph_clock = 0;
    c.profiling = false;
    c.ev_used = 0;
    memset(c.act_map_ready, 0, sizeof(c.act_map_ready));

    if (dims->dtype == 1) {
        rc = build_weight_maps(c);
        if (rc) { delete h; return rc; }
    }
    // Zero the workspace once: the error flag, the arrival counters of the attention merge, and token rows
    // beyond a launch's M that tiled loads read (never use).  A memset of device memory returns before it
    // has run and is ordered only with the legacy default stream, while the caller's allocator and every
    // later call work on other (possibly non-blocking) streams: wait for the device on both sides, so that
    // neither an earlier user of this memory nor a first kernel can overlap the zeroing.
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemset(workspace, 0, L.total);
    if (dims->block_kind == 1 && dims->dtype == 1) {
        // block with bias: fold each LayerNorm into the projection that follows it (see SumSq)
        const int H = dims->hidden, qd = dims->n_q_heads * dims->head_dim, kd = dims->n_kv_heads * dims->head_dim, F = dims->ffn;
        const size_t per_layer = 2 * (size_t)(qd + 2 * kd + F);
        for (int l = 0; l < dims->n_layers && e == cudaSuccess; ++l) {
            const spd_layer &w = c.layers[l];
            float *wg = c.lnvec + l * per_layer, *wb = wg + (qd + 2 * kd), *fg = wb + (qd + 2 * kd), *fb = fg + F;
            e = launch_ln_fold(w.wq, qd, H, w.attn_norm, w.attn_norm_b, w.bq, wg, wb, 0);
            if (e == cudaSuccess) e = launch_ln_fold(w.wk, kd, H, w.attn_norm, w.attn_norm_b, w.bk, wg + qd, wb + qd, 0);
            if (e == cudaSuccess) e = launch_ln_fold(w.wv, kd, H, w.attn_norm, w.attn_norm_b, w.bv, wg + qd + kd, wb + qd + kd, 0);
            if (e == cudaSuccess) e = launch_ln_fold(w.w_gate, F, H, w.mlp_norm, w.mlp_norm_b, w.b_fc1, fg, fb, 0);
        }
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; delete h; return SPD_ECUDA; }
    *out = h;
    return SPD_OK;
}

int spd_prefill(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table, int32_t max_pages,
                void *out, void *stream)
{
    if (!ctx || !x || !block_table || !out) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    if (B < 1 || S < 1 || B > d.max_batch || x == out) return SPD_EINVAL;
    if (S > d.max_seq_len || (long)max_pages * d.kv_block_size < S) return SPD_ECAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = esize(d);
    const int Mp = d.max_prefill_tokens;
    int total_launches = 0;
    CU_TRY(timeline_restart(&c, st));
    auto run = [&](int b0, int nb, int s0, int ns) -> int {
        TokMap tm{0, b0, ns, s0, nullptr};
        size_t off = ((size_t)b0 * S + s0) * d.hidden * es;
        const bool fused = d.dtype == 1 && d.hidden % 16 == 0 && (d.block_kind == 0 || c.bias_fused);
        int rc = d.dtype == 0 ? run_tokens<float>(&c, (const char *)x + off, (char *)out + off, nb * ns, tm, block_table, max_pages, false, S, st)
                 : fused      ? run_prefill_fused(&c, (const char *)x + off, (char *)out + off, nb * ns, tm, block_table, max_pages, S, st)
                              : run_tokens<bf16>(&c, (const char *)x + off, (char *)out + off, nb * ns, tm, block_table, max_pages, false, S, st);
        total_launches += c.launches_last;
        return rc;
    };
    if (S <= Mp) {
        int nb = Mp / S;
        for (int b0 = 0; b0 < B; b0 += nb) {
            int rc = run(b0, (B - b0 < nb) ? B - b0 : nb, 0, S);
            if (rc) return rc;
        }
    } else {
        for (int b = 0; b < B; ++b)
            for (int s0 = 0; s0 < S; s0 += Mp) {
                int rc = run(b, 1, s0, (S - s0 < Mp) ? S - s0 : Mp);
                if (rc) return rc;
            }
    }
    c.launches_last = total_launches;
    CU_TRY(timeline_fold(&c, st));
    return SPD_OK;
}

int spd_decode_step(spd_ctx *ctx, const void *x, int32_t B, const int32_t *seq_lens, const int32_t *block_table,
                    int32_t max_pages, int32_t max_context, void *out, void *stream)
{
    if (!ctx || !x || !seq_lens || !block_table || !out) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    if (B < 1 || B > d.max_batch || x == out || max_context < 1) return SPD_EINVAL;
    if (max_context > d.max_seq_len || (long)max_pages * d.kv_block_size < max_context) return SPD_ECAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    TokMap tm{1, 0, 1, 0, seq_lens};
    // The launch sequence only depends on a coarse bucket of the context bound (it sizes the
    // KV split), so a step can be replayed from a captured graph until a pointer or the
    // bucket changes.
    auto bucket_of = [&](int mc) {
        int b = (mc + 255) / 256 * 256;
        if (b > d.max_seq_len) b = d.max_seq_len;
        if ((long)b > (long)max_pages * d.kv_block_size) b = max_pages * d.kv_block_size;
        return b;
    };
    const int ctx_bucket = bucket_of(max_context);
    auto run_at = [&](int bucket) {
        return [&, bucket]() -> int {
            CU_TRY(timeline_restart(&c, st));
            const int rc = d.dtype == 0        ? run_tokens<float>(&c, x, out, B, tm, block_table, max_pages, true, bucket, st)
                           : (d.block_kind == 0 || c.bias_fused) ? run_decode_fused(&c, x, out, B, tm, block_table, max_pages, bucket, st)
                                               : run_tokens<bf16>(&c, x, out, B, tm, block_table, max_pages, true, bucket, st);
            if (rc != SPD_OK) return rc;
            CU_TRY(timeline_fold(&c, st)); // part of the captured step: every replay folds its own stamps
            return SPD_OK;
        };
    };
    const GraphKey key{x, seq_lens, block_table, out, B, max_pages, ctx_bucket, 0};
    int rc = replay_or_run(c, key, run_at(ctx_bucket), st);
    if (rc != SPD_OK) return rc;
    const int next_bucket = bucket_of(ctx_bucket + 1);
    if (next_bucket > ctx_bucket && max_context + GRAPH_AHEAD_STEPS > ctx_bucket) {
        const GraphKey ahead{x, seq_lens, block_table, out, B, max_pages, next_bucket, 0};
        rc = capture_ahead(c, ahead, run_at(next_bucket), st);
    }
    return rc;
}

static void drop_graphs(Ctx &c)
{
    for (GraphEntry &g : c.graphs) cudaGraphExecDestroy(g.exec);
    c.graphs.clear();
}

int spd_set_mask(spd_ctx *ctx, const uint8_t *sync_mask)
{
    if (!ctx || !sync_mask) return SPD_ENULL;
    Ctx &c = ctx->c;
    bool any_spd = false;
    for (int l = 0; l < c.d.n_layers; ++l) any_spd |= sync_mask[l] == 0;
    if (any_spd && !c.any_spd) return SPD_EWORKSPACE;
    c.mask.assign(sync_mask, sync_mask + c.d.n_layers);
    drop_graphs(c);
    return SPD_OK;
}

int spd_sensitivity_scan(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table, int32_t max_pages,
                         void *ref_out, void *tmp_out, double *sensitivity, double *metric, void *stream)
{
    if (!ctx || !ref_out || !tmp_out || !sensitivity) return SPD_ENULL;
    Ctx &c = ctx->c;
    const int L = c.d.n_layers;
    if (!c.any_spd) return SPD_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const std::vector<uint8_t> saved = c.mask;
    std::vector<uint8_t> m(L, 1);
    std::vector<double> met(L + 1, 0.0);
    constexpr int NB = 1024;
    std::vector<float> part(NB);
    float *dpart = c.part_o; // attention split scratch: at least NB floats, idle between the passes
    const long n = (long)B * S * c.d.hidden;
    auto restore = [&](int rc) { c.mask = saved; drop_graphs(c); return rc; };
    if ((size_t)c.d.max_batch * c.d.n_q_heads * 32 * c.d.head_dim < (size_t)NB) return SPD_EWORKSPACE;
    drop_graphs(c);
    c.mask = m; // all TP
    int rc = spd_prefill(ctx, x, B, S, block_table, max_pages, ref_out, stream);
    if (rc) return restore(rc);
    for (int i = L - 1; i >= 0; --i) {
        m[i] = 0; // blocks i .. L-1 are SPD blocks now
        c.mask = m;
        rc = spd_prefill(ctx, x, B, S, block_table, max_pages, tmp_out, stream);
        if (rc) return restore(rc);
        cudaError_t e = launch_sq_diff(tmp_out, ref_out, n, c.d.dtype == 1, dpart, NB, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(part.data(), dpart, NB * sizeof(float), cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return restore(SPD_ECUDA); }
        double tot = 0.0;
        for (int b = 0; b < NB; ++b) tot += (double)part[b];
        met[i] = tot / (double)n;
    }
    for (int i = 0; i < L; ++i) sensitivity[i] = met[i] - met[i + 1];
    if (metric) for (int i = 0; i <= L; ++i) metric[i] = met[i];
    return restore(SPD_OK);
}

int spd_head_grouping_stats(spd_ctx *ctx, int32_t layer, const void *x, int32_t B, int32_t S, const int32_t *block_table,
                            int32_t max_pages, float *sigma_scratch, float *dist_dev, float *dist, double *norms, void *stream)
{
    if (!ctx || !x || !block_table || !sigma_scratch || !dist_dev || !dist || !norms) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    if (d.dtype != 1 || d.block_kind != 0 || d.hidden % 16 || layer < 0 || layer >= d.n_layers || B < 1 || S < 1 || B > d.max_batch) return SPD_EINVAL;
    if ((long)B * S > d.max_prefill_tokens) return SPD_EINVAL; // one chunk
    if (S > d.max_seq_len || (long)max_pages * d.kv_block_size < S) return SPD_ECAPACITY;
    if (!c.any_spd) return SPD_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    HeadProbe probe{layer, B, S, sigma_scratch, dist_dev, norms};
    TokMap tm{0, 0, S, 0, nullptr};
    int rc = run_prefill_fused(&c, x, nullptr, B * S, tm, block_table, max_pages, S, st, &probe);
    if (rc) return rc;
    CU_TRY(cudaMemcpyAsync(dist, dist_dev, (size_t)d.n_q_heads * d.n_q_heads * sizeof(float), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    for (int i = 0; i < d.T * d.T; ++i) norms[i] = sqrt(norms[i]);
    return SPD_OK;
}

int spd_set_graphs(spd_ctx *ctx, int32_t enabled)
{
    if (!ctx) return SPD_ENULL;
    ctx->c.use_graphs = enabled != 0;
    return SPD_OK;
}

int spd_set_tuning(spd_ctx *ctx, const char *key, int32_t value)
{
    if (!ctx || !key) return SPD_ENULL;
    if (value < 0) return SPD_EINVAL;
    Ctx &c = ctx->c;
    static const char *const site_keys[SITE_COUNT] = {"qkv_splits", "o_proj_splits", "gate_up_splits", "down_splits", "attention_splits"};
    bool found = false;
    for (int i = 0; i < SITE_COUNT; ++i)
        if (!strcmp(key, site_keys[i])) { c.split_override[i] = value; found = true; }
    if (!strcmp(key, "o_proj_planes")) { c.oproj_planes = value > 2 ? 0 : value; found = true; }
    if (!strcmp(key, "decode_ring_stages")) { c.ring_stages = (value == 0 || (value >= 3 && value <= 5)) ? value : 0; found = true; }
    if (!strcmp(key, "prefill_rescale_log2")) { c.prefill_rescale_log2 = value > 16 ? 16 : value; found = true; }
    if (!strcmp(key, "l2_prefetch_blocks")) { c.l2_prefetch_kb = value > 64 ? 64 : value; found = true; }
    if (!strcmp(key, "prefill_group_m")) { c.prefill_group_m = value > 4096 ? 4096 : value; found = true; }
    if (!strcmp(key, "bias_fused")) { c.bias_fused = value != 0; found = true; }
    if (!strcmp(key, "prefill_pairs")) { c.prefill_pairs = value != 0; found = true; }
    if (!strcmp(key, "peer_wait_ms")) { c.peer_wait_ms = value < 1 ? 1000 : (value > 60000 ? 60000 : value); found = true; }
    if (!found) return SPD_EINVAL;
    for (GraphEntry &g : c.graphs) cudaGraphExecDestroy(g.exec); // captured steps used the old setting
    c.graphs.clear();
    return SPD_OK;
}

int spd_tp_region_bytes(const spd_ctx *ctx, int32_t T, size_t *out_bytes)
{
    if (!ctx || !out_bytes) return SPD_ENULL;
    if (T < 1 || T > TP_MAX_RANKS) return SPD_EINVAL;
    *out_bytes = tp_layout(ctx->c.d, T).total;
    return SPD_OK;
}

int spd_tp_attach(spd_ctx *ctx, int32_t T, int32_t rank_base, void *const *regions, size_t region_bytes, void *stream)
{
    if (!ctx || !regions) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    const int nl = d.T;
    if (T < 1 || T > TP_MAX_RANKS || rank_base < 0 || rank_base + nl > T) return SPD_EINVAL;
    if (!(nl == 1 || (nl == T && rank_base == 0))) return SPD_EINVAL;
    if (d.dtype != 1 || d.block_kind != 0 || d.hidden % 16 != 0 || 128 % d.head_dim != 0) return SPD_EINVAL;
    if ((d.n_q_heads / nl) * d.head_dim % 8 != 0) return SPD_EINVAL;
    const TpLayout TL = tp_layout(d, T);
    if (region_bytes < TL.total) return SPD_EWORKSPACE;
    for (int j = 0; j < T; ++j) {
        if (!regions[j]) return SPD_ENULL;
        if ((uintptr_t)regions[j] & 1023) return SPD_EWORKSPACE;
    }
    const long z_stride = nl > 1 ? (long)((char *)regions[rank_base + 1] - (char *)regions[rank_base]) : 0;
    for (int z = 1; z < nl; ++z)
        if ((char *)regions[rank_base + z] - (char *)regions[rank_base] != z * z_stride) return SPD_EINVAL;
    if (nl > 1 && (z_stride < (long)TL.total || (z_stride & 1023))) return SPD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    TpState &tp = c.tp;
    tp.on = false;
    tp.T = T; tp.rank_base = rank_base; tp.z_stride = z_stride; tp.L = TL; tp.exchanges = 0;
    for (int j = 0; j < T; ++j) tp.regions[j] = (char *)regions[j];
    const long H = d.hidden, qd = (long)d.n_q_heads * d.head_dim, kd = (long)d.n_kv_heads * d.head_dim;
    tp.qkv_maps.resize((size_t)3 * d.n_layers);
    int rc = 0;
    for (int l = 0; l < d.n_layers; ++l) {
        const spd_layer &w = c.layers[l];
        rc |= make_operand_map(&tp.qkv_maps[3 * l], w.wq, H, qd / nl, nl, H, (qd / nl) * H, 128);
        rc |= make_operand_map(&tp.qkv_maps[3 * l + 1], w.wk, H, kd / nl, nl, H, (kd / nl) * H, 128);
        rc |= make_operand_map(&tp.qkv_maps[3 * l + 2], w.wv, H, kd / nl, nl, H, (kd / nl) * H, 128);
    }
    const int boxes[4] = {16, 32, 64, 128};
    for (int i = 0; i < 4; ++i)
        rc |= make_operand_map(&tp.h_maps[i], tp.regions[rank_base] + TL.hg, H, TL.Mb, nl, H, nl > 1 ? z_stride / 2 : TL.Mb * H, boxes[i]);
    if (rc) return SPD_EINVAL;
    // the local ranks' regions start from zero: step 0, no flag set, token rows beyond a batch read as zero
    for (int z = 0; z < nl; ++z) CU_TRY(cudaMemsetAsync(tp.regions[rank_base + z], 0, TL.total, st));
    drop_graphs(c);
    tp.on = true;
    return SPD_OK;
}

int spd_tp_detach(spd_ctx *ctx)
{
    if (!ctx) return SPD_ENULL;
    ctx->c.tp.on = false;
    return SPD_OK;
}

int spd_tp_prefill(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table, int32_t max_pages,
                   void *out, void *stream)
{
    if (!ctx || !x || !block_table || !out) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    if (!c.tp.on) return SPD_EINVAL;
    if (B < 1 || S < 1 || B > d.max_batch || x == out) return SPD_EINVAL;
    if (S > d.max_seq_len || (long)max_pages * d.kv_block_size < S) return SPD_ECAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    // tokens per launch: the capacity of the ranks' planes and of the shared activation buffers
    long chunk = c.tp.L.Mb < c.Mcap ? c.tp.L.Mb : c.Mcap;
    if (chunk > d.max_prefill_tokens) chunk = d.max_prefill_tokens;
    CU_TRY(timeline_restart(&c, st));
    const long rank_stride = (long)B * S * d.hidden * 2;
    int total_launches = 0;
    auto run = [&](int b0, int nb, int s0, int ns) -> int {
        TokMap tm{0, b0, ns, s0, nullptr};
        const size_t off = ((size_t)b0 * S + s0) * d.hidden * 2;
        const int rc = run_tp_prefill(&c, (const char *)x + off, (char *)out + off, rank_stride, nb * ns, tm, block_table, max_pages, S, st);
        if (rc == SPD_OK) {
            for (int l = 0; l < d.n_layers; ++l) c.tp.exchanges += c.mask[l] ? 2 : 1;
            total_launches += c.launches_last;
        }
        return rc;
    };
    if (S <= chunk) {
        const int nb = (int)(chunk / S);
        for (int b0 = 0; b0 < B; b0 += nb) {
            const int rc = run(b0, B - b0 < nb ? B - b0 : nb, 0, S);
            if (rc) return rc;
        }
    } else {
        for (int b = 0; b < B; ++b)
            for (int s0 = 0; s0 < S; s0 += (int)chunk) {
                const int rc = run(b, 1, s0, S - s0 < chunk ? S - s0 : (int)chunk);
                if (rc) return rc;
            }
    }
    c.launches_last = total_launches;
    CU_TRY(timeline_fold(&c, st));
    return SPD_OK;
}

int spd_tp_decode_step(spd_ctx *ctx, const void *x, int32_t B, const int32_t *seq_lens, const int32_t *block_table,
                       int32_t max_pages, int32_t max_context, void *out, void *stream)
{
    if (!ctx || !x || !seq_lens || !block_table || !out) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    if (!c.tp.on) return SPD_EINVAL;
    if (B < 1 || B > d.max_batch || x == out || max_context < 1) return SPD_EINVAL;
    if (max_context > d.max_seq_len || (long)max_pages * d.kv_block_size < max_context) return SPD_ECAPACITY;
    TokMap tm{1, 0, 1, 0, seq_lens};
    int ctx_bucket = (max_context + 255) / 256 * 256;
    if (ctx_bucket > d.max_seq_len) ctx_bucket = d.max_seq_len;
    if ((long)ctx_bucket > (long)max_pages * d.kv_block_size) ctx_bucket = max_pages * d.kv_block_size;
    cudaStream_t st = (cudaStream_t)stream;
    // A captured step is valid for one receive-buffer phase: consecutive exchanges alternate between the
    // two buffers, so a stack with an odd number of exchanges per step needs one graph per phase.
    const GraphKey key{x, seq_lens, block_table, out, B, max_pages, ctx_bucket, 1 + (int)(c.tp.exchanges & 1)};
    const int rc = replay_or_run(c, key, [&]() {
        CU_TRY(timeline_restart(&c, st));
        const int rc2 = run_tp(&c, x, out, (long)B * d.hidden * 2, B, tm, block_table, max_pages, ctx_bucket, st);
        if (rc2 != SPD_OK) return rc2;
        CU_TRY(timeline_fold(&c, st));
        return SPD_OK;
    }, st);
    if (rc != SPD_OK) return rc;
    for (int l = 0; l < d.n_layers; ++l) c.tp.exchanges += c.mask[l] ? 2 : 1; // the same on every rank of the group
    return SPD_OK;
}

int spd_tp_baseline_decode_step(spd_ctx *ctx, const void *x, int32_t B, const int32_t *seq_lens, const int32_t *block_table,
                                int32_t max_pages, int32_t max_context, void *out, float *scratch, size_t scratch_floats,
                                spd_allreduce_fn fn, void *user, void *stream)
{
    if (!ctx || !x || !seq_lens || !block_table || !out || !scratch || !fn) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    if (d.T != 1 || d.dtype != 1 || d.block_kind != 0 || d.hidden % 16) return SPD_EINVAL; // one shard's stack, bf16, no bias
    if (B < 1 || B > d.max_batch || x == out || max_context < 1) return SPD_EINVAL;
    if (max_context > d.max_seq_len || (long)max_pages * d.kv_block_size < max_context) return SPD_ECAPACITY;
    if (scratch_floats < (size_t)2 * B * d.hidden) return SPD_EWORKSPACE;
    TokMap tm{1, 0, 1, 0, seq_lens};
    return run_tp_baseline(&c, x, out, B, tm, block_table, max_pages, true, max_context, scratch, fn, user, (cudaStream_t)stream);
}

int spd_tp_baseline_prefill(spd_ctx *ctx, const void *x, int32_t B, int32_t S, const int32_t *block_table, int32_t max_pages,
                            void *out, float *scratch, size_t scratch_floats, spd_allreduce_fn fn, void *user, void *stream)
{
    if (!ctx || !x || !block_table || !out || !scratch || !fn) return SPD_ENULL;
    Ctx &c = ctx->c;
    const spd_dims &d = c.d;
    if (d.T != 1 || d.dtype != 1 || d.block_kind != 0 || d.hidden % 16) return SPD_EINVAL;
    if (B < 1 || S < 1 || B > d.max_batch || x == out) return SPD_EINVAL;
    if (S > d.max_seq_len || (long)max_pages * d.kv_block_size < S) return SPD_ECAPACITY;
    const int Mp = d.max_prefill_tokens;
    const long chunk = (long)B * S < Mp ? (long)B * S : Mp;
    if (scratch_floats < (size_t)2 * chunk * d.hidden) return SPD_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    int total_launches = 0;
    auto run = [&](int b0, int nb, int s0, int ns) -> int {
        TokMap tm{0, b0, ns, s0, nullptr};
        const size_t off = ((size_t)b0 * S + s0) * d.hidden * 2;
        const int rc = run_tp_baseline(&c, (const char *)x + off, (char *)out + off, nb * ns, tm, block_table, max_pages, false, S, scratch,
                                       fn, user, st);
        total_launches += c.launches_last;
        return rc;
    };
    if (S <= Mp) {
        const int nb = Mp / S;
        for (int b0 = 0; b0 < B; b0 += nb) {
            const int rc = run(b0, B - b0 < nb ? B - b0 : nb, 0, S);
            if (rc) return rc;
        }
    } else {
        for (int b = 0; b < B; ++b)
            for (int s0 = 0; s0 < S; s0 += Mp) {
                const int rc = run(b, 1, s0, S - s0 < Mp ? S - s0 : Mp);
                if (rc) return rc;
            }
    }
    c.launches_last = total_launches;
    return SPD_OK;
}

int spd_gemm_bf16(const void *a, const void *w, float *c, int32_t M, int32_t N, int32_t K, int32_t batches,
                  int32_t a_batched, int32_t splits, int32_t swap, int32_t *err_flag, void *stream)
{
    if (!a || !w || !c || !err_flag) return SPD_ENULL;
    if (M < 1 || N < 1 || K < 8 || K % 8 || batches < 1 || splits < 1 || splits > (K + 63) / 64) return SPD_EINVAL;
    TcMap wm, am;
    const int tbox = tc_token_box(swap != 0, M);
    if (make_operand_map(&wm, w, K, N, batches, K, (long)N * K, 128)) return SPD_EINVAL;
    if (make_operand_map(&am, a, K, M, a_batched ? batches : 1, K, (long)M * K, tbox)) return SPD_EINVAL;
    TcGemmArgs g{};
    g.C = c; g.ldc = (long)batches * N; g.c_batch_stride = N; g.c_split_stride = (long)M * batches * N;
    g.t_rows = M; g.w_rows[0] = N; g.batches = batches; g.w_batched = batches > 1; g.t_batched = a_batched && batches > 1;
    g.num_kb = (K + 63) / 64; g.splits = splits; g.err = err_flag;
    const TcMap *wmaps[1] = {&wm};
    CU_TRY(launch_gemm_tc(wmaps, 1, am, g, swap != 0, (cudaStream_t)stream));
    return SPD_OK;
}

int spd_sync_points(const spd_ctx *ctx)
{
    if (!ctx) return SPD_ENULL;
    int n = 0;
    for (uint8_t m : ctx->c.mask) n += m ? 2 : 1;
    return n;
}

int spd_launches_per_decode_step(const spd_ctx *ctx) { return ctx ? ctx->c.launches_last : SPD_ENULL; }

int spd_device_error(spd_ctx *ctx, void *stream, int32_t *out_flag)
{
    if (!ctx || !out_flag) return SPD_ENULL;
    int flag = 0;
    int rc = read_err_flag(&ctx->c, (cudaStream_t)stream, &flag);
    *out_flag = flag;
    return rc;
}

int spd_profile_begin(spd_ctx *ctx)
{
    if (!ctx) return SPD_ENULL;
    ctx->c.profiling = true;
    ctx->c.ev_used = 0;
    ctx->c.ev_kind.clear();
    return SPD_OK;
}

int spd_profile_end(spd_ctx *ctx, void *stream, float *ms_by_kind, int32_t *launches_by_kind)
{
    if (!ctx || !ms_by_kind || !launches_by_kind) return SPD_ENULL;
    Ctx &c = ctx->c;
    c.profiling = false;
    CU_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    for (int k = 0; k < K_COUNT; ++k) { ms_by_kind[k] = 0.f; launches_by_kind[k] = 0; }
    for (size_t i = 0; i < c.ev_kind.size(); ++i) {
        float ms = 0.f;
        CU_TRY(cudaEventElapsedTime(&ms, c.ev_pool[2 * i], c.ev_pool[2 * i + 1]));
        ms_by_kind[c.ev_kind[i]] += ms;
        launches_by_kind[c.ev_kind[i]] += 1;
    }
    c.ev_used = 0;
    c.ev_kind.clear();
    return SPD_OK;
}

int spd_timeline_begin(spd_ctx *ctx, void *stream)
{
    if (!ctx) return SPD_ENULL;
    Ctx &c = ctx->c;
    cudaStream_t st = (cudaStream_t)stream;
    if (!c.timeline) drop_graphs(c); // steps captured so far carry no stamp slots; a second begin only clears the totals
    CU_TRY(cudaMemsetAsync(c.stamps, 0xFF, (size_t)c.stamps_cap * 16, st));
    CU_TRY(cudaMemsetAsync(c.stamps + 2 * (size_t)c.stamps_cap, 0, ((size_t)c.stamps_cap + 2) * 8, st));
    c.timeline = true;
    c.tl_next = 0;
    c.tl_kind.clear();
    return SPD_OK;
}

int spd_timeline_end(spd_ctx *ctx)
{
    if (!ctx) return SPD_ENULL;
    Ctx &c = ctx->c;
    drop_graphs(c);
    c.timeline = false;
    c.tl_next = 0;
    c.tl_kind.clear();
    return SPD_OK;
}

int spd_timeline_read(spd_ctx *ctx, void *stream, int32_t max_launches, int32_t *kinds, uint64_t *own_ns, int32_t *n_launches,
                      uint64_t *span_ns, uint64_t *n_calls)
{
    if (!ctx || !kinds || !own_ns || !n_launches || !span_ns || !n_calls) return SPD_ENULL;
    Ctx &c = ctx->c;
    if (!c.timeline || max_launches < 0) return SPD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    const int n = c.tl_next < max_launches ? c.tl_next : max_launches;
    std::vector<unsigned long long> host((size_t)c.stamps_cap + 2);
    CU_TRY(cudaMemcpyAsync(host.data(), c.stamps + 2 * (size_t)c.stamps_cap, host.size() * 8, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    for (int i = 0; i < n; ++i) { kinds[i] = c.tl_kind[i]; own_ns[i] = host[i]; }
    *n_launches = n;
    *span_ns = host[c.stamps_cap];
    *n_calls = host[(size_t)c.stamps_cap + 1];
    return SPD_OK;
}

int spd_profile_kinds(void) { return K_COUNT; }

const char *spd_profile_kind_name(int kind) { return (kind >= 0 && kind < K_COUNT) ? kind_names[kind] : "?"; }

void spd_destroy(spd_ctx *ctx)
{
    if (!ctx) return;
    for (cudaEvent_t e : ctx->c.ev_pool) cudaEventDestroy(e);
    for (GraphEntry &g : ctx->c.graphs) cudaGraphExecDestroy(g.exec);
    delete ctx;
}

const char *spd_status_string(int s)
{
    switch (s) {
    case SPD_OK: return "ok";
    case SPD_EINVAL: return "invalid argument or dimension";
    case SPD_ENULL: return "null pointer";
    case SPD_EWORKSPACE: return "workspace too small or misaligned";
    case SPD_ECAPACITY: return "sequence exceeds the KV capacity";
    case SPD_ECUDA: return "CUDA error";
    case SPD_EDEVICE: return "device-side error flag set";
    case SPD_ECALLBACK: return "the caller's all-reduce callback reported a failure";
    default: return "unknown status";
    }
}

int spd_last_cuda_error(void) { return g_last_cuda_error; }

} // extern "C"
