// Fused decode projections.  A decode step is bound by streaming every weight once, so each of
// the four projections of a block is one weight-streaming tcgen05 GEMM (weights on the 128-row
// MMA side, the few tokens on the N side), with the step that follows it folded into its tail.
//
// K is cut into P ranges so that every SM pulls weights; the P thread blocks of one output tile
// form a thread-block cluster.  After its main loop each block parks its fp32 partial tile in
// its own shared memory; after one cluster barrier block c adds up, in range order, the
// partials of the tokens c, c+P, ... through distributed shared memory and applies the fused
// step to them.  No partial ever goes through global memory and nobody spins on a flag.
//
//   EPI_QKV    : attention-RMSNorm rstd, rotary embedding, q store, K/V page append   (a2, a3)
//   EPI_OPROJ  : the cluster is the T emulated devices (K slice i gives Y_i).  sync block:
//                R = X + sum_i Y_i; SPD block (Sec. 4.1.1): R_i = X + Y_i per device, and
//                X + sum_i Y_i for the output residual; gain-scaled MLP inputs and their
//                partial sums of squares                                               (a5-a7)
//   EPI_GATEUP : MLP-RMSNorm rstd (per device in an SPD block), SwiGLU                 (a8)
//   EPI_DOWN   : the kept sync-point (sum over devices = K accumulation over all of F), output
//                residual, next block's gain-scaled input / final output               (a9, a10)
//   EPI_RESID_TP : o_proj / down of a rank that holds ONE shard (tensor parallelism across GPUs,
//                Sec. 3): the cluster adds up the K ranges of the rank's own partial, and the
//                sum over ranks - where the block keeps that sync-point - is an exchange through
//                peer-writable memory in the same tail (see TpArgs)
//
// Warps 0-3 own the accumulator rows (TMEM lanes) and run the epilogue; while the main loop runs
// they fetch what the epilogue needs (rstd, page addresses).  Warp 4 issues the TMA loads,
// warp 5 the MMAs.
#include "gemm_decode.cuh"

#include <math.h>
#include "tc_ptx.cuh"
#include "trace.cuh"

namespace spd {

namespace {

using namespace tc;

constexpr int MAX_GROUPS = 8; // emulated devices
constexpr int MAX_P = 8;      // portable cluster size
constexpr int THREADS = 192;

// ST = stages of the operand ring.  What a launch needs in flight to keep HBM busy is about 16 MB over all of its
// blocks (bandwidth x loaded latency): launches of 250-450 blocks want four stages (72-98 KB per block, three or two
// blocks per SM), not three; a third stage less only pays where it lets a launch of more than 444 blocks of 16-token
// tiles stay resident at once (four blocks per SM).  Chosen per launch, see launch_epi.
template <int BN, int ST> struct DCfg {
    static constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = ST;
    static constexpr int TMEM_COLS = BN < 32 ? 32 : BN;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 128 /*barriers, slot, flag*/;
    static_assert(8 * (2 * STAGES + 1) + 8 <= 128, "barrier area");
    static_assert(STAGES * STAGE_BYTES >= 2 * BN * 128 * 4, "ring too small for the staging tiles");
};

struct DecTile {
    int z, wt, wi, w_row0, t_row0, split, rank, P;
    int CL, zs; // blocks per cluster; partial planes per block (P = CL * zs planes add up to one output tile)
};

// Launcher-filled tiling constants travel behind the public arguments.
struct DecLaunch {
    DecGemmArgs g;
    int w_tiles_per_batch;
    int tile_start[3];
    int P;  // partial planes per output tile (K ranges, shard slices)
    int zs; // planes one block computes one after the other (row-split projection: shard slices); cluster size = gridDim.z = P / zs
};

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// 16 bytes of block `rank`'s shared memory at the offset that `local_addr` has in ours.
__device__ __forceinline__ float4 ld_peer4(uint32_t local_addr, uint32_t rank)
{
    uint32_t ra;
    float4 v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(ra) : "memory");
    return v;
}
__device__ __forceinline__ void add4(float4 &a, const float4 &b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
__device__ __forceinline__ float sq4(float4 v) { return v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w; }
__device__ __forceinline__ void store_bf16x4(bf16 *p, float4 v, float4 gn)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x * gn.x, v.y * gn.y), b = __floats2bfloat162_rn(v.z * gn.z, v.w * gn.w);
    uint2 u;
    u.x = *(uint32_t *)&a;
    u.y = *(uint32_t *)&b;
    *(uint2 *)p = u;
}

// The partials of token j, columns 4*lane..4*lane+3, from every block of the cluster (y[s] = range s).
// Plane s lies in block s / zs of the cluster, `plane_bytes` after that block's plane s - 1 (zs > 1).
__device__ __forceinline__ void load_partials(float4 (&y)[MAX_P], const float *S, int j, int lane, const DecTile &t, int plane_bytes)
{
    const float *src = S + j * 128 + 4 * lane;
    if (t.P == 1) { y[0] = *(const float4 *)src; return; }
    const uint32_t a = smem_u32(src);
    if (t.zs == 1) {
#pragma unroll
        for (int s = 0; s < MAX_P; ++s)
            if (s < t.P) y[s] = ld_peer4(a, (uint32_t)s);
    } else {
#pragma unroll
        for (int s = 0; s < MAX_P; ++s)
            if (s < t.P) y[s] = ld_peer4(a + (uint32_t)((s % t.zs) * plane_bytes), (uint32_t)(s / t.zs));
    }
}

// How many tokens of its tile this block finishes: tokens rank, rank + CL, ... below the tile's (ragged) end.
template <int BN> __device__ __forceinline__ int my_token_count(const DecGemmArgs &g, const DecTile &t)
{
    const int lim = g.t_rows - t.t_row0 < BN ? g.t_rows - t.t_row0 : BN;
    return lim > t.rank ? (lim - t.rank + t.CL - 1) / t.CL : 0;
}

// rstd of the tile's tokens from the partial sums of squares, by the 128 epilogue threads:
// thread t adds every (128/BN)-th partial of token t % BN, then the parts are added in order.
template <int BN>
__device__ __forceinline__ void compute_rstd(const SumSq &ss, int group, int t_row0, int t_rows, float *red, float *sm_rstd, float *sm_mu)
{
    constexpr int PARTS = 128 / BN;
    const int t = threadIdx.x, j = t % BN, part = t / BN, m = t_row0 + j;
    float acc = 0.f, sum = 0.f;
    if (m < t_rows)
        for (int tile = part; tile < ss.tiles; tile += PARTS) {
            const long i = ((long)tile * ss.groups + group) * ss.Mcap + m;
            acc += __ldcg(ss.part + i);
            if (ss.sum) sum += __ldcg(ss.sum + i);
        }
    // (the row sums of LayerNorm go through the same 128 words in a second round: static shared memory decides whether
    // a third block of 16-token tiles fits an SM)
    float mu = 0.f;
    if (ss.sum) {
        red[t] = sum;
        epi_sync();
        if (t < BN) {
#pragma unroll
            for (int q = 0; q < PARTS; ++q) mu += red[q * BN + t];
            mu /= (float)ss.H;
        }
        epi_sync();
    }
    red[t] = acc;
    epi_sync();
    float tot = 0.f;
    if (t < BN) {
#pragma unroll
        for (int q = 0; q < PARTS; ++q) tot += red[q * BN + t];
    }
    epi_sync(); // sm_rstd and sm_mu are the two halves of `red`: every partial has been read before they are written
    if (t < BN) {
        // LayerNorm: variance about the mean
        sm_rstd[t] = ss.sum ? rsqrtf(fmaxf(tot / (float)ss.H - mu * mu, 0.f) + ss.eps) : rsqrtf(tot / (float)ss.H + ss.eps);
        sm_mu[t] = mu;
    }
}

// ---- epilogues: block `rank` of the cluster finishes tokens rank, rank+P, ... of the tile ----------
// Gathers run with warp w on the block's w-th, (w+4)-th ... token and lane l on columns 4l..4l+3.

template <int BN>
__device__ __forceinline__ void gather_my_tokens(const DecGemmArgs &g, const DecTile &t, const float *S, float *Gb)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mine = my_token_count<BN>(g, t);
#pragma unroll 2
    for (int q = warp; q < mine; q += 4) {
        const int j = t.rank + t.CL * q;
        float4 y[MAX_P];
        load_partials(y, S, j, lane, t, BN * 128 * 4);
        float4 v = y[0];
#pragma unroll
        for (int s = 1; s < MAX_P; ++s)
            if (s < t.P) add4(v, y[s]);
        *(float4 *)(Gb + q * 128 + 4 * lane) = v;
    }
}

template <int BN>
__device__ __forceinline__ void epilogue_qkv(const DecGemmArgs &g, const DecTile &t, const float *S, float *Gb,
                                             const float *sm_rstd, const float *sm_mu, const long *sm_kvoff)
{
    const int r = threadIdx.x, d = g.head_dim, half = d >> 1;
    // weights batched by shard (rank mode): batch z holds heads z * heads_per_shard ...
    const int row = t.w_row0 + r, head = row / d + t.z * (g.w_rows[t.wi] / d), jd = row % d, nq = g.n_q_heads;
    const bool row_valid = row < g.w_rows[t.wi];
    const bool rot = t.wi < 2 && g.rope != nullptr;
    // The rotary factors do not depend on the gather: the first chunk is requested before it, and every later chunk
    // while the chunk before it is written, so that the loop never waits for a load it has only just issued.
    const int mine = my_token_count<BN>(g, t);
    constexpr int CH = 8;
    const int jj = jd < half ? jd : jd - half;
    float2 nxt[CH];
    auto fetch = [&](int q0) {
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            nxt[u] = make_float2(1.f, 0.f);
            if (rot && row_valid && q0 + u < mine) nxt[u] = g.rope[(long)(t.t_row0 + t.rank + t.CL * (q0 + u)) * half + jj];
        }
    };
    fetch(0);
    gather_my_tokens<BN>(g, t, S, Gb);
    epi_sync();
    if (!row_valid) return;
    const int partner = jd < half ? r + half : r - half;
    // LayerNorm folded into the tail: this weight row's sum of g * W and its beta * W + bias
    float wg = 0.f, wb = 0.f;
    if (g.ln_wg) {
        const int vrow = (t.wi == 0 ? 0 : (t.wi == 1 ? g.w_rows[0] : g.w_rows[0] + g.w_rows[1])) + row;
        wg = g.ln_wg[vrow];
        wb = g.ln_wb[vrow];
    }
    bf16 *const dst = t.wi == 0 ? (bf16 *)g.q_out : (bf16 *)(t.wi == 1 ? g.k_pages : g.v_pages);
    for (int q0 = 0; q0 < mine; q0 += CH) {
        float2 cur[CH];
#pragma unroll
        for (int u = 0; u < CH; ++u) cur[u] = nxt[u];
        if (rot && q0 + CH < mine) fetch(q0 + CH);
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            const int q = q0 + u;
            if (q >= mine) break;
            const int j = t.rank + t.CL * q, m = t.t_row0 + j;
            float v = (Gb[q * 128 + r] - sm_mu[j] * wg) * sm_rstd[j] + wb;
            if (rot) {
                const float o = Gb[q * 128 + partner] * sm_rstd[j];
                v = jd < half ? v * cur[u].x - o * cur[u].y : v * cur[u].x + o * cur[u].y;
            }
            if (t.wi == 0) {
                dst[((long)m * nq + head) * d + jd] = __float2bfloat16_rn(v);
            } else {
                const long off = sm_kvoff[j];
                if (off >= 0) dst[off + (long)head * g.pt.block * d + jd] = __float2bfloat16_rn(v);
            }
        }
    }
}

template <int BN>
__device__ __forceinline__ void epilogue_gateup(const DecGemmArgs &g, const DecTile &t, const float *S, float *Gb, const float *sm_rstd,
                                                const float *sm_mu)
{
    gather_my_tokens<BN>(g, t, S, Gb);
    epi_sync();
    if (g.fc1_only) {
        // block with bias: the tile holds 128 consecutive rows of fc1; LayerNorm folded in, bias, ReLU
        for (int idx = threadIdx.x;; idx += 128) {
            const int q = idx >> 6, rr = 2 * (idx & 63), j = t.rank + t.CL * q, m = t.t_row0 + j, f = t.w_row0 + rr;
            if (j >= BN || m >= g.t_rows) break;
            if (f >= g.Fs) continue;
            const float rs = sm_rstd[j], mu = sm_mu[j];
            const float2 a = *(const float2 *)(Gb + q * 128 + rr);
            const float2 wg = *(const float2 *)(g.ln_wg + (long)t.z * g.Fs + f), wb = *(const float2 *)(g.ln_wb + (long)t.z * g.Fs + f);
            *(__nv_bfloat162 *)((bf16 *)g.act + (long)m * g.F + (long)t.z * g.Fs + f) =
                __floats2bfloat162_rn(fmaxf((a.x - mu * wg.x) * rs + wb.x, 0.f), fmaxf((a.y - mu * wg.y) * rs + wb.y, 0.f));
        }
        return;
    }
    // two FFN columns per thread: 32 threads cover the tile's 64 columns of one token
    for (int idx = threadIdx.x;; idx += 128) {
        const int q = idx >> 5, rr = 2 * (idx & 31), j = t.rank + t.CL * q, m = t.t_row0 + j, f = t.w_row0 + rr;
        if (j >= BN || m >= g.t_rows) break;
        if (f >= g.Fs) continue;
        const float rs = sm_rstd[j];
        const float2 gt = *(const float2 *)(Gb + q * 128 + rr), up = *(const float2 *)(Gb + q * 128 + 64 + rr);
        const float g0 = gt.x * rs, g1 = gt.y * rs;
        *(__nv_bfloat162 *)((bf16 *)g.act + (long)m * g.F + (long)t.z * g.Fs + f) =
            __floats2bfloat162_rn(g0 / (1.f + __expf(-g0)) * (up.x * rs), g1 / (1.f + __expf(-g1)) * (up.y * rs));
    }
}

// xpre[u] for a run-time u in 0..3 without indexing the register array.
__device__ __forceinline__ float4 pick4(const float4 (&v)[4], int u)
{
    float4 r = v[0];
    if (u == 1) r = v[1];
    if (u == 2) r = v[2];
    if (u == 3) r = v[3];
    return r;
}

// Eight per-lane values, each to be summed over the warp: instead of eight butterflies (40 shuffles) the lanes swap
// halves of the value list while they halve the lane distance (4 + 2 + 1 shuffles), then two plain steps.  Returns, in
// every lane, the warp total of v[4 * bit4(lane) + 2 * bit3(lane) + bit2(lane)].
__device__ __forceinline__ float warp_sum8(const float (&v)[8], int lane)
{
    const bool h16 = (lane & 16) != 0, h8 = (lane & 8) != 0, h4 = (lane & 4) != 0;
    float a[4], b[2];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = (h16 ? v[i + 4] : v[i]) + __shfl_xor_sync(0xffffffffu, h16 ? v[i] : v[i + 4], 16);
#pragma unroll
    for (int i = 0; i < 2; ++i) b[i] = (h8 ? a[i + 2] : a[i]) + __shfl_xor_sync(0xffffffffu, h8 ? a[i] : a[i + 2], 8);
    float w = (h4 ? b[1] : b[0]) + __shfl_xor_sync(0xffffffffu, h4 ? b[0] : b[1], 4);
    w += __shfl_xor_sync(0xffffffffu, w, 2);
    w += __shfl_xor_sync(0xffffffffu, w, 1);
    return w;
}

// Residual stream out, gain-scaled bf16 copy (the next GEMM's input) and the tile's partial sums
// of squares.  spd_groups (o_proj of an SPD block): range i of the cluster is emulated device i,
// which only ever sees its own partial attention output Y_i (R_i = X + Y_i), while the carried
// residual collects every Y_i.
template <int BN>
__device__ __forceinline__ void epilogue_residual(const DecGemmArgs &g, const DecTile &t, const float *S, bool spd_groups,
                                                  const float4 (&xpre)[4])
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = t.w_row0 + 4 * lane, H = g.H;
    const bool valid = n < H;
    const int G = spd_groups ? g.n_groups : 1, per = t.P / G; // ranges per device
    const float4 one = make_float4(1.f, 1.f, 1.f, 1.f);
    float4 gn = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid && g.gain) {
        const uint2 u = *(const uint2 *)((const bf16 *)g.gain + n);
        const float2 a = __bfloat1622float2(*(const __nv_bfloat162 *)&u.x), b = __bfloat1622float2(*(const __nv_bfloat162 *)&u.y);
        gn = make_float4(a.x, a.y, b.x, b.y);
    }
    // block with bias: the bias of the row-split layer joins the residual stream once - and with it every device's X + P_i
    float4 bias = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid && g.bias) {
        const uint2 u = *(const uint2 *)((const bf16 *)g.bias + n);
        const float2 a = __bfloat1622float2(*(const __nv_bfloat162 *)&u.x), b = __bfloat1622float2(*(const __nv_bfloat162 *)&u.y);
        bias = make_float4(a.x, a.y, b.x, b.y);
    }
    auto sum4 = [](float4 v) { return v.x + v.y + v.z + v.w; };
    if (spd_groups) {
        const int rows = (g.t_rows - t.t_row0 < BN ? g.t_rows - t.t_row0 : BN) - t.rank; // this block's tokens: every P-th of them
        if (BN < 64 && rows > 3 * t.CL) {
            // Four tokens or more: one token per warp at a time, the devices of a token in turn (one gather of the
            // partials per token instead of one per warp and token).
            for (int q = warp;; q += 4) {
                const int j = t.rank + t.CL * q, m = t.t_row0 + j;
                if (j >= BN || m >= g.t_rows) break;
                const long idx = (long)m * H + n;
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (valid) { x = *(const float4 *)(g.res_in + idx); add4(x, bias); }
                float4 y[MAX_P];
                load_partials(y, S, j, lane, t, BN * 128 * 4);
                float4 tot = make_float4(0.f, 0.f, 0.f, 0.f), yi = make_float4(0.f, 0.f, 0.f, 0.f);
                int cnt = 0, i = 0;
#pragma unroll
                for (int s = 0; s < MAX_P; ++s) {
                    if (s >= t.P) continue;
                    add4(yi, y[s]);
                    if (++cnt < per) continue;
                    add4(tot, yi);
                    float4 ri = x;
                    add4(ri, yi);
                    if (valid && g.hg) store_bf16x4((bf16 *)g.hg + (long)i * g.hg_stride + idx, ri, gn);
                    const float sq = warp_sum(valid ? sq4(ri) : 0.f);
                    if (lane == 0 && g.ss_out) g.ss_out[((long)t.wt * G + i) * g.Mcap + m] = sq;
                    if (g.sum_out) {
                        const float sm = warp_sum(valid ? sum4(ri) : 0.f);
                        if (lane == 0) g.sum_out[((long)t.wt * G + i) * g.Mcap + m] = sm;
                    }
                    yi = make_float4(0.f, 0.f, 0.f, 0.f);
                    cnt = 0;
                    ++i;
                }
                add4(x, tot);
                if (valid && g.res_out) *(float4 *)(g.res_out + idx) = x;
            }
            return;
        }
        if (BN >= 64 && rows > 3 * t.CL) {
            // 64-token tiles: as above, with the per-device row sums reduced together and the residual rows fetched ahead.
            const int mine = my_token_count<BN>(g, t);
            const int dev_of_lane = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
            for (int q = warp, u = 0; q < mine; q += 4, ++u) {
                const int j = t.rank + t.CL * q, m = t.t_row0 + j;
                const long idx = (long)m * H + n;
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (valid) { x = (BN >= 64 && u < 4) ? pick4(xpre, u) : *(const float4 *)(g.res_in + idx); add4(x, bias); }
                float4 y[MAX_P];
                load_partials(y, S, j, lane, t, BN * 128 * 4);
                float4 tot = make_float4(0.f, 0.f, 0.f, 0.f), yi = make_float4(0.f, 0.f, 0.f, 0.f);
                float sq[8], sm[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) sq[i] = sm[i] = 0.f;
                int cnt = 0, i = 0;
#pragma unroll
                for (int s = 0; s < MAX_P; ++s) {
                    if (s >= t.P) continue;
                    add4(yi, y[s]);
                    if (++cnt < per) continue;
                    add4(tot, yi);
                    float4 ri = x;
                    add4(ri, yi);
                    if (valid && g.hg) store_bf16x4((bf16 *)g.hg + (long)i * g.hg_stride + idx, ri, gn);
                    // device i's slot: i only grows with s, so after unrolling every index below is a constant
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (e == i) { sq[e] = valid ? sq4(ri) : 0.f; sm[e] = valid ? sum4(ri) : 0.f; }
                    yi = make_float4(0.f, 0.f, 0.f, 0.f);
                    cnt = 0;
                    ++i;
                }
                const float sqt = warp_sum8(sq, lane);
                if ((lane & 3) == 0 && dev_of_lane < G && g.ss_out) g.ss_out[((long)t.wt * G + dev_of_lane) * g.Mcap + m] = sqt;
                if (g.sum_out) {
                    const float smt = warp_sum8(sm, lane);
                    if ((lane & 3) == 0 && dev_of_lane < G) g.sum_out[((long)t.wt * G + dev_of_lane) * g.Mcap + m] = smt;
                }
                add4(x, tot);
                if (valid && g.res_out) *(float4 *)(g.res_out + idx) = x;
            }
            return;
        }
        // All four warps work on the same token; warp w finishes devices w, w+4 (ranges i*per .. i*per+per-1 are
        // device i), so that the per-device stores and reductions of a block with few tokens run side by side.
        for (int q = 0;; ++q) {
            const int j = t.rank + t.CL * q, m = t.t_row0 + j;
            if (j >= BN || m >= g.t_rows) break;
            const long idx = (long)m * H + n;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (valid) { x = *(const float4 *)(g.res_in + idx); add4(x, bias); }
            float4 y[MAX_P];
            load_partials(y, S, j, lane, t, BN * 128 * 4);
            float4 tot = make_float4(0.f, 0.f, 0.f, 0.f), yi = make_float4(0.f, 0.f, 0.f, 0.f);
            int cnt = 0, i = 0;
#pragma unroll
            for (int s = 0; s < MAX_P; ++s) {
                if (s >= t.P) continue;
                add4(yi, y[s]);
                if (++cnt < per) continue;
                add4(tot, yi);
                if ((i & 3) == warp) {
                    float4 ri = x;
                    add4(ri, yi);
                    if (valid && g.hg) store_bf16x4((bf16 *)g.hg + (long)i * g.hg_stride + idx, ri, gn);
                    const float sq = warp_sum(valid ? sq4(ri) : 0.f);
                    if (lane == 0 && g.ss_out) g.ss_out[((long)t.wt * G + i) * g.Mcap + m] = sq;
                    if (g.sum_out) {
                        const float sm = warp_sum(valid ? sum4(ri) : 0.f);
                        if (lane == 0) g.sum_out[((long)t.wt * G + i) * g.Mcap + m] = sm;
                    }
                }
                yi = make_float4(0.f, 0.f, 0.f, 0.f);
                cnt = 0;
                ++i;
            }
            add4(x, tot);
            if (warp == 0 && valid && g.res_out) *(float4 *)(g.res_out + idx) = x;
        }
        return;
    }
    const int mine = my_token_count<BN>(g, t);
    for (int q = warp, u = 0; q < mine; q += 4, ++u) {
        const int j = t.rank + t.CL * q, m = t.t_row0 + j;
        const long idx = (long)m * H + n;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) { x = (BN >= 64 && u < 4) ? pick4(xpre, u) : *(const float4 *)(g.res_in + idx); add4(x, bias); }
        float4 y[MAX_P];
        load_partials(y, S, j, lane, t, BN * 128 * 4);
        float4 tot = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < MAX_P; ++s)
            if (s < t.P) add4(tot, y[s]);
        add4(x, tot);
        if (valid) {
            if (g.res_out) *(float4 *)(g.res_out + idx) = x;
            if (g.final_out) store_bf16x4((bf16 *)g.final_out + idx, x, one);
            if (g.hg) store_bf16x4((bf16 *)g.hg + idx, x, gn);
        }
        if (g.ss_out) {
            const float sq = warp_sum(valid ? sq4(x) : 0.f);
            if (lane == 0) g.ss_out[(long)t.wt * g.Mcap + m] = sq;
        }
        if (g.sum_out) {
            const float sm = warp_sum(valid ? sum4(x) : 0.f);
            if (lane == 0) g.sum_out[(long)t.wt * g.Mcap + m] = sm;
        }
    }
}

__device__ __forceinline__ unsigned ld_acquire_sys(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys(unsigned *p, unsigned v)
{
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Rank z's partial rows (its K ranges added up through the cluster), optionally exchanged with the
// other ranks and summed in rank order, then the residual, the gain-scaled input of the next GEMM
// and its partial sums of squares - all in rank z's own planes.
template <int BN>
__device__ __forceinline__ void epilogue_resid_tp(const DecGemmArgs &g, const DecTile &t, const float *S, volatile int *abort_flag)
{
    const TpArgs &tp = g.tp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = t.w_row0 + 4 * lane, H = g.H;
    const bool valid = n < H;
    const long zoff = (long)t.z * tp.z_stride;
    const int me = tp.rank_base + t.z;
    const unsigned step = *(const unsigned *)((const char *)tp.step + zoff);
    const long buf_off = (long)(tp.buf & 1) * tp.buf_bytes;
    const float4 one = make_float4(1.f, 1.f, 1.f, 1.f);
    float4 gn = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid && g.gain) {
        const uint2 u = *(const uint2 *)((const bf16 *)g.gain + n);
        const float2 a = __bfloat1622float2(*(const __nv_bfloat162 *)&u.x), b = __bfloat1622float2(*(const __nv_bfloat162 *)&u.y);
        gn = make_float4(a.x, a.y, b.x, b.y);
    }
    // token m, columns n..n+3: the summed update `tot` joins the rank's residual stream
    auto finish = [&](int m, float4 tot) {
        const long idx = (long)m * H + n;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) {
            x = *(const float4 *)((const char *)g.res_in + zoff + idx * 4);
            add4(x, tot);
            if (g.res_out) *(float4 *)((char *)g.res_out + zoff + idx * 4) = x;
            if (g.final_out) store_bf16x4((bf16 *)((char *)g.final_out + (long)t.z * tp.out_stride) + idx, x, one);
            if (g.hg) store_bf16x4((bf16 *)((char *)g.hg + zoff) + idx, x, gn);
        }
        if (g.ss_out) {
            const float sq = warp_sum(valid ? sq4(x) : 0.f);
            if (lane == 0) ((float *)((char *)g.ss_out + zoff))[(long)t.wt * g.Mcap + m] = sq;
        }
    };
    for (int q = warp;; q += 4) {
        const int j = t.rank + t.CL * q, m = t.t_row0 + j;
        if (j >= BN || m >= g.t_rows) break;
        const long idx = (long)m * H + n;
        float4 y[MAX_P];
        load_partials(y, S, j, lane, t, BN * 128 * 4);
        float4 p = y[0];
#pragma unroll
        for (int s = 1; s < MAX_P; ++s)
            if (s < t.P) add4(p, y[s]);
        if (valid) {
            if (tp.addend) add4(p, *(const float4 *)((const char *)tp.addend + zoff + idx * 4));
            if (tp.ysave) *(float4 *)((char *)tp.ysave + zoff + idx * 4) = p;
            if (tp.exchange)
                for (int i = 0; i < tp.T; ++i) { // own rank first, then the peers round the ring: no two ranks aim at one peer at once
                    const int r = me + i < tp.T ? me + i : me + i - tp.T;
                    *(float4 *)(tp.rx[r] + buf_off + (long)me * tp.src_bytes + idx * 4) = p;
                }
        }
        if (!tp.exchange) finish(m, p);
    }
    if (!tp.exchange) return;
    // every row of this block is on its way: publish the step on every rank, then wait for all sources
    epi_sync();
    const long tile_flags = ((long)t.wt * gridDim.y + blockIdx.y) * tp.T * TP_FLAG_RANGES;
    if ((int)threadIdx.x < tp.T) { // the release orders the block's rows (made visible to this thread by the barrier) before the flag
        st_release_sys(tp.flags[threadIdx.x] + tile_flags + me * TP_FLAG_RANGES + t.rank, step);
    }
    if (warp == 0) {
        const unsigned *mine = tp.flags[me] + tile_flags;
        const unsigned long long t0 = global_ns();
        for (;;) {
            bool done = true;
            for (int e = lane; e < tp.T * TP_FLAG_RANGES; e += 32)
                if (e % TP_FLAG_RANGES < t.P && (int)(ld_acquire_sys(mine + e) - step) < 0) done = false;
            if (__all_sync(0xffffffffu, done)) break;
            // a rank that never arrives (or an earlier give-up in this step) ends the wait: no trap, the host reads the flag
            if (*abort_flag || (*(volatile int *)g.err & ERR_PEER_TIMEOUT) || global_ns() - t0 > g.tp.wait_ns) {
                if (lane == 0) { *abort_flag = 1; atomicOr(g.err, ERR_PEER_TIMEOUT); }
                break;
            }
        }
    }
    epi_sync();
    if (*abort_flag) return;
    for (int q = warp;; q += 4) {
        const int j = t.rank + t.CL * q, m = t.t_row0 + j;
        if (j >= BN || m >= g.t_rows) break;
        float4 tot = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid)
            for (int r = 0; r < tp.T; ++r)
                add4(tot, __ldcg((const float4 *)(tp.rx[me] + buf_off + (long)r * tp.src_bytes + ((long)m * H + n) * 4)));
        finish(m, tot);
    }
}

// Resident blocks per SM the register file must allow: four at 16-token tiles (the three-stage ring), three at 32,
// two at 64 (the ring, not the registers, is the limit there).
template <int BN, int EPI, int ST>
__global__ void __launch_bounds__(THREADS, BN == 16 ? 4 : (BN == 32 ? 3 : 2)) gemm_decode_kernel(const __grid_constant__ CUtensorMap tm_w0,
                                                              const __grid_constant__ CUtensorMap tm_w1,
                                                              const __grid_constant__ CUtensorMap tm_w2,
                                                              const __grid_constant__ CUtensorMap tm_t,
                                                              const __grid_constant__ DecLaunch L)
{
    using C = DCfg<BN, ST>;
    constexpr int SUB = (EPI == EPI_GATEUP) ? 2 : 1; // weight boxes per tile
    constexpr int ROWS = BM / SUB;                   // weight rows per box
    const DecGemmArgs &g = L.g;
    extern __shared__ uint8_t smem_raw[];
    // Static shared memory counts: at 16-token tiles with a three-stage ring a fourth block fits an SM only while ring +
    // barriers + this stay under 57 KB.  The reduction scratch of the row statistics becomes their home afterwards.
    __shared__ float sm_red[128];
    float *const sm_rstd = sm_red, *const sm_mu = sm_red + 64;
    __shared__ long sm_kvoff[64];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + C::STAGES * C::STAGE_BYTES; // full[S], empty[S], tmem_full
    uint32_t *tmem_slot = (uint32_t *)(gen_base + C::STAGES * C::STAGE_BYTES + 8 * (2 * C::STAGES + 1));
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (C::STAGES + s); };
    const uint32_t tmem_full_bar = bars + 8u * (2 * C::STAGES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float4 xpre[4] = {}; // epilogue warps of the residual tails: residual rows fetched ahead
    DecTile t;
    t.P = L.P;
    t.zs = L.zs;
    t.CL = L.P / L.zs;
    t.rank = t.CL > 1 ? (int)cluster_rank() : 0;
    // zs > 1 (whole shard slices only, splits == 1): this block computes planes rank * zs ... rank * zs + zs - 1
    if (g.z_is_plane) { t.z = t.zs > 1 ? t.rank * t.zs : t.rank / g.splits; t.split = t.zs > 1 ? 0 : t.rank % g.splits; t.wt = blockIdx.x; }
    else { t.z = blockIdx.x / L.w_tiles_per_batch; t.split = t.rank; t.wt = blockIdx.x % L.w_tiles_per_batch; }
    t.wi = (SUB == 2) ? 0 : ((t.wt >= L.tile_start[2]) ? 2 : ((t.wt >= L.tile_start[1]) ? 1 : 0));
    t.w_row0 = (t.wt - L.tile_start[t.wi]) * ((EPI == EPI_GATEUP && g.fc1_only) ? BM : ROWS);
    t.t_row0 = blockIdx.y * BN;
    const CUtensorMap *tm_w = t.wi == 0 ? &tm_w0 : (t.wi == 1 ? &tm_w1 : &tm_w2);
    const int kb_begin = (int)((long)g.num_kb * t.split / g.splits);
    const int kb_end = (int)((long)g.num_kb * (t.split + 1) / g.splits);
    const int n_kb = kb_end - kb_begin;
    const int n_it = n_kb * t.zs; // ring iterations: the K blocks of plane 0, then those of plane 1, ...
    const uint32_t tmem_cols = (uint32_t)(BN * t.zs < 32 ? 32 : BN * t.zs); // zs is 1 or 2: a power of two

    pdl_launch_dependents();
    const int az0 = g.w_batched ? t.z : 0, bz0 = g.t_batched ? t.z : 0;
    const uint64_t stream_once = policy_evict_first();
    auto load_w = [&](int s, int it) {
        const int lp = it >= n_kb ? 1 : 0, kx = (kb_begin + it - lp * n_kb) * BK, a_z = az0 + lp; // at most two planes
        const uint32_t sa = base + s * C::STAGE_BYTES;
        if (SUB == 1) tma_load_3d_hint(sa, tm_w, kx, t.w_row0, a_z, full_bar(s), stream_once);
        else {
            tma_load_3d_hint(sa, &tm_w0, kx, t.w_row0, a_z, full_bar(s), stream_once);
            if (g.fc1_only) tma_load_3d_hint(sa + ROWS * BK * 2, &tm_w0, kx, t.w_row0 + ROWS, a_z, full_bar(s), stream_once);
            else tma_load_3d_hint(sa + ROWS * BK * 2, &tm_w1, kx, t.w_row0, a_z, full_bar(s), stream_once);
        }
    };
    // the same tile requested into L2 only
    auto prefetch_w = [&](int it) {
        const int lp = it >= n_kb ? 1 : 0, kx = (kb_begin + it - lp * n_kb) * BK, a_z = az0 + lp; // at most two planes
        if (SUB == 1) tma_prefetch_l2_3d(tm_w, kx, t.w_row0, a_z);
        else { tma_prefetch_l2_3d(&tm_w0, kx, t.w_row0, a_z); tma_prefetch_l2_3d(g.fc1_only ? &tm_w0 : &tm_w1, kx, t.w_row0 + (g.fc1_only ? ROWS : 0), a_z); }
    };
    const int pre = n_it < C::STAGES ? n_it : C::STAGES;
    if (warp == 4 && lane == 0) {
        // The TMA thread sets up the barriers itself and requests the first ring of weight tiles
        // at once: weights do not depend on the preceding kernel, and they need neither the
        // accumulator allocation nor the other warps, so this GEMM's weight stream starts the
        // moment the block is resident - under the tail of whatever ran before.
        SPD_TRACE_EVENT(EPI, TR_START);
        stamp_entry(g.stamp);
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(tm_w) : "memory");
        if (SUB == 2) asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w1) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_t) : "memory");
        for (int i = 0; i < pre; ++i) {
            mbar_expect_tx(full_bar(i), C::STAGE_BYTES);
            load_w(i, i);
        }
        // optionally the K blocks after the ring are pulled into L2 (once: keeping that distance through the loop
        // was measured 25 % slower at 64-token tiles)
        const int pf_end = n_it < pre + g.l2_prefetch_kb ? n_it : pre + g.l2_prefetch_kb;
        for (int i = pre; i < pf_end; ++i) prefetch_w(i);
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 4) {
        if (lane == 0) {
            pdl_wait();
            SPD_TRACE_EVENT(EPI, TR_DEP_DONE);
            for (int i = 0; i < n_it; ++i) {
                const int s = i % C::STAGES;
                if (i >= pre) {
                    if (!mbar_wait(empty_bar(s), ((i / C::STAGES) & 1) ^ 1, g.err, abort_flag)) break;
                    mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
                    load_w(s, i);
                }
                const int lp = i >= n_kb ? 1 : 0;
                tma_load_3d(base + s * C::STAGE_BYTES + C::A_BYTES, &tm_t, (kb_begin + i - lp * n_kb) * BK, t.t_row0, bz0 + lp, full_bar(s));
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BN);
            for (int i = 0; i < n_it; ++i) {
                const int s = i % C::STAGES;
                if (!mbar_wait(full_bar(s), (i / C::STAGES) & 1, g.err, abort_flag)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = base + s * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                const uint64_t da = make_desc(sa), db = make_desc(sb);
                const int lp = i >= n_kb ? 1 : 0, kk = i - lp * n_kb;
                const uint32_t acc = tmem_acc + (uint32_t)(lp * BN); // each plane has its own accumulator columns
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k)
                    umma(acc, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                         (kk > 0 || k > 0) ? 1u : 0u);
                umma_commit(empty_bar(s));
            }
            umma_commit(tmem_full_bar);
        }
        __syncwarp();
    } else {
        // epilogue warps: fetch what the tail needs while the weights stream
        pdl_wait();
        if (EPI == EPI_QKV || EPI == EPI_GATEUP) {
            SumSq ss = g.ss_in;
            if (g.tp.on) ss.part = (const float *)((const char *)ss.part + (long)t.z * g.tp.z_stride); // rank z's own sums
            compute_rstd<BN>(ss, (EPI == EPI_GATEUP && g.rstd_per_shard && !g.tp.on) ? t.z : 0, t.t_row0, g.t_rows, sm_red, sm_rstd, sm_mu);
        }
        if (EPI == EPI_QKV && t.wi > 0 && threadIdx.x < BN) {
            // where this token's K / V row of kv head 0 goes; < 0: skip (the error flag says why)
            const int m = t.t_row0 + threadIdx.x;
            long off = -1;
            if (m < g.t_rows) {
                int b, pos;
                g.tm.locate(m, b, pos);
                const int pi = pos / g.pt.block;
                if (pos < 0 || pi >= g.pt.max_pages) atomicOr(g.err, ERR_CAPACITY);
                else {
                    const int page = g.pt.block_table[(long)b * g.pt.max_pages + pi];
                    if (page < 0 || page >= g.pt.n_pages) atomicOr(g.err, ERR_PAGE_RANGE);
                    else off = ((long)page * g.pt.n_kv_heads * g.pt.block + pos % g.pt.block) * g.head_dim;
                }
            }
            sm_kvoff[threadIdx.x] = off;
        }
        if (BN >= 64 && (EPI == EPI_OPROJ || EPI == EPI_DOWN)) {
            // the residual rows this warp will finish first (tokens rank + CL * (warp + 4u)): requested while the weights stream
            const int n = t.w_row0 + 4 * lane, mine = my_token_count<BN>(g, t);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (n < g.H && warp + 4 * u < mine)
                    xpre[u] = *(const float4 *)(g.res_in + (long)(t.t_row0 + t.rank + t.CL * (warp + 4 * u)) * g.H + n);
        }
        // accumulator -> registers: warp w owns TMEM lanes [32w, 32w+32); thread r = accumulator row r
        const bool acc_ok = mbar_wait(tmem_full_bar, 0, g.err, abort_flag);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        __syncwarp();
        if (threadIdx.x == 0) SPD_TRACE_EVENT(EPI, TR_MAIN_DONE);
        // The ring is free once the accumulators are complete (every TMA write has landed and every
        // MMA has read its operands): park the partial tiles there, token-major, plane after plane.
        for (int lp = 0; lp < t.zs; ++lp) {
            float acc[BN];
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 16) {
                if (acc_ok) tmem_ld16(tmem_acc + ((uint32_t)(warp * 32) << 16) + (uint32_t)(lp * BN + c0), acc + c0);
                else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) acc[c0 + i] = 0.f;
                }
            }
            float *S = (float *)gen_base + lp * BN * 128;
#pragma unroll
            for (int j = 0; j < BN; ++j) S[j * 128 + threadIdx.x] = acc[j];
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    // partial tiles of all ranges visible cluster-wide
    if (t.CL > 1) cluster_sync_all();
    else __syncthreads();
    if (warp == 5) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(tmem_cols) : "memory");
    }
    if (warp < 4) {
        if (threadIdx.x == 0) SPD_TRACE_EVENT(EPI, TR_ARRIVED);
        const float *S = (const float *)gen_base;
        float *Gb = (float *)gen_base + BN * 128; // this block's gathered tokens
        if (EPI == EPI_QKV) epilogue_qkv<BN>(g, t, S, Gb, sm_rstd, sm_mu, sm_kvoff);
        else if (EPI == EPI_GATEUP) epilogue_gateup<BN>(g, t, S, Gb, sm_rstd, sm_mu);
        else if (EPI == EPI_RESID_TP) epilogue_resid_tp<BN>(g, t, S, abort_flag);
        else epilogue_residual<BN>(g, t, S, EPI == EPI_OPROJ && g.n_groups > 1, xpre);
        if (threadIdx.x == 0) { SPD_TRACE_EVENT(EPI, TR_END); stamp_exit(g.stamp); }
    }
    // no block may exit while a peer still reads its shared memory
    if (t.CL > 1) cluster_sync_all();
}

template <int BN, int EPI, int ST>
cudaError_t launch_cfg(const CUtensorMap *const *tw, const CUtensorMap &tt, const DecLaunch &L, dim3 grid, cudaStream_t st)
{
    using C = DCfg<BN, ST>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemm_decode_kernel<BN, EPI, ST>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(gemm_decode_kernel<BN, EPI, ST>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = 1;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = grid.z;
    cfg.attrs = at;
    cfg.numAttrs = grid.z > 1 ? 2 : 1;
    if (EPI == EPI_RESID_TP && L.g.tp.exchange && L.g.batches > 1) {
        // Several ranks in one launch: their blocks wait on one another, so all of them must be resident at once.
        // Blocks per SM from the kernel's own footprint (the launch takes the largest shared-memory carveout, which
        // the occupancy query does not assume), clusters per GPU scaled from the query's answer.
        cudaLaunchConfig_t occ = cfg;
        occ.numAttrs = 2;
        int clusters = 0, api_per_sm = 0, dev = 0, smem_sm = 0, smem_rsv = 0, regs_sm = 0;
        cudaFuncAttributes fa;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&clusters, gemm_decode_kernel<BN, EPI, ST>, &occ);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&api_per_sm, gemm_decode_kernel<BN, EPI, ST>, THREADS, C::SMEM_BYTES);
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, gemm_decode_kernel<BN, EPI, ST>);
        if (e == cudaSuccess) e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&smem_rsv, cudaDevAttrReservedSharedMemoryPerBlock, dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&regs_sm, cudaDevAttrMaxRegistersPerMultiprocessor, dev);
        if (e != cudaSuccess) return e;
        const long by_smem = smem_sm / (long)(C::SMEM_BYTES + fa.sharedSizeBytes + smem_rsv);
        const long by_regs = regs_sm / (long)(((fa.numRegs + 7) / 8 * 8) * THREADS);
        long per_sm = by_smem < by_regs ? by_smem : by_regs;
        if (per_sm > 2048 / THREADS) per_sm = 2048 / THREADS;
        if (api_per_sm < 1 || per_sm < api_per_sm) per_sm = api_per_sm < 1 ? 0 : api_per_sm;
        const long capacity = api_per_sm < 1 ? 0 : (long)clusters * per_sm / api_per_sm;
        if ((long)grid.x * grid.y > capacity) return cudaErrorCooperativeLaunchTooLarge;
    }
    return cudaLaunchKernelEx(&cfg, gemm_decode_kernel<BN, EPI, ST>, *tw[0], *tw[1], *tw[2], tt, L);
}

template <int EPI>
cudaError_t launch_epi(const CUtensorMap *const *tw, const CUtensorMap &tt, const DecLaunch &L0, int tiles, cudaStream_t st)
{
    DecLaunch L = L0;
    const int bn = tc_token_box(true, L.g.t_rows);
    const long n_sm = sm_count();
    // Shard slices as planes: one slice per block is the default.  Where that launch would not be resident at once
    // (two blocks per SM with a four-stage ring at 32- and 64-token tiles, three at 16), a block takes two slices one
    // after the other into two accumulators: half the blocks, twice the K blocks each, one wave instead of two.
    L.zs = 1;
    if (L.g.z_is_plane && L.g.splits == 1 && L.g.batches % 2 == 0 && L.g.batches >= 4) {
        const long one_each = (long)tiles * ((L.g.t_rows + bn - 1) / bn) * L.P;
        if (L.g.planes_per_block == 2 || (L.g.planes_per_block == 0 && one_each > (bn == 16 ? 3 : 2) * n_sm)) L.zs = 2;
    }
    dim3 grid(tiles * (L.g.z_is_plane ? 1 : L.g.batches), (L.g.t_rows + bn - 1) / bn, L.P / L.zs);
    // ring depth at 16-token tiles: five stages for launches of at most two blocks per SM (they all stay resident and
    // each block has more in flight), four up to three blocks per SM, three beyond (four blocks per SM keep the
    // launch resident at once); four stages at 32- and 64-token tiles
    const long blocks = (long)grid.x * grid.y * grid.z;
    int stages = L.g.ring_stages;
    if (stages == 0) stages = (bn == 16 && blocks > 3L * n_sm) ? 3 : ((bn == 16 && blocks <= 2L * n_sm) ? 5 : 4);
    // several ranks in one launch wait on one another: as many resident blocks as possible
    if (L.g.ring_stages == 0 && EPI == EPI_RESID_TP && L.g.tp.exchange && L.g.batches > 1) stages = 3;
    switch (bn) {
    case 16:
        if (stages <= 3) return launch_cfg<16, EPI, 3>(tw, tt, L, grid, st);
        if (stages == 4) return launch_cfg<16, EPI, 4>(tw, tt, L, grid, st);
        return launch_cfg<16, EPI, 5>(tw, tt, L, grid, st);
    case 32:
        if (stages <= 3) return launch_cfg<32, EPI, 3>(tw, tt, L, grid, st);
        return launch_cfg<32, EPI, 4>(tw, tt, L, grid, st);
    default:
        if (stages <= 3) return launch_cfg<64, EPI, 3>(tw, tt, L, grid, st);
        return launch_cfg<64, EPI, 4>(tw, tt, L, grid, st);
    }
}

// One thread block per 128 columns, all tokens: the same outputs EPI_DOWN leaves for the next block.
// Rank mode: blockIdx.y = local rank, whose planes lie z_stride bytes apart and whose step number advances here.
__global__ void __launch_bounds__(128) decode_prologue_kernel(PrologueArgs a, int h_tiles, double log_base)
{
    pdl_launch_dependents();
    if (threadIdx.x == 0) stamp_entry(a.stamp);
    pdl_wait();
    if ((int)blockIdx.x >= h_tiles) {
        // rotary table of this step, evaluated in double and shared by all blocks of the stack
        const int half = a.head_dim / 2, i = ((int)blockIdx.x - h_tiles) * 128 + threadIdx.x;
        if (blockIdx.y != 0 || i >= a.M * half) return;
        int m = i / half, j = i % half, b, pos;
        a.tm.locate(m, b, pos);
        const double theta = exp(-2.0 * (double)j / (double)a.head_dim * log_base);
        double sn, cs;
        sincos((double)pos * theta, &sn, &cs);
        a.rope_table[i] = make_float2((float)cs, (float)sn);
        return;
    }
    const long zoff = (long)blockIdx.y * a.z_stride;
    float *res_out = (float *)((char *)a.res_out + zoff), *ss_out = (float *)((char *)a.ss_out + zoff);
    float *sum_out = a.sum_out ? (float *)((char *)a.sum_out + zoff) : nullptr;
    bf16 *hg = (bf16 *)((char *)a.hg + zoff);
    if (a.step && blockIdx.x == 0 && threadIdx.x == 0) *(unsigned *)((char *)a.step + zoff) += 1u;
    // warp w takes tokens w, w+4, ...; lane l the columns 4l .. 4l+3 of the block's 128: no block-wide barrier
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n = blockIdx.x * 128 + 4 * lane;
    const bool valid = n < a.H; // H is a multiple of 4
    float4 gn = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid) {
        const uint2 u = *(const uint2 *)((const bf16 *)a.gain + n);
        const float2 g0 = __bfloat1622float2(*(const __nv_bfloat162 *)&u.x), g1 = __bfloat1622float2(*(const __nv_bfloat162 *)&u.y);
        gn = make_float4(g0.x, g0.y, g1.x, g1.y);
    }
    for (int m = warp; m < a.M; m += 4) {
        const long idx = (long)m * a.H + n;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) {
            const uint2 u = *(const uint2 *)((const bf16 *)a.x + idx);
            const float2 x0 = __bfloat1622float2(*(const __nv_bfloat162 *)&u.x), x1 = __bfloat1622float2(*(const __nv_bfloat162 *)&u.y);
            x = make_float4(x0.x, x0.y, x1.x, x1.y);
            *(float4 *)(res_out + idx) = x;
            store_bf16x4(hg + idx, x, gn);
        }
        const float q = warp_sum(sq4(x));
        if (lane == 0) ss_out[(long)blockIdx.x * a.Mcap + m] = q;
        if (sum_out) {
            const float sm = warp_sum(x.x + x.y + x.z + x.w);
            if (lane == 0) sum_out[(long)blockIdx.x * a.Mcap + m] = sm;
        }
    }
    if (threadIdx.x == 0) stamp_exit(a.stamp);
}

} // namespace

int decode_tiles_per_batch(DecEpilogue epi, const int *w_rows, int n_weights)
{
    if (epi == EPI_GATEUP) return (w_rows[0] + 63) / 64;
    int tiles = 0;
    for (int i = 0; i < n_weights; ++i) tiles += (w_rows[i] + BM - 1) / BM;
    return tiles;
}

cudaError_t launch_gemm_decode(DecEpilogue epi, const TcMap *const *weights, const TcMap &tokens, const DecGemmArgs &g,
                               cudaStream_t st)
{
    const int nw = g.n_weights;
    if (nw < 1 || nw > 3 || (epi == EPI_GATEUP && nw != (g.fc1_only ? 1 : 2))) return cudaErrorInvalidValue;
    if (epi == EPI_GATEUP && g.fc1_only && (!g.ln_wg || !g.ln_wb || g.Fs % 2)) return cudaErrorInvalidValue;
    if (g.t_rows <= 0) return cudaSuccess;
    if (g.splits < 1 || g.splits > g.num_kb || g.n_groups > MAX_GROUPS) return cudaErrorInvalidValue;
    const int P = g.z_is_plane ? g.batches * g.splits : g.splits;
    if (P > MAX_P) return cudaErrorInvalidValue;
    if (epi == EPI_OPROJ && g.n_groups > 1 && (g.n_groups != g.batches || !g.z_is_plane)) return cudaErrorInvalidValue;
    if (epi == EPI_QKV && (BM % g.head_dim) != 0) return cudaErrorInvalidValue;
    if (epi == EPI_RESID_TP && (!g.tp.on || g.z_is_plane || g.tp.T < 1 || g.tp.T > TP_MAX_RANKS || P > TP_FLAG_RANGES ||
                                g.tp.rank_base < 0 || g.tp.rank_base + g.batches > g.tp.T || !g.tp.step || !g.res_in))
        return cudaErrorInvalidValue;
    const CUtensorMap *tw[3];
    for (int i = 0; i < 3; ++i) tw[i] = (const CUtensorMap *)weights[i < nw ? i : 0];
    const CUtensorMap &tt = *(const CUtensorMap *)&tokens;
    DecLaunch L;
    L.g = g;
    int tiles = 0;
    for (int i = 0; i < 3; ++i) {
        L.tile_start[i] = tiles;
        if (i < nw && epi != EPI_GATEUP) {
            if (g.w_rows[i] <= 0) return cudaErrorInvalidValue;
            tiles += (g.w_rows[i] + BM - 1) / BM;
        } else if (i >= nw) {
            L.tile_start[i] = 1 << 30; // never selected
        }
    }
    if (epi == EPI_GATEUP) {
        tiles = g.fc1_only ? (g.w_rows[0] + BM - 1) / BM : (g.w_rows[0] + 63) / 64;
        L.tile_start[0] = 0;
        L.tile_start[1] = L.tile_start[2] = 1 << 30;
    }
    L.w_tiles_per_batch = tiles;
    L.P = P;
    L.zs = 1;
    switch (epi) {
    case EPI_QKV: return launch_epi<EPI_QKV>(tw, tt, L, tiles, st);
    case EPI_OPROJ: return launch_epi<EPI_OPROJ>(tw, tt, L, tiles, st);
    case EPI_GATEUP: return launch_epi<EPI_GATEUP>(tw, tt, L, tiles, st);
    case EPI_RESID_TP: return launch_epi<EPI_RESID_TP>(tw, tt, L, tiles, st);
    default: return launch_epi<EPI_DOWN>(tw, tt, L, tiles, st);
    }
}

cudaError_t launch_decode_prologue(const PrologueArgs &a, cudaStream_t st)
{
    if (a.M <= 0) return cudaSuccess;
    const int h_tiles = (a.H + 127) / 128;
    const int table_blocks = a.rope_table ? (a.M * (a.head_dim / 2) + 127) / 128 : 0;
    return launch_kernel(decode_prologue_kernel, dim3(h_tiles + table_blocks, a.n_z > 1 ? a.n_z : 1), dim3(128), 0, st, 0, a, h_tiles,
                         a.rope_table ? log((double)a.rope_base) : 0.0);
}

} // namespace spd
