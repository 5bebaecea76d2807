// Fused prefill projections.  With thousands of tokens in flight the projections are bound by
// the tensor cores, so each is one persistent tcgen05 GEMM: one thread block per SM walks the
// output tiles (128 tokens x 256 weight rows), a TMA warp keeps a shared-memory ring of
// K blocks full, an MMA warp accumulates into one of two tensor-memory buffers, and the four
// epilogue warps drain the other buffer meanwhile - applying the step that follows the
// projection to the fp32 accumulator (thread = token row), so nothing but the next operand
// (bf16) and the fp32 residual stream goes to memory.
//
//   PRE_QKV       : attention-RMSNorm rstd, rotary embedding, q store, K/V page append   (a2, a3)
//   PRE_RESID     : sync block o_proj (R = X + sum_i Y_i as ONE GEMM over all of K) and down
//                   (sum_i Z_i likewise): residual add, gain-scaled next operand, sums of squares
//   PRE_GATEUP    : MLP-RMSNorm rstd (per emulated device in an SPD block), SwiGLU       (a8)
//   PRE_OPROJ_SPD : SPD block (Sec. 4.1.1): the T K-slices of a 128 x 128 output tile in turn;
//                   device i's pass gives Y_i, from which R_i = X + Y_i (its own MLP input) is
//                   stored, while a third tensor-memory buffer adds up sum_i Y_i for the
//                   residual that is carried to the block output.
// Launches with more than 128 tokens run on pairs of thread blocks (cta_group::2): one 256-token tile
// and one M = 256 instruction over two SMs, each block loading its own token rows and half of the
// tile's weight rows.  The operand ring takes all of a block's shared memory: tile loads have a
// loaded latency of about 1.6 us, so bytes in flight are what bounds the feed of the tensor cores.
#include "gemm_prefill.cuh"
#include "tc_ptx.cuh"
#include "trace.cuh"

namespace spd {

namespace {

using namespace tc;

constexpr int TMEM_ALL = 512;
constexpr int X_COL = 256;   // PRE_OPROJ_SPD: the X tile (columns 0-255 hold the two accumulators)

// PAIR: two CTAs of a cluster work on one tile of 256 tokens as one M = 256 MMA (cta_group::2): each loads its own
// 128 token rows and HALF of the tile's weight rows, so per MMA flop only two thirds (three quarters for the SPD
// o_proj) of the operand bytes cross from L2 into shared memory, and the ring holds more K blocks.
template <int EPI, int PAIR> struct PCfg {
    static constexpr int BN = (EPI == PRE_OPROJ_SPD) ? 128 : 256;
    static_assert(EPI != PRE_SCATTER || PAIR, "the scatter epilogue is only built for CTA pairs");
    static constexpr int A_BYTES = BM * BK * 2, B_BYTES = (BN / (PAIR ? 2 : 1)) * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    // the ring takes all the shared memory a block may have: the loaded latency of a tile load is about 1.6 us, so
    // what the tensor cores can be fed per SM is (bytes in flight) / 1.6 us
    static constexpr int STAGES = (216 * 1024) / STAGE_BYTES;
    static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
    static constexpr int SMEM_BYTES = RING_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
    // Epilogue warps: 0-3 (one per accumulator lane quarter); PRE_OPROJ_SPD, whose tail is T times the work per MMA
    // of the others, adds warps 6-9: two threads per row, 64 of the tile's 128 columns each.
    static constexpr int EPI_WARPS = (EPI == PRE_OPROJ_SPD) ? 8 : 4;
    static constexpr int THREADS_ = 64 + 32 * EPI_WARPS;
};

struct PreLaunch {
    PreGemmArgs g;
    int m_tiles, n_tiles, passes; // m_tiles: token tiles of 128 rows, or of 256 for a CTA pair
    int group_m;                  // token tiles per group of the tile order (see decode_tile)
    int tile_start[3]; // QKV: first n-tile of weight i
    int f_tiles;       // GATEUP: n-tiles per device
};

struct PreTile {
    int m0;     // first token
    int wi;     // QKV: which weight
    int row0;   // first weight row (QKV, RESID, OPROJ_SPD: output column; GATEUP: FFN column within the device)
    int z;      // GATEUP: device
    int nt;     // n-tile index (for the sums of squares)
};

__device__ __forceinline__ PreTile decode_tile(const PreLaunch &L, int EPI, int tile, int pair, int crank)
{
    PreTile t;
    // Tile order: groups of group_m token tiles; inside a group the token tile runs fastest, then the weight tile.
    // The blocks at work at any time then cover about group_m token tiles x (blocks / group_m) weight tiles - a
    // near-square patch, whose operand panels are fetched from HBM once and shared through L2 - and a group's
    // token panels stay in L2 for the whole sweep over the weight tiles, instead of being streamed again for
    // every few weight tiles as they are when ALL token tiles run fastest (they do not fit L2 at thousands of tokens).
    const int per_group = L.group_m * L.n_tiles, grp = tile / per_group, r = tile % per_group;
    const int gm = min(L.group_m, L.m_tiles - grp * L.group_m);
    const int mt = grp * L.group_m + r % gm, nt = r / gm;
    t.m0 = pair ? mt * 2 * BM + crank * BM : mt * BM; // this CTA's 128 token rows
    t.nt = nt;
    t.wi = 0;
    t.z = 0;
    if (EPI == PRE_QKV) {
        t.wi = nt >= L.tile_start[2] ? 2 : (nt >= L.tile_start[1] ? 1 : 0);
        t.row0 = (nt - L.tile_start[t.wi]) * 256;
    } else if (EPI == PRE_GATEUP) {
        t.z = nt / L.f_tiles;
        t.row0 = (nt % L.f_tiles) * (L.g.fc1_only ? 256 : 128);
    } else if (EPI == PRE_OPROJ_SPD) {
        t.row0 = nt * 128;
    } else {
        t.row0 = nt * 256;
    }
    return t;
}

// two 16-column accumulator chunks of this thread's row, one wait
__device__ __forceinline__ void tmem_ld16x2(uint32_t ta, uint32_t tb, float *va, float *vb)
{
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%32];\n\t"
                 "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%33];\n\t"
                 "tcgen05.wait::ld.sync.aligned;"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(ta), "r"(tb)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) { va[i] = __uint_as_float(r[i]); vb[i] = __uint_as_float(r[16 + i]); }
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float *v)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
                   "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
                   "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
                   "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
                   "r"(__float_as_uint(v[15]))
                 : "memory");
}

// two 32-column chunks of this thread's row, one wait
__device__ __forceinline__ void tmem_ld32x2(uint32_t ta, uint32_t tb, float *va, float *vb)
{
    uint32_t r[64];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%64];\n\t"
                 "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%65];\n\t"
                 "tcgen05.wait::ld.sync.aligned;"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
                 : "r"(ta), "r"(tb)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) { va[i] = __uint_as_float(r[i]); vb[i] = __uint_as_float(r[32 + i]); }
}
// 8 consecutive bf16 (16 bytes) from 8 floats
__device__ __forceinline__ uint4 pack8(const float *v)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
    return make_uint4(*(uint32_t *)&a, *(uint32_t *)&b, *(uint32_t *)&c, *(uint32_t *)&d);
}
__device__ __forceinline__ void unpack8(uint4 u, float *v)
{
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}

// 32-byte global accesses (one row piece per thread: half as many instructions, whole 32-byte sectors)
__device__ __forceinline__ void ldg8(const float *p, float *v)
{
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]) : "l"(p) : "memory");
}
__device__ __forceinline__ void stg8(float *p, const float *v)
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
}
// 16 consecutive bf16 (32 bytes, 32-byte aligned) from 16 floats
__device__ __forceinline__ void stg16_bf16(bf16 *p, const float *v)
{
    const uint4 a = pack8(v), b = pack8(v + 8);
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

// rstd of a token row from the partial sums of squares (RMSNorm); with partial sums as well (LayerNorm) also the mean
__device__ __forceinline__ float row_rstd(const SumSq &s, int group, int m, float &mu)
{
    float acc = 0.f, sum = 0.f;
    for (int t = 0; t < s.tiles; ++t) {
        const long i = ((long)t * s.groups + group) * s.Mcap + m;
        acc += s.part[i];
        if (s.sum) sum += s.sum[i];
    }
    mu = sum / (float)s.H;
    return s.sum ? rsqrtf(fmaxf(acc / (float)s.H - mu * mu, 0.f) + s.eps) : rsqrtf(acc / (float)s.H + s.eps);
}

// ---- epilogues: thread = token row m, columns read from tensor memory 16 at a time ----------------

__device__ __forceinline__ void epi_qkv(const PreGemmArgs &g, const PreTile &t, uint32_t tacc, int m, bool valid)
{
    const int d = g.head_dim, half = d >> 1, nq = g.n_q_heads;
    float mu = 0.f;
    const float rs = valid ? row_rstd(g.ss_in, 0, m, mu) : 0.f;
    const bool rot = t.wi < 2 && g.rope != nullptr;
    // block with bias: first entry of this weight in the folded-LayerNorm vectors (rows of q, k, v one after the other)
    const int vbase = t.wi == 0 ? 0 : (t.wi == 1 ? g.w_rows[0] : g.w_rows[0] + g.w_rows[1]);
    long kv_off = -1;
    if (t.wi > 0 && valid) {
        int b, pos;
        g.tm.locate(m, b, pos);
        const int pi = pos / g.pt.block;
        if (pos < 0 || pi >= g.pt.max_pages) atomicOr(g.err, ERR_CAPACITY);
        else {
            const int page = g.pt.block_table[(long)b * g.pt.max_pages + pi];
            if (page < 0 || page >= g.pt.n_pages) atomicOr(g.err, ERR_PAGE_RANGE);
            else kv_off = ((long)page * g.pt.n_kv_heads * g.pt.block + pos % g.pt.block) * d;
        }
    }
    const int heads = 256 / d;
    for (int hh = 0; hh < heads; ++hh) {
        const int row_h = t.row0 + hh * d;
        if (row_h >= g.w_rows[t.wi]) break;
        const int head = row_h / d + (t.wi == 0 ? g.q_head0 : g.kv_head0);
        bf16 *dst = nullptr;
        if (valid) {
            if (t.wi == 0) dst = (bf16 *)g.q_out + ((long)m * nq + head) * d;
            else if (kv_off >= 0) dst = (bf16 *)(t.wi == 1 ? g.k_pages : g.v_pages) + kv_off + (long)head * g.pt.block * d;
        }
        for (int j0 = 0; j0 < half; j0 += 16) {
            float lo[16], hi[16];
            tmem_ld16x2(tacc + hh * d + j0, tacc + hh * d + half + j0, lo, hi);
            if (!dst) continue;
            float olo[16], ohi[16];
            if (rot) {
                const float4 *cs = (const float4 *)(g.rope + (long)m * half + j0);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 c2 = cs[i]; // cos, sin of two consecutive dims
                    const float a0 = lo[2 * i] * rs, b0 = hi[2 * i] * rs, a1 = lo[2 * i + 1] * rs, b1 = hi[2 * i + 1] * rs;
                    olo[2 * i] = a0 * c2.x - b0 * c2.y;
                    ohi[2 * i] = b0 * c2.x + a0 * c2.y;
                    olo[2 * i + 1] = a1 * c2.z - b1 * c2.w;
                    ohi[2 * i + 1] = b1 * c2.z + a1 * c2.w;
                }
            } else if (g.ln_wg) {
                const float *wgl = g.ln_wg + vbase + row_h + j0, *wbl = g.ln_wb + vbase + row_h + j0;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    olo[i] = (lo[i] - mu * wgl[i]) * rs + wbl[i];
                    ohi[i] = (hi[i] - mu * wgl[half + i]) * rs + wbl[half + i];
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) { olo[i] = lo[i] * rs; ohi[i] = hi[i] * rs; }
            }
            stg16_bf16(dst + j0, olo);
            stg16_bf16(dst + half + j0, ohi);
        }
    }
}

__device__ __forceinline__ void epi_gateup(const PreGemmArgs &g, const PreTile &t, uint32_t tacc, int m, bool valid)
{
    float mu = 0.f;
    const float rs = valid ? row_rstd(g.ss_in, g.rstd_per_shard ? t.z : 0, m, mu) : 0.f;
    bf16 *dst = (bf16 *)g.act + (long)m * g.F + g.act_col0 + (long)((t.z + g.w_rot) % g.batches) * g.Fs + t.row0;
    if (g.fc1_only) {
        // block with bias: the tile's 256 columns are 256 consecutive rows of fc1; LayerNorm folded in, bias, ReLU
        const float *wgl = g.ln_wg + (long)t.z * g.Fs + t.row0, *wbl = g.ln_wb + (long)t.z * g.Fs + t.row0;
#pragma unroll 1
        for (int c = 0; c < 16; c += 2) {
            const int f = t.row0 + c * 16;
            if (f >= g.Fs) break;
            float a[16], b[16], o[16];
            tmem_ld16x2(tacc + c * 16, tacc + c * 16 + 16, a, b);
            if (!valid) continue;
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] = fmaxf((a[i] - mu * wgl[c * 16 + i]) * rs + wbl[c * 16 + i], 0.f);
            *(uint4 *)(dst + c * 16) = pack8(o);
            if (f + 8 < g.Fs) *(uint4 *)(dst + c * 16 + 8) = pack8(o + 8);
            if (f + 16 < g.Fs) {
#pragma unroll
                for (int i = 0; i < 16; ++i) o[i] = fmaxf((b[i] - mu * wgl[c * 16 + 16 + i]) * rs + wbl[c * 16 + 16 + i], 0.f);
                *(uint4 *)(dst + c * 16 + 16) = pack8(o);
                if (f + 24 < g.Fs) *(uint4 *)(dst + c * 16 + 24) = pack8(o + 8);
            }
        }
        return;
    }
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
        const int f = t.row0 + c * 16;
        if (f >= g.Fs) break;
        float gt[16], up[16], o[16];
        tmem_ld16x2(tacc + c * 16, tacc + 128 + c * 16, gt, up);
        if (!valid) continue;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float x = gt[i] * rs;
            o[i] = x / (1.f + __expf(-x)) * (up[i] * rs);
        }
        *(uint4 *)(dst + c * 16) = pack8(o);
        if (f + 8 < g.Fs) *(uint4 *)(dst + c * 16 + 8) = pack8(o + 8);
    }
}

// y: 16 accumulator columns at output column n.  r = x + y; stores what the arguments ask for.
__device__ __forceinline__ float resid_chunk(const PreGemmArgs &g, long idx, int n, const float *x, const float *y, bf16 *hg,
                                             bool store_res, float &sum)
{
    float r[16], sq = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) { r[i] = x[i] + y[i]; sq = fmaf(r[i], r[i], sq); sum += r[i]; }
    if (store_res) {
        if (g.res_out) { stg8(g.res_out + idx, r); stg8(g.res_out + idx + 8, r + 8); }
        if (g.final_out) stg16_bf16((bf16 *)g.final_out + idx, r);
    }
    if (hg) {
        float gn[16];
        unpack8(*(const uint4 *)((const bf16 *)g.gain + n), gn);
        unpack8(*(const uint4 *)((const bf16 *)g.gain + n + 8), gn + 8);
#pragma unroll
        for (int i = 0; i < 16; ++i) gn[i] *= r[i];
        stg16_bf16(hg + idx, gn);
    }
    return sq;
}

__device__ __forceinline__ void load_x16(const float *p, float *x)
{
    ldg8(p, x);
    ldg8(p + 8, x + 8);
}
// x += bias[n .. n+16) (bf16), the bias of a row-split layer of the block with bias
__device__ __forceinline__ void add_bias16(const void *bias, int n, float *x)
{
    if (!bias) return;
    float b[16];
    unpack8(*(const uint4 *)((const bf16 *)bias + n), b);
    unpack8(*(const uint4 *)((const bf16 *)bias + n + 8), b + 8);
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] += b[i];
}

__device__ __forceinline__ void epi_resid(const PreGemmArgs &g, const PreTile &t, uint32_t tacc, int m, bool valid)
{
    float ssq = 0.f, sum = 0.f;
#pragma unroll 1
    for (int c = 0; c < 16; c += 2) {
        const int n = t.row0 + c * 16;
        if (n >= g.H) break;
        float ya[16], yb[16];
        tmem_ld16x2(tacc + c * 16, tacc + c * 16 + 16, ya, yb);
        if (!valid) continue;
        const long idx = (long)m * g.H + n;
        float x[16];
        load_x16(g.res_in + idx, x);
        add_bias16(g.bias, n, x);
        if (g.ysave) { stg8(g.ysave + idx, ya); stg8(g.ysave + idx + 8, ya + 8); }
        ssq += resid_chunk(g, idx, n, x, ya, g.hg ? (bf16 *)g.hg : nullptr, true, sum);
        if (n + 16 < g.H) {
            load_x16(g.res_in + idx + 16, x);
            add_bias16(g.bias, n + 16, x);
            if (g.ysave) { stg8(g.ysave + idx + 16, yb); stg8(g.ysave + idx + 24, yb + 8); }
            ssq += resid_chunk(g, idx + 16, n + 16, x, yb, g.hg ? (bf16 *)g.hg : nullptr, true, sum);
        }
    }
    if (valid && g.ss_out) g.ss_out[(long)t.nt * g.Mcap + m] = ssq;
    if (valid && g.sum_out) g.sum_out[(long)t.nt * g.Mcap + m] = sum;
}

// Rank mode, shot one of a two-shot exchange (see TpScatter): this block's 128 partial rows go to the rank that owns
// the tile, then the step number is published in the owner's flag word for (slot, column tile, this rank).
__device__ __forceinline__ void epi_scatter(const PreGemmArgs &g, const PreTile &t, uint32_t tacc, int m, bool valid, int r)
{
    const TpScatter &sc = g.sc;
    const int tile128 = t.m0 / BM, owner = tile128 % sc.T, slot = tile128 / sc.T;
    float *dst = (float *)(sc.rx[owner] + (long)sc.me * sc.src_stride) + ((long)slot * BM + r) * g.H;
#pragma unroll 1
    for (int c = 0; c < 16; c += 2) {
        const int n = t.row0 + c * 16;
        if (n >= g.H) break;
        float ya[16], yb[16];
        tmem_ld16x2(tacc + c * 16, tacc + c * 16 + 16, ya, yb);
        if (!valid) continue;
        if (sc.addend) {
            float a[16];
            load_x16(sc.addend + (long)m * g.H + n, a);
#pragma unroll
            for (int i = 0; i < 16; ++i) ya[i] += a[i];
        }
        stg8(dst + n, ya);
        stg8(dst + n + 8, ya + 8);
        if (n + 16 < g.H) {
            if (sc.addend) {
                float a[16];
                load_x16(sc.addend + (long)m * g.H + n + 16, a);
#pragma unroll
                for (int i = 0; i < 16; ++i) yb[i] += a[i];
            }
            stg8(dst + n + 16, yb);
            stg8(dst + n + 24, yb + 8);
        }
    }
}

template <int N_THREADS> __device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(N_THREADS) : "memory"); }

// SPD o_proj: the X tile of an output tile is parked in tensor memory (every device's R_i = X + Y_i needs it) by
// the thread that owns the row, while the MMA warp works on the first K slice; the same thread starts its running
// X + sum_i Y_i - 64 columns, kept in registers across the passes - from it.  (Tensor memory serves the MMAs'
// accumulator traffic and the epilogue's loads and stores alike: with a K slice of only a few hundred per pass the
// epilogue's share decides the MMA rate, so the running sum stays out of it.)
__device__ __forceinline__ void spd_park_x(const PreGemmArgs &g, const PreTile &t, uint32_t tx, int m, bool valid, int half, float (&tot)[64])
{
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
        const int c = half * 4 + cc, n = t.row0 + c * 16;
        float x[16];
        if (valid && n < g.H) {
            load_x16(g.res_in + (long)m * g.H + n, x);
            add_bias16(g.bias, n, x); // block with bias: b joins X once - and so every device's X + P_i + b and the carried sum
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) x[i] = 0.f;
        }
        tmem_st16(tx + c * 16, x);
#pragma unroll
        for (int i = 0; i < 16; ++i) tot[cc * 16 + i] = x[i];
    }
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Sum of squares of this row's 128 accumulator columns (MLP matching: norm of a partition's output).
__device__ __forceinline__ float epi_row_sumsq(const PreGemmArgs &g, const PreTile &t, uint32_t tacc, int half)
{
    float ssq = 0.f;
#pragma unroll 1
    for (int c = half * 4; c < half * 4 + 4; c += 2) {
        const int n = t.row0 + c * 16;
        if (n >= g.H) break;
        float ya[16], yb[16];
        tmem_ld16x2(tacc + c * 16, tacc + c * 16 + 16, ya, yb);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            ssq = fmaf(ya[i], ya[i], ssq);
            if (n + 16 < g.H) ssq = fmaf(yb[i], yb[i], ssq);
        }
    }
    return ssq;
}

// One pass (device z) of an SPD o_proj tile: R_z * g goes straight from the thread's registers to device z's
// plane (32-byte stores, whole sectors; shared memory is left to the operand ring); X + sum_i Y_i, carried in
// tot, is written by the last pass.
__device__ __forceinline__ float epi_oproj_spd(const PreGemmArgs &g, const PreTile &t, uint32_t tacc, uint32_t tx, int z,
                                               int m, bool valid, int half, float (&tot)[64], float &sum)
{
    const int T = g.batches;
    float ssq = 0.f;
    bf16 *plane = (bf16 *)g.hg + (long)z * g.hg_stride + (long)m * g.H;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) { // 32 columns per round: few tensor-memory round trips on the critical path
        const int c = half * 2 + cc, n = t.row0 + c * 32;
        float y[32], x[32];
        tmem_ld32x2(tacc + c * 32, tx + c * 32, y, x);
#pragma unroll
        for (int i = 0; i < 32; ++i) tot[cc * 32 + i] += y[i];
        // device z only ever sees its own partial attention output: R_z = X + Y_z
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            if (!valid || n + 16 * q >= g.H) continue; // a tile may reach past the last column (H is a multiple of 16)
            float gn[16];
            unpack8(*(const uint4 *)((const bf16 *)g.gain + n + 16 * q), gn);
            unpack8(*(const uint4 *)((const bf16 *)g.gain + n + 16 * q + 8), gn + 8);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float ri = x[16 * q + i] + y[16 * q + i];
                ssq = fmaf(ri, ri, ssq);
                sum += ri;
                gn[i] *= ri;
            }
            stg16_bf16(plane + n + 16 * q, gn);
        }
        if (z + 1 == T && valid) {
            // the residual carried to the block output has collected every Y_i
            float *dst = g.res_out + (long)m * g.H + n;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (n + 8 * k < g.H) stg8(dst + 8 * k, &tot[cc * 32 + 8 * k]);
        }
    }
    return ssq;
}

template <int EPI, int PAIR>
__global__ void __launch_bounds__(PCfg<EPI, PAIR>::THREADS_, 1) gemm_prefill_kernel(const __grid_constant__ CUtensorMap tm_w0,
                                                                  const __grid_constant__ CUtensorMap tm_w1,
                                                                  const __grid_constant__ CUtensorMap tm_w2,
                                                                  const __grid_constant__ CUtensorMap tm_t,
                                                                  const __grid_constant__ PreLaunch L)
{
    using C = PCfg<EPI, PAIR>;
    constexpr int BN = C::BN, S = C::STAGES;
    const PreGemmArgs &g = L.g;
    // a pair's leader (even cluster rank) issues the MMAs for both CTAs and owns the barriers they are counted on
    const int crank = PAIR ? (int)cluster_ctarank() : 0;
    const bool leader = crank == 0;
    const int tile0 = PAIR ? (int)blockIdx.x / 2 : (int)blockIdx.x, tile_step = PAIR ? (int)gridDim.x / 2 : (int)gridDim.x;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + C::RING_BYTES; // full[S], empty[S], tmem_full[2], tmem_empty[2]
    uint32_t *tmem_slot = (uint32_t *)(gen_base + C::RING_BYTES + 8 * (2 * S + 4));
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (S + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * S + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * S + 2 + b); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = L.m_tiles * L.n_tiles;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        stamp_entry(g.stamp);
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        // an accumulator is free again when the epilogue warps of both CTAs of a pair have drained their rows
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), C::EPI_WARPS * (PAIR ? 2 : 1)); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        if (PAIR) { // one allocation over the tensor memory of both CTAs, made by the same warp of each
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_ALL) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_ALL) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (PAIR) cluster_sync(); // the partner's barriers are initialised before anything of ours can reach them
    else __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    if (warp == 4) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w0) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_t) : "memory");
            const uint64_t keep = policy_evict_normal();
            uint32_t it = 0;
            bool ok = true;
            for (int tile = tile0; tile < total_tiles && ok; tile += tile_step) {
                const PreTile t = decode_tile(L, EPI, tile, PAIR, crank);
                const CUtensorMap *tm_w = t.wi == 0 ? &tm_w0 : (t.wi == 1 ? &tm_w1 : &tm_w2);
                for (int pass = 0; pass < L.passes && ok; ++pass) {
                    const int tz = g.t_z + (EPI == PRE_OPROJ_SPD ? pass : (EPI == PRE_GATEUP && g.t_batched ? t.z : 0));
                    const int wz = g.w_z + (EPI == PRE_OPROJ_SPD ? pass : (EPI == PRE_GATEUP ? (t.z + g.w_rot) % g.batches : t.z));
                    for (int kb = 0; kb < g.num_kb; ++kb, ++it) {
                        const int s = it % S;
                        if (!mbar_wait(empty_bar(s), ((it / S) & 1) ^ 1, g.err, abort_flag)) { ok = false; break; }
                        const uint32_t sa = base + s * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                        if (PAIR) {
                            // both CTAs' bytes of this stage are counted on the leader's barrier, which the MMA thread waits on
                            if (leader) mbar_expect_tx(full_bar(s), 2 * C::STAGE_BYTES);
                            const uint32_t fb = mapa_shared(full_bar(s), 0);
                            tma_load_3d_pair(sa, &tm_t, kb * BK, t.m0, tz, fb, keep);
                            // this CTA's half of the tile's weight rows (GATEUP: the leader holds the gate rows, its partner the up rows)
                            if (EPI == PRE_GATEUP && g.fc1_only) tma_load_3d_pair(sb, &tm_w0, kb * BK, t.row0 + crank * 128, wz, fb, keep);
                            else if (EPI == PRE_GATEUP) tma_load_3d_pair(sb, leader ? &tm_w0 : &tm_w1, kb * BK, t.row0, wz, fb, keep);
                            else tma_load_3d_pair(sb, tm_w, kb * BK, t.row0 + crank * (BN / 2), wz, fb, keep);
                        } else {
                            mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
                            tma_load_3d(sa, &tm_t, kb * BK, t.m0, tz, full_bar(s));
                            if (EPI == PRE_GATEUP) {
                                tma_load_3d(sb, &tm_w0, kb * BK, t.row0, wz, full_bar(s));
                                if (g.fc1_only) tma_load_3d(sb + 128 * BK * 2, &tm_w0, kb * BK, t.row0 + 128, wz, full_bar(s));
                                else tma_load_3d(sb + 128 * BK * 2, &tm_w1, kb * BK, t.row0, wz, full_bar(s));
                            } else {
                                tma_load_3d(sb, tm_w, kb * BK, t.row0, wz, full_bar(s));
                            }
                        }
                    }
                }
            }
            // A pair member must not leave while the leader's last commits are still on their way to its barriers:
            // wait (bounded) until every stage it filled has been released.
            if (PAIR)
                for (uint32_t j = it; j < it + S && ok; ++j)
                    if (j >= (uint32_t)S && !mbar_wait(empty_bar(j % S), ((j / S) & 1) ^ 1, g.err, abort_flag)) ok = false;
        }
        __syncwarp();
    } else if (warp == 5) {
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = make_idesc(BN, PAIR ? 2 * BM : BM);
            uint32_t it = 0, pc = 0;
            bool ok = true;
            for (int tile = tile0; tile < total_tiles && ok; tile += tile_step) {
                for (int pass = 0; pass < L.passes && ok; ++pass, ++pc) {
                    const int buf = pc & 1;
                    SPD_TRACE_EVENT(TRK_PREFILL + 8 + EPI, TR_START);
                    if (!mbar_wait(tempty_bar(buf), ((pc >> 1) & 1) ^ 1, g.err, abort_flag)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    SPD_TRACE_EVENT(TRK_PREFILL + 8 + EPI, TR_DEP_DONE);
                    const uint32_t tacc = tmem_base + (uint32_t)(buf * BN);
                    for (int kb = 0; kb < g.num_kb; ++kb, ++it) {
                        const int s = it % S;
                        if (kb == 0 || kb == g.num_kb - 1) SPD_TRACE_EVENT(TRK_PREFILL + 8 + EPI, TR_ARRIVED);
                        if (!mbar_wait(full_bar(s), (it / S) & 1, g.err, abort_flag)) { ok = false; break; }
                        if (kb == 0 || kb == g.num_kb - 1) SPD_TRACE_EVENT(TRK_PREFILL + 8 + EPI, TR_MAIN_DONE);
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t sa = base + s * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                        const uint64_t da = make_desc(sa), db = make_desc(sb);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            if (PAIR) umma_pair(tacc, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                                                (kb > 0 || k > 0) ? 1u : 0u);
                            else umma(tacc, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                                      (kb > 0 || k > 0) ? 1u : 0u);
                        }
                        // the stage is free in both CTAs once these MMAs have read it
                        if (PAIR) umma_commit_pair(empty_bar(s));
                        else umma_commit(empty_bar(s));
                    }
                    if (ok) {
                        if (PAIR) umma_commit_pair(tfull_bar(buf));
                        else umma_commit(tfull_bar(buf));
                    }
                    SPD_TRACE_EVENT(TRK_PREFILL + 8 + EPI, TR_END);
                }
            }
        }
        __syncwarp();
    } else {
        uint32_t pc = 0, tile_cnt = 0;
        bool ok = true;
        float tot[64]; // PRE_OPROJ_SPD only: this thread's 64 columns of X + sum_i Y_i (optimised away elsewhere)
        // accumulator lane quarter of this warp (a warp reaches lanes 32 * (warp % 4) ..), and which half of the
        // columns it finishes when two warps share a quarter
        const int quarter = warp & 3, half = warp >= 6 ? 1 : 0;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t tempty_leader0 = PAIR ? mapa_shared(tempty_bar(0), 0) : 0, tempty_leader1 = PAIR ? mapa_shared(tempty_bar(1), 0) : 0;
        for (int tile = tile0; tile < total_tiles && ok; tile += tile_step, ++tile_cnt) {
            const PreTile t = decode_tile(L, EPI, tile, PAIR, crank);
            const int m = t.m0 + quarter * 32 + lane;
            const bool valid = m < g.t_rows;
            if (EPI == PRE_OPROJ_SPD && !g.norm_only) spd_park_x(g, t, tmem_base + lane_base + X_COL, m, valid, half, tot);
            for (int pass = 0; pass < L.passes; ++pass, ++pc) {
                const int buf = pc & 1;
                if (!mbar_wait(tfull_bar(buf), (pc >> 1) & 1, g.err, abort_flag)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_PREFILL + EPI, TR_START);
                const uint32_t tacc = tmem_base + lane_base + (uint32_t)(buf * BN);
                if (EPI == PRE_QKV) epi_qkv(g, t, tacc, m, valid);
                else if (EPI == PRE_GATEUP) epi_gateup(g, t, tacc, m, valid);
                else if (EPI == PRE_RESID) epi_resid(g, t, tacc, m, valid);
                else if (EPI == PRE_SCATTER) {
                    epi_scatter(g, t, tacc, m, valid, quarter * 32 + lane);
                    // every row of the tile is on its way: the release below orders them (made visible to the
                    // publishing thread by the barrier) before the flag
                    epi_sync<32 * C::EPI_WARPS>();
                    if (threadIdx.x == 0 && t.m0 < g.t_rows) { // (a pair's second block may lie wholly past the last token: nobody owns that tile)
                        const int tile128 = t.m0 / BM, owner = tile128 % g.sc.T, slot = tile128 / g.sc.T;
                        unsigned *flag = g.sc.flags[owner] + ((long)slot * g.sc.n_tiles + t.nt) * g.sc.T + g.sc.me;
                        asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(flag), "r"(*g.sc.step) : "memory");
                    }
                }
                else if (g.norm_only) {
                    const float ssq = epi_row_sumsq(g, t, tacc, half);
                    if (valid) g.ss_out[((long)(t.nt * 2 + half) * g.batches + pass) * g.Mcap + m] = ssq;
                } else {
                    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_PREFILL + EPI, TR_DEP_DONE);
                    float sum = 0.f;
                    const float ssq = epi_oproj_spd(g, t, tacc, tmem_base + lane_base + X_COL, pass, m, valid, half, tot, sum);
                    if (valid && g.ss_out) g.ss_out[((long)(t.nt * 2 + half) * g.batches + pass) * g.Mcap + m] = ssq;
                    if (valid && g.sum_out) g.sum_out[((long)(t.nt * 2 + half) * g.batches + pass) * g.Mcap + m] = sum;
                    if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_PREFILL + EPI, TR_MAIN_DONE);
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) mbar_arrive_cluster(buf ? tempty_leader1 : tempty_leader0); // the leader's MMA thread waits for both CTAs' warps
                    else asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tempty_bar(buf)) : "memory");
                }
                if (threadIdx.x == 0) SPD_TRACE_EVENT(TRK_PREFILL + EPI, TR_END);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    // a pair ends together: neither CTA's shared or tensor memory may go while the partner's MMAs or arrivals can reach it
    if (PAIR) cluster_sync();
    else __syncthreads();
    if (threadIdx.x == 0) stamp_exit(g.stamp);
    if (warp == 5) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_ALL) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_ALL) : "memory");
    }
}

template <int EPI, int PAIR>
cudaError_t launch_epi(const CUtensorMap *const *tw, const CUtensorMap &tt, const PreLaunch &L, cudaStream_t st)
{
    using C = PCfg<EPI, PAIR>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemm_prefill_kernel<EPI, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    const int n_sm = sm_count();
    const int total = L.m_tiles * L.n_tiles;
    if (PAIR) { // one pair per two SMs, persistent over the 256-token tiles
        const int pairs = total < n_sm / 2 ? total : n_sm / 2;
        return launch_kernel(gemm_prefill_kernel<EPI, PAIR>, dim3(2 * pairs), dim3(C::THREADS_), C::SMEM_BYTES, st, 2, *tw[0], *tw[1], *tw[2], tt, L);
    }
    const dim3 grid(total < n_sm ? total : n_sm);
    return launch_kernel(gemm_prefill_kernel<EPI, PAIR>, grid, dim3(C::THREADS_), C::SMEM_BYTES, st, 0, *tw[0], *tw[1], *tw[2], tt, L);
}

// One thread block per token: whole-row sum of squares in one partial.
__global__ void __launch_bounds__(256) prefill_prologue_kernel(PrologueArgs a)
{
    pdl_launch_dependents();
    if (threadIdx.x == 0) stamp_entry(a.stamp);
    pdl_wait();
    if (a.step && blockIdx.x == 0 && threadIdx.x == 0) *a.step += 1u; // rank mode: the rank's step number advances with every launch sequence
    __shared__ float red[8];
    const int m = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float sq = 0.f, sum = 0.f;
    for (int n = threadIdx.x * 8; n < a.H; n += blockDim.x * 8) {
        const long idx = (long)m * a.H + n;
        float x[8], gn[8];
        unpack8(*(const uint4 *)((const bf16 *)a.x + idx), x);
        unpack8(*(const uint4 *)((const bf16 *)a.gain + n), gn);
#pragma unroll
        for (int i = 0; i < 8; ++i) { sq = fmaf(x[i], x[i], sq); sum += x[i]; gn[i] *= x[i]; }
        *(float4 *)(a.res_out + idx) = make_float4(x[0], x[1], x[2], x[3]);
        *(float4 *)(a.res_out + idx + 4) = make_float4(x[4], x[5], x[6], x[7]);
        *(uint4 *)((bf16 *)a.hg + idx) = pack8(gn);
    }
    sq = warp_sum(sq);
    sum = warp_sum(sum);
    __shared__ float red_sum[8];
    if (lane == 0) { red[warp] = sq; red_sum[warp] = sum; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f, tsum = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { tot += red[w]; tsum += red_sum[w]; }
        a.ss_out[m] = tot;
        if (a.sum_out) a.sum_out[m] = tsum;
        stamp_exit(a.stamp);
    }
}

} // namespace

// (PRE_OPROJ_SPD: two partials per 128-column tile, one per thread of a row)
int pre_ss_tiles(PreEpilogue epi, int H) { return epi == PRE_OPROJ_SPD ? 2 * ((H + 127) / 128) : (H + 255) / 256; }

cudaError_t launch_gemm_prefill(PreEpilogue epi, const TcMap *const *weights, const TcMap &tokens, const PreGemmArgs &g,
                                cudaStream_t st)
{
    const int nw = g.n_weights;
    if (nw < 1 || nw > 3 || (epi == PRE_GATEUP && nw != (g.fc1_only ? 1 : 2))) return cudaErrorInvalidValue;
    if (epi == PRE_GATEUP && g.fc1_only && (!g.ln_wg || !g.ln_wb)) return cudaErrorInvalidValue;
    if (g.t_rows <= 0) return cudaSuccess;
    if (g.num_kb < 1 || g.batches < 1 || g.batches > 8) return cudaErrorInvalidValue;
    if (epi == PRE_QKV && (256 % g.head_dim || g.head_dim < 32)) return cudaErrorInvalidValue;
    if ((epi == PRE_RESID || epi == PRE_OPROJ_SPD || epi == PRE_SCATTER) && g.H % 16) return cudaErrorInvalidValue;
    if (epi == PRE_SCATTER && (!g.pair || g.sc.T < 1 || g.sc.T > TP_MAX_RANKS || !g.sc.step)) return cudaErrorInvalidValue;
    if (epi == PRE_OPROJ_SPD && !g.norm_only && (!g.gain || !g.hg || !g.res_out)) return cudaErrorInvalidValue;
    if (epi == PRE_OPROJ_SPD && g.norm_only && !g.ss_out) return cudaErrorInvalidValue;
    if (g.w_rot < 0 || g.w_rot >= g.batches) return cudaErrorInvalidValue;
    if (epi == PRE_GATEUP && g.Fs % 8) return cudaErrorInvalidValue;
    const CUtensorMap *tw[3];
    for (int i = 0; i < 3; ++i) tw[i] = (const CUtensorMap *)weights[i < nw ? i : 0];
    PreLaunch L;
    L.g = g;
    const bool pair = g.pair != 0;
    if (pair && g.norm_only) return cudaErrorInvalidValue;
    L.m_tiles = pair ? (g.t_rows + 2 * BM - 1) / (2 * BM) : (g.t_rows + BM - 1) / BM;
    L.group_m = g.group_m > 0 ? g.group_m : (pair ? 8 : 16);
    L.passes = 1;
    L.f_tiles = 1;
    for (int i = 0; i < 3; ++i) L.tile_start[i] = 1 << 30;
    switch (epi) {
    case PRE_QKV: {
        int tiles = 0;
        for (int i = 0; i < nw; ++i) {
            if (g.w_rows[i] <= 0) return cudaErrorInvalidValue;
            L.tile_start[i] = tiles;
            tiles += (g.w_rows[i] + 255) / 256;
        }
        L.n_tiles = tiles;
        return pair ? launch_epi<PRE_QKV, 1>(tw, *(const CUtensorMap *)&tokens, L, st) : launch_epi<PRE_QKV, 0>(tw, *(const CUtensorMap *)&tokens, L, st);
    }
    case PRE_GATEUP:
        L.f_tiles = g.fc1_only ? (g.Fs + 255) / 256 : (g.Fs + 127) / 128;
        L.n_tiles = L.f_tiles * g.batches;
        return pair ? launch_epi<PRE_GATEUP, 1>(tw, *(const CUtensorMap *)&tokens, L, st) : launch_epi<PRE_GATEUP, 0>(tw, *(const CUtensorMap *)&tokens, L, st);
    case PRE_OPROJ_SPD:
        L.n_tiles = (g.H + 127) / 128;
        L.passes = g.batches;
        return pair ? launch_epi<PRE_OPROJ_SPD, 1>(tw, *(const CUtensorMap *)&tokens, L, st) : launch_epi<PRE_OPROJ_SPD, 0>(tw, *(const CUtensorMap *)&tokens, L, st);
    case PRE_SCATTER:
        L.n_tiles = (g.H + 255) / 256;
        return launch_epi<PRE_SCATTER, 1>(tw, *(const CUtensorMap *)&tokens, L, st);
    default:
        L.n_tiles = (g.H + 255) / 256;
        return pair ? launch_epi<PRE_RESID, 1>(tw, *(const CUtensorMap *)&tokens, L, st) : launch_epi<PRE_RESID, 0>(tw, *(const CUtensorMap *)&tokens, L, st);
    }
}

cudaError_t launch_prefill_prologue(const PrologueArgs &a, cudaStream_t st)
{
    if (a.M <= 0) return cudaSuccess;
    if (a.H % 8) return cudaErrorInvalidValue;
    return launch_kernel(prefill_prologue_kernel, dim3(a.M), dim3(256), 0, st, 0, a);
}

} // namespace spd
