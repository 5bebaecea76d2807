/*
 * CPU oracle for the Sync-Point Drop (SPD) decoder block and the fully
 * synchronous tensor-parallel (TP) decoder block.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * step-by-step restatement of the method, used by the tests, by the smoke
 * check and by the timed CPU baseline of the benchmark.  The CUDA library
 * shares no code with it and never calls it.
 *
 * Arithmetic: inputs and weights arrive as float (for bf16 workloads the
 * caller passes bf16-representable values); every intermediate and every
 * output is double.  No blocking, no fusion, no reordering: one loop nest
 * per step, in the order the paper gives them.
 *
 * What follows the paper and what is a stated reading of it:
 *   - TP block, column split of Q/K/V and gate/up, row split of the attention
 *     output projection and of the down projection, all-reduce after each
 *     row-split layer                         : Sec. 3, Fig. 1(a), Sec. 4.1.2
 *   - SPD block without bias: MLP input of device i is X + Y_i; Y_i joins the
 *     MLP output before the kept all-reduce, X after it, giving
 *     X + sum_i Y_i + sum_i Z_i                : Sec. 4.1.1, Fig. 3(a)
 *   - rejected design "Y_i after the MLP all-reduce" : Table 1(a)
 *   - pre-normalisation LLaMA-2 block (RMSNorm, rotary embedding in the
 *     rotate-half pairing, SwiGLU, grouped-query attention, causal softmax
 *     with scale 1/sqrt(d)): the paper is silent; these are the conventions
 *     of the LLaMA-2 models it evaluates (Sec. 5.1).  In an SPD block the MLP
 *     RMSNorm is applied per device to X + Y_i.
 *
 *   - decoder block with bias (OPT-style): Y_i = P_i + b; MLP input of device i is
 *     X + P_i + b; P_i joins before the kept all-reduce, b and X after it, giving
 *     X + sum_i P_i + b + sum_i Z_i             : Sec. 4.1.2, Fig. 3(b); rejected design
 *     "b before the all-reduce"                 : Table 1(b).  Pre-LayerNorm OPT block
 *     (LayerNorm, biased projections, ReLU, no rotary embedding): the OPT models of Sec. 5.1.
 *     Pins: tests/test_oracle_bias_pins.py (transformers OPT decoder layer, invariants).
 *
 * Parity pins (tests/test_oracle_pins.py): the unsharded block against the
 * `transformers` LLaMA decoder layer and torch library attention; all-sync
 * stacks of any T against the unsharded block; T = 1 SPD against sync;
 * degenerate weights; permutation invariants; decode-vs-prefill cache
 * consistency; the sync-point count.  Absolute block outputs are otherwise
 * "parity unpinned": the paper prints no numeric block output.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, T;
    double rms_eps;
    double rope_base; /* <= 0: no rotary embedding */
} oracle_dims;

typedef struct {
    const float *attn_norm; /* [H]            */
    const float *wq;        /* [nq*d, H]      */
    const float *wk;        /* [nkv*d, H]     */
    const float *wv;        /* [nkv*d, H]     */
    const float *wo;        /* [H, nq*d]      */
    const float *mlp_norm;  /* [H]            */
    const float *w_gate;    /* [F, H]         */
    const float *w_up;      /* [F, H]         */
    const float *w_down;    /* [H, F]         */
} oracle_layer;

/* ------------------------------------------------------------------ */
/* primitives                                                          */
/* ------------------------------------------------------------------ */

/* y[m, n] = sum_k x[m, k] * w[n0 + n, k0 + k], w row-major with row length ldw.
 * A linear layer in torch.nn.Linear layout restricted to a row range (column
 * split) and/or an input range (row split). */
static void linear_slice(const double *x, int M, int ldx, int k_len,
                         const float *w, int ldw, int n0, int n_len, int k0,
                         double *y, int ldy)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < n_len; ++n) {
            const double *xr = x + (size_t)m * ldx;
            const float *wr = w + (size_t)(n0 + n) * ldw + k0;
            double acc = 0.0;
#pragma omp simd reduction(+ : acc)
            for (int k = 0; k < k_len; ++k) acc += xr[k] * (double)wr[k];
            y[(size_t)m * ldy + n] = acc;
        }
}

/* RMSNorm: out = x / sqrt(mean(x^2) + eps) * g, row by row. */
void oracle_rmsnorm(const double *x, const float *g, int M, int H, double eps, double *out)
{
    for (int m = 0; m < M; ++m) {
        double ss = 0.0;
        for (int j = 0; j < H; ++j) ss += x[(size_t)m * H + j] * x[(size_t)m * H + j];
        double r = 1.0 / sqrt(ss / (double)H + eps);
        for (int j = 0; j < H; ++j) out[(size_t)m * H + j] = x[(size_t)m * H + j] * r * (double)g[j];
    }
}

/* Rotary embedding on one head vector v[d] at absolute position pos:
 * pairs (j, j + d/2), angle pos * base^(-2j/d). */
void oracle_rope(double *v, int d, int pos, double base)
{
    int half = d / 2;
    for (int j = 0; j < half; ++j) {
        double theta = pow(base, -2.0 * (double)j / (double)d);
        double c = cos((double)pos * theta), s = sin((double)pos * theta);
        double a = v[j], b = v[j + half];
        v[j] = a * c - b * s;
        v[j + half] = b * c + a * s;
    }
}

static double silu(double x) { return x / (1.0 + exp(-x)); }

/* Causal attention of ONE query head vector q[d] at absolute position pos of
 * sequence b against kv head kvh of the cache (positions 0..pos inclusive). */
static void attend_one(const double *q, int d, int pos, const double *kc, const double *vc,
                       size_t tok_stride, double *out)
{
    int n = pos + 1;
    double *p = (double *)malloc(sizeof(double) * (size_t)n);
    double scale = 1.0 / sqrt((double)d), mx = -INFINITY;
    for (int t = 0; t < n; ++t) {
        double s = 0.0;
        for (int j = 0; j < d; ++j) s += q[j] * kc[(size_t)t * tok_stride + j];
        p[t] = s * scale;
        if (p[t] > mx) mx = p[t];
    }
    double den = 0.0;
    for (int t = 0; t < n; ++t) { p[t] = exp(p[t] - mx); den += p[t]; }
    for (int j = 0; j < d; ++j) out[j] = 0.0;
    for (int t = 0; t < n; ++t) {
        double w = p[t] / den;
        for (int j = 0; j < d; ++j) out[j] += w * vc[(size_t)t * tok_stride + j];
    }
    free(p);
}

/* ------------------------------------------------------------------ */
/* one TP / SPD block over T emulated devices                          */
/* ------------------------------------------------------------------ */

/* KV cache of the oracle: double [n_layers][B][max_len][nkv*d], contiguous
 * (paging is a storage detail of the CUDA library, not of the method).
 *
 * x      : [B, S, H]  block input X (S new tokens per sequence)
 * pos0   : [B]        tokens already cached for each sequence
 * mode   : 1 = synchronous TP block, 0 = SPD block,
 *          2 = rejected design of Table 1(a) (Y_i added after the MLP sum;
 *              the output then differs per device and `out` is [T, B, S, H])
 * out    : [B, S, H]
 * y_out  : optional [T, B*S, H] per-device partial attention outputs Y_i
 * returns the number of shard sums ("sync-points") executed: 2 or 1.
 */
static int block_sharded(const oracle_dims *D, const oracle_layer *W, int mode, const double *x,
                         int B, int S, const int32_t *pos0, double *kcache, double *vcache,
                         int max_len, double *out, double *y_out)
{
    const int H = D->hidden, nq = D->n_q_heads, nkv = D->n_kv_heads, d = D->head_dim;
    const int F = D->ffn, T = D->T, M = B * S;
    const int qh = nq / T, kvh = nkv / T, Fs = F / T, group = nq / nkv;
    const size_t kvw = (size_t)nkv * d; /* cache width per token */
    int sync_points = 0;

    double *h = malloc(sizeof(double) * (size_t)M * H);
    double *Y = malloc(sizeof(double) * (size_t)T * M * H); /* Y_i, i = 0..T-1 */
    double *Z = malloc(sizeof(double) * (size_t)T * M * H); /* Z_i             */

    /* pre-attention norm of the replicated block input */
    oracle_rmsnorm(x, W->attn_norm, M, H, D->rms_eps, h);

    /* pass 1 over devices: projections of the device's own heads, rotary, cache write */
    double **Qs = malloc(sizeof(double *) * (size_t)T);
    for (int i = 0; i < T; ++i) {
        double *Q = malloc(sizeof(double) * (size_t)M * qh * d);
        double *K = malloc(sizeof(double) * (size_t)M * kvh * d);
        double *V = malloc(sizeof(double) * (size_t)M * kvh * d);
        linear_slice(h, M, H, H, W->wq, H, i * qh * d, qh * d, 0, Q, qh * d);
        linear_slice(h, M, H, H, W->wk, H, i * kvh * d, kvh * d, 0, K, kvh * d);
        linear_slice(h, M, H, H, W->wv, H, i * kvh * d, kvh * d, 0, V, kvh * d);
        for (int b = 0; b < B; ++b)
            for (int s = 0; s < S; ++s) {
                int m = b * S + s, pos = pos0[b] + s;
                if (D->rope_base > 0.0) {
                    for (int j = 0; j < qh; ++j) oracle_rope(Q + ((size_t)m * qh + j) * d, d, pos, D->rope_base);
                    for (int j = 0; j < kvh; ++j) oracle_rope(K + ((size_t)m * kvh + j) * d, d, pos, D->rope_base);
                }
                double *kc = kcache + ((size_t)b * max_len + pos) * kvw + (size_t)i * kvh * d;
                double *vc = vcache + ((size_t)b * max_len + pos) * kvw + (size_t)i * kvh * d;
                memcpy(kc, K + (size_t)m * kvh * d, sizeof(double) * (size_t)kvh * d);
                memcpy(vc, V + (size_t)m * kvh * d, sizeof(double) * (size_t)kvh * d);
            }
        Qs[i] = Q;
        free(K);
        free(V);
    }

    /* pass 2 over devices: attention over own heads, own slice of the output projection */
    for (int i = 0; i < T; ++i) {
        double *A = malloc(sizeof(double) * (size_t)M * qh * d);
#pragma omp parallel for collapse(2) schedule(dynamic)
        for (int m = 0; m < M; ++m)
            for (int j = 0; j < qh; ++j) {
                int b = m / S, s = m % S, pos = pos0[b] + s;
                int gq = i * qh + j;   /* global query head */
                int gkv = gq / group;  /* its KV head (always on device i) */
                attend_one(Qs[i] + ((size_t)m * qh + j) * d, d, pos,
                           kcache + (size_t)b * max_len * kvw + (size_t)gkv * d,
                           vcache + (size_t)b * max_len * kvw + (size_t)gkv * d, kvw,
                           A + ((size_t)m * qh + j) * d);
            }
        /* Y_i = A_i W_O^(i)T : the rows of W_O^T (input features) owned by device i */
        linear_slice(A, M, qh * d, qh * d, W->wo, nq * d, 0, H, i * qh * d, Y + (size_t)i * M * H, H);
        free(A);
        free(Qs[i]);
    }
    free(Qs);
    if (y_out) memcpy(y_out, Y, sizeof(double) * (size_t)T * M * H);

    double *R = malloc(sizeof(double) * (size_t)M * H);
    double *u = malloc(sizeof(double) * (size_t)M * H);
    double *g = malloc(sizeof(double) * (size_t)M * Fs);
    double *up = malloc(sizeof(double) * (size_t)M * Fs);

    if (mode == 1) {
        /* sync-point #1: all-reduce of the attention outputs, then the residual add */
        for (size_t e = 0; e < (size_t)M * H; ++e) {
            double acc = 0.0;
            for (int i = 0; i < T; ++i) acc += Y[(size_t)i * M * H + e];
            R[e] = x[e] + acc;
        }
        sync_points++;
        oracle_rmsnorm(R, W->mlp_norm, M, H, D->rms_eps, u);
    }

    for (int i = 0; i < T; ++i) {
        if (mode != 1) {
            /* SPD: device i only has its own Y_i; MLP input is X + Y_i */
            for (size_t e = 0; e < (size_t)M * H; ++e) R[e] = x[e] + Y[(size_t)i * M * H + e];
            oracle_rmsnorm(R, W->mlp_norm, M, H, D->rms_eps, u);
        }
        linear_slice(u, M, H, H, W->w_gate, H, i * Fs, Fs, 0, g, Fs);
        linear_slice(u, M, H, H, W->w_up, H, i * Fs, Fs, 0, up, Fs);
        for (size_t e = 0; e < (size_t)M * Fs; ++e) g[e] = silu(g[e]) * up[e];
        linear_slice(g, M, Fs, Fs, W->w_down, F, 0, H, i * Fs, Z + (size_t)i * M * H, H);
    }

    if (mode == 1) {
        /* sync-point #2: all-reduce of Z_i; residual is the synchronised MLP input */
        for (size_t e = 0; e < (size_t)M * H; ++e) {
            double acc = 0.0;
            for (int i = 0; i < T; ++i) acc += Z[(size_t)i * M * H + e];
            out[e] = R[e] + acc;
        }
        sync_points++;
    } else if (mode == 0) {
        /* the one kept sync-point: Y_i is added before the all-reduce, X after it */
        for (size_t e = 0; e < (size_t)M * H; ++e) {
            double acc = 0.0;
            for (int i = 0; i < T; ++i) acc += Y[(size_t)i * M * H + e] + Z[(size_t)i * M * H + e];
            out[e] = x[e] + acc;
        }
        sync_points++;
    } else {
        /* Table 1(a), rejected: only Z_i is all-reduced; X and the local Y_i are added after */
        for (size_t e = 0; e < (size_t)M * H; ++e) {
            double acc = 0.0;
            for (int i = 0; i < T; ++i) acc += Z[(size_t)i * M * H + e];
            for (int i = 0; i < T; ++i) out[(size_t)i * M * H + e] = x[e] + Y[(size_t)i * M * H + e] + acc;
        }
        sync_points++;
    }

    free(h); free(Y); free(Z); free(R); free(u); free(g); free(up);
    return sync_points;
}

/* ------------------------------------------------------------------ */
/* the single-device block, written without any device loop            */
/* ------------------------------------------------------------------ */
static void block_unsharded(const oracle_dims *D, const oracle_layer *W, const double *x, int B,
                            int S, const int32_t *pos0, double *kcache, double *vcache,
                            int max_len, double *out)
{
    const int H = D->hidden, nq = D->n_q_heads, nkv = D->n_kv_heads, d = D->head_dim;
    const int F = D->ffn, M = B * S, group = nq / nkv;
    const size_t kvw = (size_t)nkv * d;

    double *h = malloc(sizeof(double) * (size_t)M * H);
    double *Q = malloc(sizeof(double) * (size_t)M * nq * d);
    double *K = malloc(sizeof(double) * (size_t)M * nkv * d);
    double *V = malloc(sizeof(double) * (size_t)M * nkv * d);
    double *A = malloc(sizeof(double) * (size_t)M * nq * d);
    double *R = malloc(sizeof(double) * (size_t)M * H);
    double *u = malloc(sizeof(double) * (size_t)M * H);
    double *g = malloc(sizeof(double) * (size_t)M * F);
    double *up = malloc(sizeof(double) * (size_t)M * F);

    oracle_rmsnorm(x, W->attn_norm, M, H, D->rms_eps, h);
    linear_slice(h, M, H, H, W->wq, H, 0, nq * d, 0, Q, nq * d);
    linear_slice(h, M, H, H, W->wk, H, 0, nkv * d, 0, K, nkv * d);
    linear_slice(h, M, H, H, W->wv, H, 0, nkv * d, 0, V, nkv * d);
    for (int m = 0; m < M; ++m) {
        int b = m / S, pos = pos0[b] + m % S;
        if (D->rope_base > 0.0) {
            for (int j = 0; j < nq; ++j) oracle_rope(Q + ((size_t)m * nq + j) * d, d, pos, D->rope_base);
            for (int j = 0; j < nkv; ++j) oracle_rope(K + ((size_t)m * nkv + j) * d, d, pos, D->rope_base);
        }
        memcpy(kcache + ((size_t)b * max_len + pos) * kvw, K + (size_t)m * kvw, sizeof(double) * kvw);
        memcpy(vcache + ((size_t)b * max_len + pos) * kvw, V + (size_t)m * kvw, sizeof(double) * kvw);
    }
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int m = 0; m < M; ++m)
        for (int j = 0; j < nq; ++j) {
            int b = m / S, pos = pos0[b] + m % S, gkv = j / group;
            attend_one(Q + ((size_t)m * nq + j) * d, d, pos,
                       kcache + (size_t)b * max_len * kvw + (size_t)gkv * d,
                       vcache + (size_t)b * max_len * kvw + (size_t)gkv * d, kvw,
                       A + ((size_t)m * nq + j) * d);
        }
    linear_slice(A, M, nq * d, nq * d, W->wo, nq * d, 0, H, 0, R, H);
    for (size_t e = 0; e < (size_t)M * H; ++e) R[e] += x[e];
    oracle_rmsnorm(R, W->mlp_norm, M, H, D->rms_eps, u);
    linear_slice(u, M, H, H, W->w_gate, H, 0, F, 0, g, F);
    linear_slice(u, M, H, H, W->w_up, H, 0, F, 0, up, F);
    for (size_t e = 0; e < (size_t)M * F; ++e) g[e] = silu(g[e]) * up[e];
    linear_slice(g, M, F, F, W->w_down, F, 0, H, 0, out, H);
    for (size_t e = 0; e < (size_t)M * H; ++e) out[e] += R[e];

    free(h); free(Q); free(K); free(V); free(A); free(R); free(u); free(g); free(up);
}

/* ------------------------------------------------------------------ */
/* the decoder block with bias (OPT-style), Sec. 4.1.2, Fig. 3(b)      */
/* ------------------------------------------------------------------ */

/* Pre-LayerNorm OPT decoder block (the OPT models of Sec. 5.1): LayerNorm with gain and shift,
 * biased q/k/v/out projections, no rotary embedding (OPT adds learned position embeddings
 * before the first block, i.e. outside it), fc1 + ReLU + fc2 with biases.
 * Tensor parallelism as in Sec. 3: q/k/v and fc1 column-split (their biases split with them),
 * out_proj and fc2 row-split; the bias of a row-split layer cannot be split and is added once,
 * after the all-reduce (Sec. 4.1.2: "the bias residual ... after the sync operation"). */
typedef struct {
    const float *attn_norm, *attn_norm_b; /* [H] gain, shift of the LayerNorm before attention */
    const float *wq, *bq;                 /* [nq*d, H], [nq*d]   */
    const float *wk, *bk, *wv, *bv;       /* [nkv*d, H], [nkv*d] */
    const float *wo, *bo;                 /* [H, nq*d], [H]: Y_i = P_i + b with b = bo */
    const float *mlp_norm, *mlp_norm_b;   /* [H] */
    const float *w_fc1, *b_fc1;           /* [F, H], [F] */
    const float *w_fc2, *b_fc2;           /* [H, F], [H] */
} oracle_bias_layer;

/* LayerNorm: out = (x - mean) / sqrt(var + eps) * g + b, biased variance, row by row. */
void oracle_layernorm(const double *x, const float *g, const float *b, int M, int H, double eps, double *out)
{
    for (int m = 0; m < M; ++m) {
        double mean = 0.0, var = 0.0;
        for (int j = 0; j < H; ++j) mean += x[(size_t)m * H + j];
        mean /= (double)H;
        for (int j = 0; j < H; ++j) { double c = x[(size_t)m * H + j] - mean; var += c * c; }
        var /= (double)H;
        double r = 1.0 / sqrt(var + eps);
        for (int j = 0; j < H; ++j) out[(size_t)m * H + j] = (x[(size_t)m * H + j] - mean) * r * (double)g[j] + (double)b[j];
    }
}

static void add_bias_cols(double *y, int M, int n_len, int ldy, const float *bias, int n0)
{
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < n_len; ++n) y[(size_t)m * ldy + n] += (double)bias[n0 + n];
}

/* mode 1: synchronous TP block.  mode 0: SPD block with bias (Sec. 4.1.2): the MLP input of device i
 * is X + P_i + b; P_i is added before the kept all-reduce, b and X after it:
 * X + sum_i P_i + b + sum_i Z_i.  mode 2: the rejected design of Table 1(b), b added before the
 * all-reduce (and so T times).  p_out: optional [T, B*S, H] partial products P_i (without b). */
static int block_sharded_bias(const oracle_dims *D, const oracle_bias_layer *W, int mode, const double *x, int B, int S,
                              const int32_t *pos0, double *kcache, double *vcache, int max_len, double *out, double *p_out)
{
    const int H = D->hidden, nq = D->n_q_heads, nkv = D->n_kv_heads, d = D->head_dim;
    const int F = D->ffn, T = D->T, M = B * S;
    const int qh = nq / T, kvh = nkv / T, Fs = F / T, group = nq / nkv;
    const size_t kvw = (size_t)nkv * d;
    int sync_points = 0;

    double *h = malloc(sizeof(double) * (size_t)M * H);
    double *P = malloc(sizeof(double) * (size_t)T * M * H);
    double *Z = malloc(sizeof(double) * (size_t)T * M * H);
    oracle_layernorm(x, W->attn_norm, W->attn_norm_b, M, H, D->rms_eps, h);

    double **Qs = malloc(sizeof(double *) * (size_t)T);
    for (int i = 0; i < T; ++i) {
        double *Q = malloc(sizeof(double) * (size_t)M * qh * d);
        double *K = malloc(sizeof(double) * (size_t)M * kvh * d);
        double *V = malloc(sizeof(double) * (size_t)M * kvh * d);
        linear_slice(h, M, H, H, W->wq, H, i * qh * d, qh * d, 0, Q, qh * d);
        linear_slice(h, M, H, H, W->wk, H, i * kvh * d, kvh * d, 0, K, kvh * d);
        linear_slice(h, M, H, H, W->wv, H, i * kvh * d, kvh * d, 0, V, kvh * d);
        add_bias_cols(Q, M, qh * d, qh * d, W->bq, i * qh * d);
        add_bias_cols(K, M, kvh * d, kvh * d, W->bk, i * kvh * d);
        add_bias_cols(V, M, kvh * d, kvh * d, W->bv, i * kvh * d);
        for (int b = 0; b < B; ++b)
            for (int s = 0; s < S; ++s) {
                int m = b * S + s, pos = pos0[b] + s;
                memcpy(kcache + ((size_t)b * max_len + pos) * kvw + (size_t)i * kvh * d, K + (size_t)m * kvh * d, sizeof(double) * (size_t)kvh * d);
                memcpy(vcache + ((size_t)b * max_len + pos) * kvw + (size_t)i * kvh * d, V + (size_t)m * kvh * d, sizeof(double) * (size_t)kvh * d);
            }
        Qs[i] = Q;
        free(K);
        free(V);
    }
    for (int i = 0; i < T; ++i) {
        double *A = malloc(sizeof(double) * (size_t)M * qh * d);
#pragma omp parallel for collapse(2) schedule(dynamic)
        for (int m = 0; m < M; ++m)
            for (int j = 0; j < qh; ++j) {
                int b = m / S, s = m % S, pos = pos0[b] + s;
                int gkv = (i * qh + j) / group;
                attend_one(Qs[i] + ((size_t)m * qh + j) * d, d, pos, kcache + (size_t)b * max_len * kvw + (size_t)gkv * d,
                           vcache + (size_t)b * max_len * kvw + (size_t)gkv * d, kvw, A + ((size_t)m * qh + j) * d);
            }
        /* P_i: the partial product of device i's slice of the row-split out_proj, without its bias */
        linear_slice(A, M, qh * d, qh * d, W->wo, nq * d, 0, H, i * qh * d, P + (size_t)i * M * H, H);
        free(A);
        free(Qs[i]);
    }
    free(Qs);
    if (p_out) memcpy(p_out, P, sizeof(double) * (size_t)T * M * H);

    double *R = malloc(sizeof(double) * (size_t)M * H);
    double *u = malloc(sizeof(double) * (size_t)M * H);
    double *a = malloc(sizeof(double) * (size_t)M * Fs);
    if (mode == 1) {
        /* sync-point #1: all-reduce of P_i, then the bias once, then the residual */
        for (size_t e = 0; e < (size_t)M * H; ++e) {
            double acc = 0.0;
            for (int i = 0; i < T; ++i) acc += P[(size_t)i * M * H + e];
            R[e] = x[e] + acc + (double)W->bo[e % H];
        }
        sync_points++;
        oracle_layernorm(R, W->mlp_norm, W->mlp_norm_b, M, H, D->rms_eps, u);
    }
    for (int i = 0; i < T; ++i) {
        if (mode != 1) {
            /* SPD: the MLP input of device i is X + P_i + b */
            for (size_t e = 0; e < (size_t)M * H; ++e) R[e] = x[e] + P[(size_t)i * M * H + e] + (double)W->bo[e % H];
            oracle_layernorm(R, W->mlp_norm, W->mlp_norm_b, M, H, D->rms_eps, u);
        }
        linear_slice(u, M, H, H, W->w_fc1, H, i * Fs, Fs, 0, a, Fs);
        add_bias_cols(a, M, Fs, Fs, W->b_fc1, i * Fs);
        for (size_t e = 0; e < (size_t)M * Fs; ++e) a[e] = a[e] > 0.0 ? a[e] : 0.0;
        linear_slice(a, M, Fs, Fs, W->w_fc2, F, 0, H, i * Fs, Z + (size_t)i * M * H, H);
    }
    for (size_t e = 0; e < (size_t)M * H; ++e) {
        double accz = 0.0, accp = 0.0;
        for (int i = 0; i < T; ++i) { accz += Z[(size_t)i * M * H + e]; accp += P[(size_t)i * M * H + e]; }
        const double bo = (double)W->bo[e % H], b2 = (double)W->b_fc2[e % H];
        if (mode == 1) out[e] = R[e] + accz + b2;                       /* sync-point #2 */
        else if (mode == 0) out[e] = x[e] + (accp + accz) + bo + b2;    /* P_i before the all-reduce, b and X after */
        else out[e] = x[e] + (accp + (double)T * bo + accz) + b2;       /* Table 1(b), rejected: b before the all-reduce */
    }
    sync_points++;
    free(h); free(P); free(Z); free(R); free(u); free(a);
    return sync_points;
}

/* the same block on one device, no device loop */
static void block_unsharded_bias(const oracle_dims *D, const oracle_bias_layer *W, const double *x, int B, int S,
                                 const int32_t *pos0, double *kcache, double *vcache, int max_len, double *out)
{
    const int H = D->hidden, nq = D->n_q_heads, nkv = D->n_kv_heads, d = D->head_dim;
    const int F = D->ffn, M = B * S, group = nq / nkv;
    const size_t kvw = (size_t)nkv * d;
    double *h = malloc(sizeof(double) * (size_t)M * H);
    double *Q = malloc(sizeof(double) * (size_t)M * nq * d);
    double *K = malloc(sizeof(double) * (size_t)M * nkv * d);
    double *V = malloc(sizeof(double) * (size_t)M * nkv * d);
    double *A = malloc(sizeof(double) * (size_t)M * nq * d);
    double *R = malloc(sizeof(double) * (size_t)M * H);
    double *u = malloc(sizeof(double) * (size_t)M * H);
    double *a = malloc(sizeof(double) * (size_t)M * F);
    oracle_layernorm(x, W->attn_norm, W->attn_norm_b, M, H, D->rms_eps, h);
    linear_slice(h, M, H, H, W->wq, H, 0, nq * d, 0, Q, nq * d);
    linear_slice(h, M, H, H, W->wk, H, 0, nkv * d, 0, K, nkv * d);
    linear_slice(h, M, H, H, W->wv, H, 0, nkv * d, 0, V, nkv * d);
    add_bias_cols(Q, M, nq * d, nq * d, W->bq, 0);
    add_bias_cols(K, M, nkv * d, nkv * d, W->bk, 0);
    add_bias_cols(V, M, nkv * d, nkv * d, W->bv, 0);
    for (int m = 0; m < M; ++m) {
        int b = m / S, pos = pos0[b] + m % S;
        memcpy(kcache + ((size_t)b * max_len + pos) * kvw, K + (size_t)m * kvw, sizeof(double) * kvw);
        memcpy(vcache + ((size_t)b * max_len + pos) * kvw, V + (size_t)m * kvw, sizeof(double) * kvw);
    }
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int m = 0; m < M; ++m)
        for (int j = 0; j < nq; ++j) {
            int b = m / S, pos = pos0[b] + m % S, gkv = j / group;
            attend_one(Q + ((size_t)m * nq + j) * d, d, pos, kcache + (size_t)b * max_len * kvw + (size_t)gkv * d,
                       vcache + (size_t)b * max_len * kvw + (size_t)gkv * d, kvw, A + ((size_t)m * nq + j) * d);
        }
    linear_slice(A, M, nq * d, nq * d, W->wo, nq * d, 0, H, 0, R, H);
    add_bias_cols(R, M, H, H, W->bo, 0);
    for (size_t e = 0; e < (size_t)M * H; ++e) R[e] += x[e];
    oracle_layernorm(R, W->mlp_norm, W->mlp_norm_b, M, H, D->rms_eps, u);
    linear_slice(u, M, H, H, W->w_fc1, H, 0, F, 0, a, F);
    add_bias_cols(a, M, F, F, W->b_fc1, 0);
    for (size_t e = 0; e < (size_t)M * F; ++e) a[e] = a[e] > 0.0 ? a[e] : 0.0;
    linear_slice(a, M, F, F, W->w_fc2, F, 0, H, 0, out, H);
    add_bias_cols(out, M, H, H, W->b_fc2, 0);
    for (size_t e = 0; e < (size_t)M * H; ++e) out[e] += R[e];
    free(h); free(Q); free(K); free(V); free(A); free(R); free(u); free(a);
}

/* ------------------------------------------------------------------ */
/* exported entry points                                               */
/* ------------------------------------------------------------------ */

static int dims_ok(const oracle_dims *D)
{
    if (D->n_layers < 1 || D->hidden < 1 || D->head_dim < 2 || (D->head_dim & 1) || D->T < 1) return 0;
    if (D->n_kv_heads < 1 || D->n_q_heads % D->n_kv_heads) return 0;
    if (D->n_q_heads % D->T || D->n_kv_heads % D->T || D->ffn % D->T) return 0;
    return 1;
}

/* A stack of blocks, each TP (mask[l] = 1) or SPD (mask[l] = 0): Algorithm 1's
 * block list after the replacement step.
 * x, out       : [B, S, H] double
 * kcache/vcache: [n_layers, B, max_len, nkv*d] double, caller-owned, updated
 * layer_out    : optional [n_layers, B*S, H], the output of every block
 * returns the total number of shard sums executed, or -1 on bad dims. */
int oracle_stack_forward(const oracle_dims *D, const uint8_t *mask, const oracle_layer *layers,
                         const double *x, int B, int S, const int32_t *pos0, double *kcache,
                         double *vcache, int max_len, double *out, double *layer_out)
{
    if (!dims_ok(D)) return -1;
    for (int b = 0; b < B; ++b)
        if (pos0[b] < 0 || pos0[b] + S > max_len) return -1;
    const size_t MH = (size_t)B * S * D->hidden;
    const size_t cache_l = (size_t)B * max_len * D->n_kv_heads * D->head_dim;
    double *cur = malloc(sizeof(double) * MH), *nxt = malloc(sizeof(double) * MH);
    memcpy(cur, x, sizeof(double) * MH);
    int sync_points = 0;
    for (int l = 0; l < D->n_layers; ++l) {
        sync_points += block_sharded(D, &layers[l], mask[l] ? 1 : 0, cur, B, S, pos0,
                                     kcache + (size_t)l * cache_l, vcache + (size_t)l * cache_l,
                                     max_len, nxt, NULL);
        if (layer_out) memcpy(layer_out + (size_t)l * MH, nxt, sizeof(double) * MH);
        double *t = cur; cur = nxt; nxt = t;
    }
    memcpy(out, cur, sizeof(double) * MH);
    free(cur); free(nxt);
    return sync_points;
}

/* The same stack on a single device: no shards, no mask. */
int oracle_unsharded_stack_forward(const oracle_dims *D, const oracle_layer *layers, const double *x,
                                   int B, int S, const int32_t *pos0, double *kcache, double *vcache,
                                   int max_len, double *out)
{
    if (!dims_ok(D)) return -1;
    for (int b = 0; b < B; ++b)
        if (pos0[b] < 0 || pos0[b] + S > max_len) return -1;
    const size_t MH = (size_t)B * S * D->hidden;
    const size_t cache_l = (size_t)B * max_len * D->n_kv_heads * D->head_dim;
    double *cur = malloc(sizeof(double) * MH), *nxt = malloc(sizeof(double) * MH);
    memcpy(cur, x, sizeof(double) * MH);
    for (int l = 0; l < D->n_layers; ++l) {
        block_unsharded(D, &layers[l], cur, B, S, pos0, kcache + (size_t)l * cache_l,
                        vcache + (size_t)l * cache_l, max_len, nxt);
        double *t = cur; cur = nxt; nxt = t;
    }
    memcpy(out, cur, sizeof(double) * MH);
    free(cur); free(nxt);
    return 0;
}

/* One block with access to what the figures mark: mode as in block_sharded
 * (0 SPD, 1 sync, 2 the rejected Table 1(a) design whose `out` is [T,B,S,H]);
 * y_out optional [T, B*S, H]. */
int oracle_block_forward(const oracle_dims *D, const oracle_layer *layer, int mode, const double *x,
                         int B, int S, const int32_t *pos0, double *kcache, double *vcache,
                         int max_len, double *out, double *y_out)
{
    if (!dims_ok(D) || mode < 0 || mode > 2) return -1;
    for (int b = 0; b < B; ++b)
        if (pos0[b] < 0 || pos0[b] + S > max_len) return -1;
    return block_sharded(D, layer, mode, x, B, S, pos0, kcache, vcache, max_len, out, y_out);
}

/* A plain linear layer y = x W^T (W in torch.nn.Linear layout), the building block of every
 * projection above; exported so that the GEMM kernels can be checked in isolation. */
void oracle_linear(const double *x, const float *w, int M, int N, int K, double *y)
{
    linear_slice(x, M, K, K, w, K, 0, N, 0, y, N);
}

/* ---- the block with bias: stack, single-device stack, one block ------------------------------- */

int oracle_bias_stack_forward(const oracle_dims *D, const uint8_t *mask, const oracle_bias_layer *layers, const double *x, int B,
                              int S, const int32_t *pos0, double *kcache, double *vcache, int max_len, double *out)
{
    if (!dims_ok(D)) return -1;
    for (int b = 0; b < B; ++b)
        if (pos0[b] < 0 || pos0[b] + S > max_len) return -1;
    const size_t MH = (size_t)B * S * D->hidden;
    const size_t cache_l = (size_t)B * max_len * D->n_kv_heads * D->head_dim;
    double *cur = malloc(sizeof(double) * MH), *nxt = malloc(sizeof(double) * MH);
    memcpy(cur, x, sizeof(double) * MH);
    int sync_points = 0;
    for (int l = 0; l < D->n_layers; ++l) {
        sync_points += block_sharded_bias(D, &layers[l], mask[l] ? 1 : 0, cur, B, S, pos0, kcache + (size_t)l * cache_l,
                                          vcache + (size_t)l * cache_l, max_len, nxt, NULL);
        double *t = cur; cur = nxt; nxt = t;
    }
    memcpy(out, cur, sizeof(double) * MH);
    free(cur); free(nxt);
    return sync_points;
}

int oracle_bias_unsharded_stack_forward(const oracle_dims *D, const oracle_bias_layer *layers, const double *x, int B, int S,
                                        const int32_t *pos0, double *kcache, double *vcache, int max_len, double *out)
{
    if (!dims_ok(D)) return -1;
    for (int b = 0; b < B; ++b)
        if (pos0[b] < 0 || pos0[b] + S > max_len) return -1;
    const size_t MH = (size_t)B * S * D->hidden;
    const size_t cache_l = (size_t)B * max_len * D->n_kv_heads * D->head_dim;
    double *cur = malloc(sizeof(double) * MH), *nxt = malloc(sizeof(double) * MH);
    memcpy(cur, x, sizeof(double) * MH);
    for (int l = 0; l < D->n_layers; ++l) {
        block_unsharded_bias(D, &layers[l], cur, B, S, pos0, kcache + (size_t)l * cache_l, vcache + (size_t)l * cache_l, max_len, nxt);
        double *t = cur; cur = nxt; nxt = t;
    }
    memcpy(out, cur, sizeof(double) * MH);
    free(cur); free(nxt);
    return 0;
}

/* mode 0 SPD (Sec. 4.1.2), 1 sync, 2 the rejected design of Table 1(b); p_out optional [T, B*S, H]. */
int oracle_bias_block_forward(const oracle_dims *D, const oracle_bias_layer *layer, int mode, const double *x, int B, int S,
                              const int32_t *pos0, double *kcache, double *vcache, int max_len, double *out, double *p_out)
{
    if (!dims_ok(D) || mode < 0 || mode > 2) return -1;
    for (int b = 0; b < B; ++b)
        if (pos0[b] < 0 || pos0[b] + S > max_len) return -1;
    return block_sharded_bias(D, layer, mode, x, B, S, pos0, kcache, vcache, max_len, out, p_out);
}
