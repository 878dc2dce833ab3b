/*
 * CPU checker for the batched autoregressive Transformer decoder of attention
 * encoder-decoder (AED) speech models.  TEST INFRASTRUCTURE ONLY: it exists to
 * check the CUDA library and to be timed as a CPU baseline.  It is deliberately
 * plain and slow, shares no code with the CUDA path, and must never be called
 * by the product.
 *
 * What it computes.  The paper (Section "Methods", paragraph on transferring
 * capacity from decoder to encoder; abstract) names the autoregressive
 * cross-attention Transformer decoder as the inference bottleneck but prints
 * no equations for it.  The definition evaluated here is therefore the
 * textbook pre-LN Transformer decoder (Vaswani et al., the lineage the paper
 * cites in "Related work"), with the readings listed below; the per-layer
 * parameter budget 16 d^2 agrees with the paper's parameter arithmetic
 * (1016M -> 680M when 20 layers are removed, Table "rtfx").
 *
 *   x_t^0 = E[y_t] * sqrt(d) + PE(t)      PE(t)[2i] = sin(t / 10000^(2i/d)), PE(t)[2i+1] = cos(same)
 *   for each layer:
 *     a   = LN1(x);   q,k,v = a Wq^T + bq, a Wk^T + bk, a Wv^T + bv     (w_qkv rows: q block, k block, v block)
 *     s   = concat_h softmax_{j<=t}(q_h . k_{j,h} / sqrt(dh)) v_{j,h}
 *     x'  = x + s Wo^T + bo
 *     c   = LN2(x');  q' = c Wqc^T + bqc;  Kc = X Wkc^T + bkc;  Vc = X Wvc^T + bvc   (w_kv_c rows: k block, v block)
 *     s'  = concat_h softmax_{j<T}(q'_h . Kc_{j,h} / sqrt(dh)) Vc_{j,h}     (exactly the T frames of this utterance)
 *     x'' = x' + s' Woc^T + boc
 *     f   = LN3(x''); x_next = x'' + relu(f W1^T + b1) W2^T + b2
 *   z_t = LNf(x_t) Wout^T + bout;   next_t = lowest index attaining max z_t
 *   LN(x) = g * (x - mean) / sqrt(mean((x - mean)^2) + eps) + b     (biased variance over d)
 *
 * Readings where the paper is silent: fixed sinusoidal positions, embedding
 * scaled by sqrt(d), no embedding LayerNorm, untied output projection, biases
 * on every projection (NULL = none), ReLU, final LayerNorm, attention scale
 * 1/sqrt(dh), positions outside the causal prefix / the utterance's own frames
 * are left out of the softmax sum rather than masked with a constant, no
 * LayerNorm on the encoder states, argmax ties go to the lowest index.
 *
 * Pins (tests/test_oracle_pins.py): incremental == full recompute, batch
 * composition invariance, softmax rows sum to 1, encoder-frame permutation
 * invariance, closed forms (T=1, t=0, Wq=0, zeroed output projections, LN of
 * constants), agreement with torch.nn.TransformerDecoderLayer in fp64, the
 * paper's per-layer parameter count, planted argmax ties.  The absolute logit
 * values of the seeded workloads have no external ground truth: beyond those
 * pins they are "parity unpinned".
 *
 * Precision: arithmetic in `real` (double by default; -DORC_REAL=float gives
 * the fp32 build that is timed as the CPU baseline).  Parameters and encoder
 * states arrive as float (exact for both fp32 and bf16-representable inputs).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef ORC_REAL
#define ORC_REAL double
#endif
typedef ORC_REAL real;

typedef struct {
    int32_t n_layers, d_model, n_heads, d_ffn, vocab, d_enc;
    double ln_eps;
    int32_t cross_kv_e4m3;   /* nonzero: the cross-attention keys and values are stored as 8-bit floats (see below) */
} orc_config_t;

/* Row-major [out, in] matrices; per-layer members are arrays of n_layers pointers; NULL bias = no bias. */
typedef struct {
    const float *embed, *final_ln_g, *final_ln_b, *w_out, *b_out;
    const float *const *ln1_g, *const *ln1_b, *const *w_qkv, *const *b_qkv, *const *w_o, *const *b_o;
    const float *const *ln2_g, *const *ln2_b, *const *w_q_c, *const *b_q_c, *const *w_kv_c, *const *b_kv_c,
                *const *w_o_c, *const *b_o_c;
    const float *const *ln3_g, *const *ln3_b, *const *w_ff1, *const *b_ff1, *const *w_ff2, *const *b_ff2;
} orc_weights_t;

/* Optional record of every softmax row, for the "rows sum to 1" pin.
 * self_probs  [L][n_layers][n_heads][L]   (entries j > t are left at 0)
 * cross_probs [L][n_layers][n_heads][T]                                    */
typedef struct {
    double *self_probs;
    double *cross_probs;
} orc_trace_t;

int orc_real_bytes(void) { return (int)sizeof(real); }

/* y = W x + b */
static void linear(const float *W, const float *b, const real *x, int n_out, int n_in, real *y)
{
    for (int o = 0; o < n_out; ++o) {
        real acc = b ? (real)b[o] : (real)0;
        const float *w = W + (size_t)o * n_in;
        for (int i = 0; i < n_in; ++i) acc += (real)w[i] * x[i];
        y[o] = acc;
    }
}

/* same with a float input vector (encoder frames) */
static void linear_f(const float *W, const float *b, const float *x, int n_out, int n_in, real *y)
{
    for (int o = 0; o < n_out; ++o) {
        real acc = b ? (real)b[o] : (real)0;
        const float *w = W + (size_t)o * n_in;
        for (int i = 0; i < n_in; ++i) acc += (real)w[i] * (real)x[i];
        y[o] = acc;
    }
}

void orc_layernorm(const real *x, const float *g, const float *b, int d, double eps, real *y)
{
    real mean = 0;
    for (int i = 0; i < d; ++i) mean += x[i];
    mean /= (real)d;
    real var = 0;
    for (int i = 0; i < d; ++i) var += (x[i] - mean) * (x[i] - mean);
    var /= (real)d;
    real inv = (real)1 / (real)sqrt((double)var + eps);
    for (int i = 0; i < d; ++i) y[i] = (real)g[i] * (x[i] - mean) * inv + (real)b[i];
}

/* lowest index attaining the maximum; *margin = top1 - top2 (0 when vocab == 1) */
int32_t orc_argmax(const real *z, int n, double *margin)
{
    int best = 0;
    for (int i = 1; i < n; ++i) if (z[i] > z[best]) best = i;
    if (margin) {
        double second = -INFINITY;
        for (int i = 0; i < n; ++i) if (i != best && (double)z[i] > second) second = (double)z[i];
        *margin = (n > 1) ? (double)z[best] - second : 0.0;
    }
    return best;
}

/* One query against n_pos cached positions, every head.  K, V: [n_pos][d] with head h in columns h*dh..h*dh+dh-1.
 * probs (nullable): [n_heads][probs_stride] receives the softmax row of each head. */
static void attend(const real *q, const real *K, const real *V, int n_pos, int n_heads, int dh,
                   real *out, double *probs, int probs_stride, real *score)
{
    int d = n_heads * dh;
    real scale = (real)1 / (real)sqrt((double)dh);
    for (int h = 0; h < n_heads; ++h) {
        real mx = -INFINITY;
        for (int j = 0; j < n_pos; ++j) {
            real s = 0;
            for (int c = 0; c < dh; ++c) s += q[h * dh + c] * K[(size_t)j * d + h * dh + c];
            s *= scale;
            score[j] = s;
            if (s > mx) mx = s;
        }
        real denom = 0;
        for (int j = 0; j < n_pos; ++j) { score[j] = (real)exp((double)(score[j] - mx)); denom += score[j]; }
        for (int c = 0; c < dh; ++c) out[h * dh + c] = 0;
        for (int j = 0; j < n_pos; ++j) {
            real p = score[j] / denom;
            if (probs) probs[(size_t)h * probs_stride + j] = (double)p;
            for (int c = 0; c < dh; ++c) out[h * dh + c] += p * V[(size_t)j * d + h * dh + c];
        }
    }
}

static void embed_token(const orc_config_t *cfg, const orc_weights_t *w, int32_t tok, int t, real *x)
{
    int d = cfg->d_model;
    double sq = sqrt((double)d);
    for (int i = 0; i < d; ++i) {
        int pair = i / 2;
        double angle = (double)t / pow(10000.0, (2.0 * pair) / (double)d);
        double pe = (i % 2 == 0) ? sin(angle) : cos(angle);
        x[i] = (real)((double)w->embed[(size_t)tok * d + i] * sq + pe);
    }
}

/* Nearest value of the 8-bit floating-point format E4M3 (OCP 8-bit Floating Point Specification: 1 sign bit, 4
 * exponent bits with bias 7, 3 mantissa bits, subnormals at exponent field 0, no infinities, largest finite value
 * 448), ties to the even mantissa, magnitudes beyond the largest finite value saturate to it.  A storage format the
 * paper does not discuss: the cross-attention K/V store is the largest stream of a decode step, and storing it in
 * 8 bits is this repository's extension; both sides of a parity test round the same way. */
double orc_round_e4m3(double x)
{
    if (x != x || x == 0.0) return x;
    double a = fabs(x);
    int e;
    (void)frexp(a, &e);                 /* a = m * 2^e with m in [0.5, 1): the leading bit has weight 2^(e-1) */
    int lead = e - 1;
    if (lead < -6) lead = -6;           /* subnormals share the quantum of the smallest normal binade: 2^-9 */
    double quantum = ldexp(1.0, lead - 3);
    double r = nearbyint(a / quantum) * quantum;     /* default rounding mode: to nearest, ties to even */
    if (r > 448.0) r = 448.0;
    return x < 0 ? -r : r;
}

/* Kc, Vc of one layer: [T][d] each */
static void cross_kv(const orc_config_t *cfg, const orc_weights_t *w, int layer, const float *enc, int T,
                     real *Kc, real *Vc, real *tmp /* [2d] */)
{
    int d = cfg->d_model;
    for (int j = 0; j < T; ++j) {
        linear_f(w->w_kv_c[layer], w->b_kv_c ? w->b_kv_c[layer] : NULL, enc + (size_t)j * cfg->d_enc, 2 * d, cfg->d_enc, tmp);
        if (cfg->cross_kv_e4m3)
            for (int o = 0; o < 2 * d; ++o) tmp[o] = (real)orc_round_e4m3((double)tmp[o]);
        memcpy(Kc + (size_t)j * d, tmp, sizeof(real) * d);
        memcpy(Vc + (size_t)j * d, tmp + d, sizeof(real) * d);
    }
}

#define BIAS(member, l) (w->member ? w->member[l] : NULL)

/* Incremental decoding of ONE utterance with self and cross K/V caches.
 *   enc [T][d_enc]; forced (nullable) [L]: the input token of every step (forced[0] is the start token);
 *   when forced == NULL the run is free-running greedy from `bos`.
 *   logits (nullable) [L][vocab] double; next [L]; margin (nullable) [L].
 *   eos: end-of-sequence token id, or a negative value to disable it.  When enabled, the step that emits
 *   eos is the utterance's last: the token is recorded and counted, nothing is computed after it, and
 *   next[t] = -1 for the remaining steps.  out_len (nullable) receives the number of emitted tokens.
 * Returns 0, or -1 on allocation failure / bad sizes.                                                   */
int orc_decode(const orc_config_t *cfg, const orc_weights_t *w, const float *enc, int32_t T,
               const int32_t *forced, int32_t bos, int32_t L,
               double *logits, int32_t *next, double *margin, const orc_trace_t *trace,
               int32_t eos, int32_t *out_len)
{
    int NL = cfg->n_layers, d = cfg->d_model, H = cfg->n_heads, F = cfg->d_ffn, V = cfg->vocab;
    if (T < 1 || L < 1 || d % H != 0) return -1;
    int dh = d / H;
    size_t kv = (size_t)NL * ((size_t)T + (size_t)L) * d * 2;
    real *pool = (real *)malloc(sizeof(real) * (kv + (size_t)8 * d + 3 * (size_t)d + F + V + (size_t)(T > L ? T : L)));
    if (!pool) return -1;
    real *Kc = pool, *Vc = Kc + (size_t)NL * T * d, *Ks = Vc + (size_t)NL * T * d, *Vs = Ks + (size_t)NL * L * d;
    real *x = Vs + (size_t)NL * L * d, *a = x + d, *qkv = a + d, *s = qkv + 3 * d, *o = s + d, *tmp2 = o + d;
    real *hid = tmp2 + 2 * d, *z = hid + F, *score = z + V;

    for (int l = 0; l < NL; ++l) cross_kv(cfg, w, l, enc, T, Kc + (size_t)l * T * d, Vc + (size_t)l * T * d, tmp2);

    int32_t tok = forced ? forced[0] : bos;
    for (int t = 0; t < L; ++t) {
        if (forced) tok = forced[t];
        if (tok < 0 || tok >= V) { free(pool); return -1; }
        embed_token(cfg, w, tok, t, x);
        for (int l = 0; l < NL; ++l) {
            real *Kl = Ks + (size_t)l * L * d, *Vl = Vs + (size_t)l * L * d;
            /* masked self-attention over positions 0..t */
            orc_layernorm(x, w->ln1_g[l], w->ln1_b[l], d, cfg->ln_eps, a);
            linear(w->w_qkv[l], BIAS(b_qkv, l), a, 3 * d, d, qkv);
            memcpy(Kl + (size_t)t * d, qkv + d, sizeof(real) * d);
            memcpy(Vl + (size_t)t * d, qkv + 2 * d, sizeof(real) * d);
            attend(qkv, Kl, Vl, t + 1, H, dh, s,
                   trace && trace->self_probs ? trace->self_probs + (((size_t)t * NL + l) * H) * L : NULL, L, score);
            linear(w->w_o[l], BIAS(b_o, l), s, d, d, o);
            for (int i = 0; i < d; ++i) x[i] += o[i];
            /* cross-attention over this utterance's T encoder frames */
            orc_layernorm(x, w->ln2_g[l], w->ln2_b[l], d, cfg->ln_eps, a);
            linear(w->w_q_c[l], BIAS(b_q_c, l), a, d, d, qkv);
            attend(qkv, Kc + (size_t)l * T * d, Vc + (size_t)l * T * d, T, H, dh, s,
                   trace && trace->cross_probs ? trace->cross_probs + (((size_t)t * NL + l) * H) * T : NULL, T, score);
            linear(w->w_o_c[l], BIAS(b_o_c, l), s, d, d, o);
            for (int i = 0; i < d; ++i) x[i] += o[i];
            /* feed-forward */
            orc_layernorm(x, w->ln3_g[l], w->ln3_b[l], d, cfg->ln_eps, a);
            linear(w->w_ff1[l], BIAS(b_ff1, l), a, F, d, hid);
            for (int i = 0; i < F; ++i) if (hid[i] < 0) hid[i] = 0;
            linear(w->w_ff2[l], BIAS(b_ff2, l), hid, d, F, o);
            for (int i = 0; i < d; ++i) x[i] += o[i];
        }
        orc_layernorm(x, w->final_ln_g, w->final_ln_b, d, cfg->ln_eps, a);
        linear(w->w_out, w->b_out, a, V, d, z);
        if (logits) for (int v = 0; v < V; ++v) logits[(size_t)t * V + v] = (double)z[v];
        tok = orc_argmax(z, V, margin ? margin + t : NULL);
        next[t] = tok;
        if (eos >= 0 && tok == eos) {          /* emitted and counted; the utterance ends here */
            for (int r = t + 1; r < L; ++r) { next[r] = -1; if (margin) margin[r] = 0.0; }
            if (out_len) *out_len = t + 1;
            free(pool);
            return 0;
        }
    }
    if (out_len) *out_len = L;
    free(pool);
    return 0;
}

/* Brute force: at every step t the whole prefix y_0..y_t is pushed through the decoder from scratch,
 * every position attending causally to the positions before it; nothing is cached between steps.
 * Same arguments as orc_decode (no trace).  Cost grows as L^2 layers: tiny inputs only.            */
int orc_decode_full_recompute(const orc_config_t *cfg, const orc_weights_t *w, const float *enc, int32_t T,
                              const int32_t *forced, int32_t bos, int32_t L,
                              double *logits, int32_t *next, double *margin)
{
    int NL = cfg->n_layers, d = cfg->d_model, H = cfg->n_heads, F = cfg->d_ffn, V = cfg->vocab;
    if (T < 1 || L < 1 || d % H != 0) return -1;
    int dh = d / H;
    size_t Ld = (size_t)L * d;
    real *pool = (real *)malloc(sizeof(real) * (2 * (size_t)T * d + 6 * Ld + 4 * (size_t)d + F + V + (size_t)(T > L ? T : L)));
    int32_t *y = (int32_t *)malloc(sizeof(int32_t) * L);
    if (!pool || !y) { free(pool); free(y); return -1; }
    real *Kc = pool, *Vc = Kc + (size_t)T * d;
    real *X = Vc + (size_t)T * d, *A = X + Ld, *Q = A + Ld, *K = Q + Ld, *Vv = K + Ld, *S = Vv + Ld;
    real *o = S + Ld, *tmp2 = o + d, *hid = tmp2 + 2 * d + d, *z = hid + F, *score = z + V;
    real *qkv = (real *)malloc(sizeof(real) * 3 * d);
    if (!qkv) { free(pool); free(y); return -1; }

    y[0] = forced ? forced[0] : bos;
    for (int t = 0; t < L; ++t) {
        if (forced) y[t] = forced[t];
        int n = t + 1;
        for (int i = 0; i < n; ++i) {
            if (y[i] < 0 || y[i] >= V) { free(pool); free(y); free(qkv); return -1; }
            embed_token(cfg, w, y[i], i, X + (size_t)i * d);
        }
        for (int l = 0; l < NL; ++l) {
            for (int i = 0; i < n; ++i) {
                orc_layernorm(X + (size_t)i * d, w->ln1_g[l], w->ln1_b[l], d, cfg->ln_eps, A + (size_t)i * d);
                linear(w->w_qkv[l], BIAS(b_qkv, l), A + (size_t)i * d, 3 * d, d, qkv);
                memcpy(Q + (size_t)i * d, qkv, sizeof(real) * d);
                memcpy(K + (size_t)i * d, qkv + d, sizeof(real) * d);
                memcpy(Vv + (size_t)i * d, qkv + 2 * d, sizeof(real) * d);
            }
            for (int i = 0; i < n; ++i)   /* causal: position i sees 0..i */
                attend(Q + (size_t)i * d, K, Vv, i + 1, H, dh, S + (size_t)i * d, NULL, 0, score);
            for (int i = 0; i < n; ++i) {
                linear(w->w_o[l], BIAS(b_o, l), S + (size_t)i * d, d, d, o);
                for (int c = 0; c < d; ++c) X[(size_t)i * d + c] += o[c];
            }
            cross_kv(cfg, w, l, enc, T, Kc, Vc, tmp2);
            for (int i = 0; i < n; ++i) {
                orc_layernorm(X + (size_t)i * d, w->ln2_g[l], w->ln2_b[l], d, cfg->ln_eps, A + (size_t)i * d);
                linear(w->w_q_c[l], BIAS(b_q_c, l), A + (size_t)i * d, d, d, Q + (size_t)i * d);
                attend(Q + (size_t)i * d, Kc, Vc, T, H, dh, S + (size_t)i * d, NULL, 0, score);
                linear(w->w_o_c[l], BIAS(b_o_c, l), S + (size_t)i * d, d, d, o);
                for (int c = 0; c < d; ++c) X[(size_t)i * d + c] += o[c];
            }
            for (int i = 0; i < n; ++i) {
                orc_layernorm(X + (size_t)i * d, w->ln3_g[l], w->ln3_b[l], d, cfg->ln_eps, A + (size_t)i * d);
                linear(w->w_ff1[l], BIAS(b_ff1, l), A + (size_t)i * d, F, d, hid);
                for (int c = 0; c < F; ++c) if (hid[c] < 0) hid[c] = 0;
                linear(w->w_ff2[l], BIAS(b_ff2, l), hid, d, F, o);
                for (int c = 0; c < d; ++c) X[(size_t)i * d + c] += o[c];
            }
        }
        orc_layernorm(X + (size_t)t * d, w->final_ln_g, w->final_ln_b, d, cfg->ln_eps, A);
        linear(w->w_out, w->b_out, A, V, d, z);
        if (logits) for (int v = 0; v < V; ++v) logits[(size_t)t * V + v] = (double)z[v];
        next[t] = orc_argmax(z, V, margin ? margin + t : NULL);
        if (t + 1 < L && !forced) y[t + 1] = next[t];
    }
    free(pool); free(y); free(qkv);
    return 0;
}

/* A batch of utterances, each decoded on its own (they are independent), spread over OpenMP threads.
 *   enc_packed [sum T][d_enc] with enc_offsets [B+1] (in frames); lens [B];
 *   forced (nullable) [B][stride]; next [B][stride]; margin (nullable) [B][stride];
 *   logits (nullable): utterance u's [lens[u]][vocab] block starts at logit_offsets[u] rows.
 *   eos (negative = disabled) and out_lens (nullable) [B]: as in orc_decode.
 * Returns the number of threads used, or a negative value if any utterance failed.                     */
int orc_decode_batch(const orc_config_t *cfg, const orc_weights_t *w, const float *enc_packed,
                     const int64_t *enc_offsets, int32_t B, const int32_t *forced, int32_t stride, int32_t bos,
                     const int32_t *lens, double *logits, const int64_t *logit_offsets,
                     int32_t *next, double *margin, int32_t n_threads, int32_t eos, int32_t *out_lens)
{
    int failed = 0, used = 1;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel
    {
#pragma omp single
        used = omp_get_num_threads();
#pragma omp for schedule(dynamic, 1)
        for (int u = 0; u < B; ++u) {
            int rc = orc_decode(cfg, w, enc_packed + (size_t)enc_offsets[u] * cfg->d_enc,
                                (int32_t)(enc_offsets[u + 1] - enc_offsets[u]),
                                forced ? forced + (size_t)u * stride : NULL, bos, lens[u],
                                logits ? logits + (size_t)logit_offsets[u] * cfg->vocab : NULL,
                                next + (size_t)u * stride, margin ? margin + (size_t)u * stride : NULL, NULL,
                                eos, out_lens ? out_lens + u : NULL);
            if (rc != 0) {
#pragma omp atomic write
                failed = 1;
            }
        }
    }
#else
    (void)n_threads;
    for (int u = 0; u < B; ++u) {
        int rc = orc_decode(cfg, w, enc_packed + (size_t)enc_offsets[u] * cfg->d_enc,
                            (int32_t)(enc_offsets[u + 1] - enc_offsets[u]),
                            forced ? forced + (size_t)u * stride : NULL, bos, lens[u],
                            logits ? logits + (size_t)logit_offsets[u] * cfg->vocab : NULL,
                            next + (size_t)u * stride, margin ? margin + (size_t)u * stride : NULL, NULL,
                                eos, out_lens ? out_lens + u : NULL);
        if (rc != 0) failed = 1;
    }
#endif
    return failed ? -1 : used;
}

/* Thin exports of the building blocks, so that tests can pin them one by one (double in, double out). */
void orc_layernorm_f64(const double *x, const float *g, const float *b, int d, double eps, double *y)
{
    real *xi = (real *)malloc(sizeof(real) * 2 * d), *yo = xi + d;
    for (int i = 0; i < d; ++i) xi[i] = (real)x[i];
    orc_layernorm(xi, g, b, d, eps, yo);
    for (int i = 0; i < d; ++i) y[i] = (double)yo[i];
    free(xi);
}

int32_t orc_argmax_f64(const double *z, int n, double *margin)
{
    real *zi = (real *)malloc(sizeof(real) * n);
    for (int i = 0; i < n; ++i) zi[i] = (real)z[i];
    int32_t r = orc_argmax(zi, n, margin);
    free(zi);
    return r;
}
