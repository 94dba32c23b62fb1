/*
 * st_oracle.c -- CPU oracle for Speculative Thinking decode.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * hot path computes: two Qwen2-style decoder-only transformers (RMSNorm,
 * rotary position embedding, grouped-query attention, SwiGLU FFN) run with a
 * key/value cache, a greedy sampler, and the Speculative Thinking handoff rule
 * (paper Section 3, item (1) "Affirmation/Reflection Takeover", with the
 * hyper-parameters of the appendix "Hyperparameters of Speculative Thinking").
 * It shares no code with the CUDA library and must never be reached from the
 * product path.
 *
 * Precision: every weight is a bf16 value (exactly representable in float, and
 * stored as float); all arithmetic -- projections, normalisation, rotary
 * embedding, softmax, residuals, logits -- is done in IEEE double.  There is
 * no blocking, fusion or reordering: each function follows the textbook
 * definition of the layer it names.
 *
 * Parity status of the readings that the paper leaves open:
 *   - "replace" vs "keep" of the probe token (does the target's segment start
 *     right after the delimiter, or after the keyword?): parity unpinned; both
 *     are implemented (keep_probe flag), each pinned to a hand-traced stream.
 *   - everything else in this file is pinned by tests/test_oracle_*.py
 *     (closed forms, brute force, a hand-computed model, library routines).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Seeded weights: SplitMix64 counter streams -> Irwin-Hall(12) -> bf16       */
/* ------------------------------------------------------------------------- */

#define ORC_GAMMA 0x9e3779b97f4a7c15ULL

/* SplitMix64 output function (Steele, Lea, Flood 2014; Vigna's splitmix64.c):
 * the n-th output of a stream with initial state s is mix(s + n * GAMMA). */
uint64_t orc_sm64_mix(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
    return z ^ (z >> 31);
}

/* n-th output (n >= 1) of the SplitMix64 stream whose initial state is s. */
uint64_t orc_sm64_nth(uint64_t s, uint64_t n)
{
    return orc_sm64_mix(s + n * ORC_GAMMA);
}

/* Stream key of one tensor: three chained SplitMix64 steps over
 * (seed, model tag, tensor id). */
uint64_t orc_stream_key(uint64_t seed, uint32_t tag, uint32_t tid)
{
    uint64_t a = orc_sm64_mix(seed + ORC_GAMMA);
    uint64_t b = orc_sm64_mix(a + ORC_GAMMA + (uint64_t)tag);
    return orc_sm64_mix(b + ORC_GAMMA + (uint64_t)tid);
}

/* float -> nearest bf16 (ties to even), returned widened back to float. */
float orc_round_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return f;
}

/* Element idx of the stream with key K: outputs 3*idx+1 .. 3*idx+3 of the
 * stream give twelve 16-bit uniforms; their sum S is Irwin-Hall(12) on an
 * integer grid with mean 6*65535 and standard deviation ~65536, so
 * z = (S - 6*65535) / 65536 is approximately N(0,1) (tails end at +-6).
 * The weight is bf16(0.02f * z): the N(0, 0.02) initialisation. */
float orc_weight_value(uint64_t K, uint64_t idx)
{
    uint32_t S = 0;
    for (int lane = 0; lane < 3; ++lane) {
        uint64_t r = orc_sm64_nth(K, 3 * idx + (uint64_t)lane + 1);
        S += (uint32_t)(r & 0xffff) + (uint32_t)((r >> 16) & 0xffff) +
             (uint32_t)((r >> 32) & 0xffff) + (uint32_t)((r >> 48) & 0xffff);
    }
    float z = (float)((int32_t)S - 6 * 65535) / 65536.0f;
    return orc_round_bf16(0.02f * z);
}

void orc_fill_tensor(uint64_t seed, uint32_t tag, uint32_t tid, uint64_t idx0, uint64_t n, float *out)
{
    uint64_t K = orc_stream_key(seed, tag, tid);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) out[i] = orc_weight_value(K, idx0 + (uint64_t)i);
}

/* ------------------------------------------------------------------------- */
/* Model                                                                      */
/* ------------------------------------------------------------------------- */

typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    double rope_theta, rms_eps;
    int32_t tie_embeddings, qkv_bias;
} orc_config;

/* Tensor ids.  Gains (norm weights) are all ones and are not drawn. */
enum { T_EMBED = 0, T_LMHEAD = 1 };
enum { T_WQ = 1, T_WK = 2, T_WV = 3, T_BQ = 4, T_BK = 5, T_BV = 6, T_WO = 7, T_WG = 9, T_WU = 10, T_WD = 11 };
static uint32_t layer_tid(int layer, int which) { return 16u * (uint32_t)(layer + 1) + (uint32_t)which; }

#define ORC_MAX_TENSORS (16 * 130)

typedef struct {
    orc_config c;
    uint64_t seed;
    uint32_t tag;
    /* Optional explicit tensors (materialised or set by a test); NULL means
     * "generate element (tid, idx) from the seeded stream when needed". */
    float *tensor[ORC_MAX_TENSORS];
    double *gain[ORC_MAX_TENSORS]; /* norm gains; NULL = ones */
} orc_model;

static uint64_t tensor_numel(const orc_config *c, uint32_t tid)
{
    uint64_t h = c->hidden, qd = (uint64_t)c->n_q_heads * c->head_dim, kd = (uint64_t)c->n_kv_heads * c->head_dim;
    if (tid == T_EMBED || tid == T_LMHEAD) return (uint64_t)c->vocab * h;
    switch (tid % 16) {
    case T_WQ: return qd * h;
    case T_WK: case T_WV: return kd * h;
    case T_BQ: return qd;
    case T_BK: case T_BV: return kd;
    case T_WO: return h * qd;
    case T_WG: case T_WU: return (uint64_t)c->ffn * h;
    case T_WD: return h * (uint64_t)c->ffn;
    }
    return 0;
}

orc_model *orc_model_create(const orc_config *c, uint64_t seed, uint32_t tag, int materialize)
{
    if (c->n_layers < 1 || c->n_layers > 128 || c->n_q_heads % c->n_kv_heads != 0 || (c->head_dim & 1)) return NULL;
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    if (!m) return NULL;
    m->c = *c;
    m->seed = seed;
    m->tag = tag;
    if (materialize) {
        static const int which[] = {T_WQ, T_WK, T_WV, T_BQ, T_BK, T_BV, T_WO, T_WG, T_WU, T_WD};
        uint32_t tids[2 + 10 * 128];
        int nt = 0;
        tids[nt++] = T_EMBED;
        if (!c->tie_embeddings) tids[nt++] = T_LMHEAD;
        for (int l = 0; l < c->n_layers; ++l)
            for (int w = 0; w < 10; ++w) tids[nt++] = layer_tid(l, which[w]);
        for (int t = 0; t < nt; ++t) {
            uint64_t n = tensor_numel(c, tids[t]);
            float *p = (float *)malloc(n * sizeof(float));
            if (!p) return NULL;
            orc_fill_tensor(seed, tag, tids[t], 0, n, p);
            m->tensor[tids[t]] = p;
        }
    }
    return m;
}

void orc_model_destroy(orc_model *m)
{
    if (!m) return;
    for (int i = 0; i < ORC_MAX_TENSORS; ++i) { free(m->tensor[i]); free(m->gain[i]); }
    free(m);
}

/* Test hook: replace a tensor by explicit values (copied).  layer < 0 selects
 * the embedding (which 0) or LM head (which 1). */
int orc_model_set_tensor(orc_model *m, int layer, int which, const float *data, uint64_t n)
{
    uint32_t tid = layer < 0 ? (uint32_t)which : layer_tid(layer, which);
    if (tensor_numel(&m->c, tid) != n) return -1;
    float *p = (float *)malloc(n * sizeof(float));
    memcpy(p, data, n * sizeof(float));
    free(m->tensor[tid]);
    m->tensor[tid] = p;
    return 0;
}

/* Test hook: set a norm gain vector.  which: 0 = input norm, 8 = post-attention
 * norm of `layer`; layer < 0 = final norm. */
int orc_model_set_gain(orc_model *m, int layer, int which, const double *g)
{
    uint32_t tid = layer < 0 ? 2u : layer_tid(layer, which);
    double *p = (double *)malloc((size_t)m->c.hidden * sizeof(double));
    memcpy(p, g, (size_t)m->c.hidden * sizeof(double));
    free(m->gain[tid]);
    m->gain[tid] = p;
    return 0;
}

/* Row r (k values) of tensor tid into buf; returns a pointer to the row. */
static const float *tensor_row(const orc_model *m, uint32_t tid, uint64_t r, uint64_t k, float *buf)
{
    if (m->tensor[tid]) return m->tensor[tid] + r * k;
    uint64_t K = orc_stream_key(m->seed, m->tag, tid);
    for (uint64_t j = 0; j < k; ++j) buf[j] = orc_weight_value(K, r * k + j);
    return buf;
}

/* Y[i][r] = sum_j W[r][j] * X[i][j] (+ b[r]) for i < rows: the plain
 * definition of a linear layer; W is tensor tid with shape [n][k]. */
static void linear(const orc_model *m, uint32_t tid, int64_t n, int64_t k, uint32_t bias_tid, int use_bias,
                   const double *X, int rows, double *Y)
{
    float *bias = NULL, *bbuf = NULL;
    if (use_bias) {
        bbuf = (float *)malloc((size_t)n * sizeof(float));
        const float *b = tensor_row(m, bias_tid, 0, (uint64_t)n, bbuf);
        bias = (float *)malloc((size_t)n * sizeof(float));
        memcpy(bias, b, (size_t)n * sizeof(float));
    }
#pragma omp parallel
    {
        float *buf = (float *)malloc((size_t)k * sizeof(float));
#pragma omp for schedule(static)
        for (int64_t r = 0; r < n; ++r) {
            const float *w = tensor_row(m, tid, (uint64_t)r, (uint64_t)k, buf);
            for (int i = 0; i < rows; ++i) {
                const double *x = X + (int64_t)i * k;
                double acc = 0.0;
                for (int64_t j = 0; j < k; ++j) acc += (double)w[j] * x[j];
                if (bias) acc += (double)bias[r];
                Y[(int64_t)i * n + r] = acc;
            }
        }
        free(buf);
    }
    free(bias);
    free(bbuf);
}

/* RMSNorm: y_i = x_i * g_i / sqrt(mean_j x_j^2 + eps). */
void orc_rmsnorm(const double *x, const double *g, int n, double eps, double *y)
{
    double ss = 0.0;
    for (int i = 0; i < n; ++i) ss += x[i] * x[i];
    double inv = 1.0 / sqrt(ss / (double)n + eps);
    for (int i = 0; i < n; ++i) y[i] = x[i] * inv * (g ? g[i] : 1.0);
}

/* Rotary embedding of one head vector (length d) at position pos, half-split
 * pairing: (x_i, x_{i+d/2}) is rotated by the angle pos * theta^(-2i/d). */
void orc_rope(double *x, int d, int64_t pos, double theta)
{
    int half = d / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)pos * pow(theta, -2.0 * (double)i / (double)d);
        double c = cos(ang), s = sin(ang);
        double a = x[i], b = x[i + half];
        x[i] = a * c - b * s;
        x[i + half] = b * c + a * s;
    }
}

double orc_silu(double z) { return z / (1.0 + exp(-z)); }

/* Softmax attention of one query over n keys/values of width d:
 * out = sum_t softmax_t(q.k_t / sqrt(d)) v_t.  k and v rows are `stride`
 * doubles apart. */
void orc_attend(const double *q, const double *k, const double *v, int64_t n, int d, int64_t stride, double *out)
{
    double *p = (double *)malloc((size_t)n * sizeof(double));
    double mx = -INFINITY, scale = 1.0 / sqrt((double)d);
    for (int64_t t = 0; t < n; ++t) {
        double s = 0.0;
        for (int j = 0; j < d; ++j) s += q[j] * k[t * stride + j];
        p[t] = s * scale;
        if (p[t] > mx) mx = p[t];
    }
    double den = 0.0;
    for (int64_t t = 0; t < n; ++t) { p[t] = exp(p[t] - mx); den += p[t]; }
    for (int j = 0; j < d; ++j) out[j] = 0.0;
    for (int64_t t = 0; t < n; ++t) {
        double w = p[t] / den;
        for (int j = 0; j < d; ++j) out[j] += w * v[t * stride + j];
    }
    free(p);
}

/* ------------------------------------------------------------------------- */
/* KV cache and the cached forward pass                                       */
/* ------------------------------------------------------------------------- */

typedef struct {
    int64_t cap, len;
    int n_layers;
    int64_t width; /* n_kv_heads * head_dim */
    double *k, *v; /* [layer][pos][width]; k is stored rotated */
} orc_kv;

orc_kv *orc_kv_create(const orc_model *m, int64_t cap)
{
    orc_kv *kv = (orc_kv *)calloc(1, sizeof(orc_kv));
    kv->cap = cap;
    kv->n_layers = m->c.n_layers;
    kv->width = (int64_t)m->c.n_kv_heads * m->c.head_dim;
    size_t n = (size_t)kv->n_layers * (size_t)cap * (size_t)kv->width;
    kv->k = (double *)calloc(n, sizeof(double));
    kv->v = (double *)calloc(n, sizeof(double));
    if (!kv->k || !kv->v) return NULL;
    return kv;
}
void orc_kv_destroy(orc_kv *kv) { if (kv) { free(kv->k); free(kv->v); free(kv); } }
int64_t orc_kv_len(const orc_kv *kv) { return kv->len; }
void orc_kv_truncate(orc_kv *kv, int64_t n) { if (n < kv->len) kv->len = n; }

static void embed_rows(const orc_model *m, const int32_t *tokens, int rows, double *X)
{
    int h = m->c.hidden;
    float *buf = (float *)malloc((size_t)h * sizeof(float));
    for (int i = 0; i < rows; ++i) {
        const float *e = tensor_row(m, T_EMBED, (uint64_t)tokens[i], (uint64_t)h, buf);
        for (int j = 0; j < h; ++j) X[(int64_t)i * h + j] = (double)e[j];
    }
    free(buf);
}

/* logits_i = W_lm . rmsnorm(x_i) for the rows selected (all, or last only). */
static void lm_head(const orc_model *m, const double *X, int rows, int all_rows, double *logits)
{
    const orc_config *c = &m->c;
    int h = c->hidden;
    int first = all_rows ? 0 : rows - 1, cnt = rows - first;
    double *xn = (double *)malloc((size_t)cnt * h * sizeof(double));
    for (int i = 0; i < cnt; ++i) orc_rmsnorm(X + (int64_t)(first + i) * h, m->gain[2], h, c->rms_eps, xn + (int64_t)i * h);
    linear(m, c->tie_embeddings ? T_EMBED : T_LMHEAD, c->vocab, h, 0, 0, xn, cnt, logits);
    free(xn);
}

/* Feed `rows` new tokens at positions kv->len .. kv->len+rows-1.  Each new
 * position attends to every cached position and to the new positions up to
 * and including itself.  logits: [rows][vocab] if all_rows, else [vocab] for
 * the last fed position; may be NULL.  Returns 0, or -1 when the cache is
 * too small. */
static int forward_rows(const orc_model *m, orc_kv *kv, const int32_t *tokens, int rows, int all_rows, double *logits, int skip_unread)
{
    const orc_config *c = &m->c;
    int h = c->hidden, d = c->head_dim, Hq = c->n_q_heads, Hkv = c->n_kv_heads, f = c->ffn;
    int qd = Hq * d, kd = Hkv * d, grp = Hq / Hkv;
    if (rows < 1 || kv->len + rows > kv->cap) return -1;
    int64_t p0 = kv->len;
    double *X = (double *)malloc((size_t)rows * h * sizeof(double));
    double *XN = (double *)malloc((size_t)rows * h * sizeof(double));
    double *Q = (double *)malloc((size_t)rows * qd * sizeof(double));
    double *Kn = (double *)malloc((size_t)rows * kd * sizeof(double));
    double *Vn = (double *)malloc((size_t)rows * kd * sizeof(double));
    double *A = (double *)malloc((size_t)rows * qd * sizeof(double));
    double *D = (double *)malloc((size_t)rows * h * sizeof(double));
    double *G = (double *)malloc((size_t)rows * f * sizeof(double));
    double *U = (double *)malloc((size_t)rows * f * sizeof(double));
    embed_rows(m, tokens, rows, X);
    for (int l = 0; l < c->n_layers; ++l) {
        double *kl = kv->k + (size_t)l * kv->cap * kd, *vl = kv->v + (size_t)l * kv->cap * kd;
        /* r0: first row whose attention / FFN result anything reads.  Keys and values are needed for every
         * row; with skip_unread the last layer's remaining work is done for the last row only (the only row
         * the returned logits depend on). */
        int r0 = (skip_unread && !all_rows && l == c->n_layers - 1) ? rows - 1 : 0;
        int nr = rows - r0;
        for (int i = 0; i < rows; ++i) orc_rmsnorm(X + (int64_t)i * h, m->gain[layer_tid(l, 0)], h, c->rms_eps, XN + (int64_t)i * h);
        linear(m, layer_tid(l, T_WQ), qd, h, layer_tid(l, T_BQ), c->qkv_bias, XN + (int64_t)r0 * h, nr, Q + (int64_t)r0 * qd);
        linear(m, layer_tid(l, T_WK), kd, h, layer_tid(l, T_BK), c->qkv_bias, XN, rows, Kn);
        linear(m, layer_tid(l, T_WV), kd, h, layer_tid(l, T_BV), c->qkv_bias, XN, rows, Vn);
        for (int i = 0; i < rows; ++i) {
            if (i >= r0)
                for (int hq = 0; hq < Hq; ++hq) orc_rope(Q + (int64_t)i * qd + hq * d, d, p0 + i, c->rope_theta);
            for (int hk = 0; hk < Hkv; ++hk) orc_rope(Kn + (int64_t)i * kd + hk * d, d, p0 + i, c->rope_theta);
            memcpy(kl + (p0 + i) * kd, Kn + (int64_t)i * kd, (size_t)kd * sizeof(double));
            memcpy(vl + (p0 + i) * kd, Vn + (int64_t)i * kd, (size_t)kd * sizeof(double));
        }
#pragma omp parallel for collapse(2) schedule(dynamic)
        for (int i = r0; i < rows; ++i)
            for (int hq = 0; hq < Hq; ++hq) {
                int hk = hq / grp; /* consecutive q heads share a kv head */
                orc_attend(Q + (int64_t)i * qd + hq * d, kl + hk * d, vl + hk * d, p0 + i + 1, d, kd, A + (int64_t)i * qd + hq * d);
            }
        linear(m, layer_tid(l, T_WO), h, qd, 0, 0, A + (int64_t)r0 * qd, nr, D + (int64_t)r0 * h);
        for (int64_t i = (int64_t)r0 * h; i < (int64_t)rows * h; ++i) X[i] += D[i];
        for (int i = r0; i < rows; ++i) orc_rmsnorm(X + (int64_t)i * h, m->gain[layer_tid(l, 8)], h, c->rms_eps, XN + (int64_t)i * h);
        linear(m, layer_tid(l, T_WG), f, h, 0, 0, XN + (int64_t)r0 * h, nr, G + (int64_t)r0 * f);
        linear(m, layer_tid(l, T_WU), f, h, 0, 0, XN + (int64_t)r0 * h, nr, U + (int64_t)r0 * f);
        for (int64_t i = (int64_t)r0 * f; i < (int64_t)rows * f; ++i) G[i] = orc_silu(G[i]) * U[i];
        linear(m, layer_tid(l, T_WD), h, f, 0, 0, G + (int64_t)r0 * f, nr, D + (int64_t)r0 * h);
        for (int64_t i = (int64_t)r0 * h; i < (int64_t)rows * h; ++i) X[i] += D[i];
    }
    kv->len += rows;
    if (logits) lm_head(m, X, rows, all_rows, logits);
    free(X); free(XN); free(Q); free(Kn); free(Vn); free(A); free(D); free(G); free(U);
    return 0;
}

int orc_forward(const orc_model *m, orc_kv *kv, const int32_t *tokens, int rows, int all_rows, double *logits)
{
    return forward_rows(m, kv, tokens, rows, all_rows, logits, 0);
}

/* The same pass with the work nothing reads left out: when only the last row's logits are returned, the last
 * layer's attention, output projection and FFN are evaluated for that row alone (keys and values are still stored
 * for every row).  No result changes; long contexts get affordable (a one-layer model's pass becomes linear in
 * the number of rows).  Pinned to orc_forward by equality in tests/test_oracle_model.py. */
int orc_forward_last(const orc_model *m, orc_kv *kv, const int32_t *tokens, int rows, double *logits)
{
    return forward_rows(m, kv, tokens, rows, 0, logits, 1);
}

/* Full recompute without any cache: the reference definition of the causal
 * transformer.  Attention is written with an explicit [p][p] score matrix per
 * head, masked above the diagonal.  logits: [p][vocab]. */
int orc_forward_full(const orc_model *m, const int32_t *tokens, int p, double *logits)
{
    const orc_config *c = &m->c;
    int h = c->hidden, d = c->head_dim, Hq = c->n_q_heads, Hkv = c->n_kv_heads, f = c->ffn;
    int qd = Hq * d, kd = Hkv * d, grp = Hq / Hkv;
    double *X = (double *)malloc((size_t)p * h * sizeof(double));
    double *XN = (double *)malloc((size_t)p * h * sizeof(double));
    double *Q = (double *)malloc((size_t)p * qd * sizeof(double));
    double *K = (double *)malloc((size_t)p * kd * sizeof(double));
    double *V = (double *)malloc((size_t)p * kd * sizeof(double));
    double *A = (double *)malloc((size_t)p * qd * sizeof(double));
    double *D = (double *)malloc((size_t)p * h * sizeof(double));
    double *G = (double *)malloc((size_t)p * f * sizeof(double));
    double *U = (double *)malloc((size_t)p * f * sizeof(double));
    double *S = (double *)malloc((size_t)p * p * sizeof(double));
    embed_rows(m, tokens, p, X);
    for (int l = 0; l < c->n_layers; ++l) {
        for (int i = 0; i < p; ++i) orc_rmsnorm(X + (int64_t)i * h, m->gain[layer_tid(l, 0)], h, c->rms_eps, XN + (int64_t)i * h);
        linear(m, layer_tid(l, T_WQ), qd, h, layer_tid(l, T_BQ), c->qkv_bias, XN, p, Q);
        linear(m, layer_tid(l, T_WK), kd, h, layer_tid(l, T_BK), c->qkv_bias, XN, p, K);
        linear(m, layer_tid(l, T_WV), kd, h, layer_tid(l, T_BV), c->qkv_bias, XN, p, V);
        for (int i = 0; i < p; ++i) {
            for (int hq = 0; hq < Hq; ++hq) orc_rope(Q + (int64_t)i * qd + hq * d, d, i, c->rope_theta);
            for (int hk = 0; hk < Hkv; ++hk) orc_rope(K + (int64_t)i * kd + hk * d, d, i, c->rope_theta);
        }
        for (int hq = 0; hq < Hq; ++hq) {
            int hk = hq / grp;
            for (int i = 0; i < p; ++i)
                for (int t = 0; t < p; ++t) {
                    double s = 0.0;
                    for (int j = 0; j < d; ++j) s += Q[(int64_t)i * qd + hq * d + j] * K[(int64_t)t * kd + hk * d + j];
                    S[(int64_t)i * p + t] = t <= i ? s / sqrt((double)d) : -INFINITY;
                }
            for (int i = 0; i < p; ++i) {
                double mx = -INFINITY, den = 0.0;
                for (int t = 0; t < p; ++t) if (S[(int64_t)i * p + t] > mx) mx = S[(int64_t)i * p + t];
                for (int t = 0; t < p; ++t) { S[(int64_t)i * p + t] = exp(S[(int64_t)i * p + t] - mx); den += S[(int64_t)i * p + t]; }
                for (int j = 0; j < d; ++j) {
                    double o = 0.0;
                    for (int t = 0; t < p; ++t) o += S[(int64_t)i * p + t] / den * V[(int64_t)t * kd + hk * d + j];
                    A[(int64_t)i * qd + hq * d + j] = o;
                }
            }
        }
        linear(m, layer_tid(l, T_WO), h, qd, 0, 0, A, p, D);
        for (int64_t i = 0; i < (int64_t)p * h; ++i) X[i] += D[i];
        for (int i = 0; i < p; ++i) orc_rmsnorm(X + (int64_t)i * h, m->gain[layer_tid(l, 8)], h, c->rms_eps, XN + (int64_t)i * h);
        linear(m, layer_tid(l, T_WG), f, h, 0, 0, XN, p, G);
        linear(m, layer_tid(l, T_WU), f, h, 0, 0, XN, p, U);
        for (int64_t i = 0; i < (int64_t)p * f; ++i) G[i] = orc_silu(G[i]) * U[i];
        linear(m, layer_tid(l, T_WD), h, f, 0, 0, G, p, D);
        for (int64_t i = 0; i < (int64_t)p * h; ++i) X[i] += D[i];
    }
    lm_head(m, X, p, 1, logits);
    free(X); free(XN); free(Q); free(K); free(V); free(A); free(D); free(G); free(U); free(S);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Greedy sampler                                                             */
/* ------------------------------------------------------------------------- */

/* Lowest-id argmax over ids < limit; also the gap to the runner-up. */
int32_t orc_argmax(const double *z, int32_t limit, double *margin)
{
    int32_t best = 0;
    double second = -INFINITY;
    for (int32_t i = 1; i < limit; ++i) {
        if (z[i] > z[best]) { second = z[best]; best = i; }
        else if (z[i] > second) second = z[i];
    }
    if (margin) *margin = z[best] - second;
    return best;
}

/* Temperature sampling by the Gumbel-max rule (Gumbel 1954; Maddison, Tarlow, Minka 2014): with independent
 * standard Gumbel variates g_i, argmax_i (z_i / T + g_i) is distributed as softmax(z / T).  The variates come from a
 * counter-based generator so that any implementation can reproduce them: u is built from the top 23 bits k of the
 * SplitMix64 output number (step * 2^32 + i + 1) of the stream with initial state `seed`, u = (k + 0.5) * 2^-23 (so
 * 0 < u < 1, exactly representable in single and double precision), and g = -ln(-ln u).  Lowest id on ties; *margin
 * (optional) is the gap between the two largest perturbed values.  temperature <= 0 is plain greedy. */
double orc_gumbel(uint64_t seed, uint32_t step, uint32_t i)
{
    uint64_t x = orc_sm64_nth(seed, (((uint64_t)step << 32) | (uint64_t)i) + 1);
    double u = ((double)(x >> 41) + 0.5) * (1.0 / 8388608.0);
    return -log(-log(u));
}

int32_t orc_sample(const double *z, int32_t limit, double temperature, uint64_t seed, uint32_t step, double *margin)
{
    if (!(temperature > 0.0)) return orc_argmax(z, limit, margin);
    int32_t best = 0;
    double vbest = z[0] / temperature + orc_gumbel(seed, step, 0), second = -INFINITY;
    for (int32_t i = 1; i < limit; ++i) {
        double v = z[i] / temperature + orc_gumbel(seed, step, (uint32_t)i);
        if (v > vbest) { second = vbest; vbest = v; best = i; }
        else if (v > second) second = v;
    }
    if (margin) *margin = vbest - second;
    return best;
}

/* Nucleus (top-p) of softmax(z / T) (Holtzman et al. 2020): order the ids by probability, largest first; the nucleus
 * is the shortest prefix whose probabilities sum to at least top_p, and -- so that the set does not depend on how
 * equal probabilities are ordered -- every id that ties with the prefix's last member.  Returns the logit of that last
 * member: the nucleus is { i : z[i] >= threshold }.  *gap (optional) is the distance between top_p and the nearest of
 * the two cumulative sums around the cut (the sum that reaches top_p and the one before it): a cut with a small gap
 * may fall differently in lower precision.  The paper names no sampler; this is the standard definition written out
 * (the ids sorted with the C library's qsort, sums in double precision). */
typedef struct { double z; int32_t id; } orc_zid;
static int orc_zid_desc(const void *a, const void *b)   /* larger logit first, lower id first among equals */
{
    const orc_zid *x = (const orc_zid *)a, *y = (const orc_zid *)b;
    if (x->z != y->z) return x->z > y->z ? -1 : 1;
    return x->id < y->id ? -1 : x->id > y->id;
}
double orc_nucleus_threshold(const double *z, int32_t limit, double temperature, double top_p, double *gap)
{
    double zmax = z[0], Z = 0.0;
    for (int32_t i = 1; i < limit; ++i) if (z[i] > zmax) zmax = z[i];
    for (int32_t i = 0; i < limit; ++i) Z += exp((z[i] - zmax) / temperature);
    orc_zid *order = (orc_zid *)malloc((size_t)limit * sizeof(orc_zid));
    for (int32_t i = 0; i < limit; ++i) { order[i].z = z[i]; order[i].id = i; }
    qsort(order, (size_t)limit, sizeof(orc_zid), orc_zid_desc);
    double cum = 0.0, thr = zmax, before = 0.0;
    for (int32_t k = 0; k < limit; ++k) {
        before = cum;
        cum += exp((order[k].z - zmax) / temperature) / Z;
        thr = order[k].z;
        if (cum >= top_p) break;
    }
    free(order);
    if (gap) {
        double a = fabs(cum - top_p), b = fabs(top_p - before);
        *gap = a < b ? a : b;
    }
    return thr;
}

/* Top-p sampling: the Gumbel-max draw of orc_sample restricted to the nucleus (ids outside it cannot win), which is
 * a draw from softmax(z / T) renormalised over the nucleus.  top_p <= 0 or >= 1: no restriction. */
int32_t orc_sample_top_p(const double *z, int32_t limit, double temperature, double top_p, uint64_t seed, uint32_t step,
                         double *margin, double *gap)
{
    if (gap) *gap = 1.0;
    if (!(temperature > 0.0) || !(top_p > 0.0) || top_p >= 1.0) return orc_sample(z, limit, temperature, seed, step, margin);
    const double thr = orc_nucleus_threshold(z, limit, temperature, top_p, gap);
    int32_t best = -1;
    double vbest = -INFINITY, second = -INFINITY;
    for (int32_t i = 0; i < limit; ++i) {
        if (z[i] < thr) continue;
        double v = z[i] / temperature + orc_gumbel(seed, step, (uint32_t)i);
        if (best < 0 || v > vbest) { second = vbest; vbest = v; best = i; }
        else if (v > second) second = v;
    }
    if (margin) *margin = vbest - second;
    return best;
}

/* ------------------------------------------------------------------------- */
/* Speculative Thinking generation (Section 3, takeover (1))                  */
/* ------------------------------------------------------------------------- */

typedef struct {
    int32_t delimiter_id;
    const int32_t *keyword_ids;
    int32_t n_keywords;
    int32_t n1;          /* tokens the target writes per takeover (paper: 20) */
    int32_t keep_probe;  /* 0: the target's segment replaces the probe token; 1: probe kept */
    int32_t eos_id;      /* -1: none */
    int32_t vocab_limit; /* sample over ids < vocab_limit */
    int32_t max_new_tokens;
    /* Variant for a speculative model without reflective cues (Section "Reasoning Models Monitor
     * Non-Reasoning Models", paragraph "Modification ..."): */
    int32_t takeover_every_delimiter; /* 1: no keyword test; the target writes the n1 tokens after every
                                         delimiter the speculative model writes */
    int32_t target_first_n;           /* > 0: the target writes the first target_first_n tokens (paper: 100) */
    /* Section 3, takeovers (1)-(3) in token-id form (the token sampled right after a delimiter stands for
     * the sentence that follows it).  All off when the sets are empty and neg_threshold < 0. */
    const int32_t *affirmation_ids;   /* (1): an affirmation cue hands over n1 tokens like a reflection cue */
    int32_t n_affirmation;
    const int32_t *verification_ids;  /* (2): a verification cue after a delimiter, whoever samples it: n2 target tokens */
    int32_t n_verification;
    int32_t n2;                       /* paper: 125 */
    int32_t neg_threshold;            /* (3): once more than this many reflection cues were sampled by the speculative
                                         model (paper: 15), aux_ids are inserted and the target writes n3 tokens; < 0: off */
    int32_t n3;                       /* paper: 125 */
    const int32_t *aux_ids;           /* the auxiliary sentence of (3) */
    int32_t n_aux;
    int32_t probe_len;                /* tokens of the speculative model's sentence after a delimiter that are classified
                                         (paper: "one full sentence (i.e. n1 tokens)"); <= 1: only its first token */
    /* The delimiter as a family of ids (the paper's Table 1 / Appendix B: any token ending in a blank line closes a
     * paragraph).  n_delimiters == 0: delimiter_id alone; otherwise delimiter_id is ignored. */
    const int32_t *delimiter_ids;
    int32_t n_delimiters;
    /* Sampling (the paper reports pass@1 and names no sampler; greedy is the default here): temperature > 0 draws
     * every token by orc_sample with this seed and the emission step as the counter. */
    double temperature;
    uint64_t sample_seed;
    double top_p;        /* 0 < top_p < 1: every draw is restricted to the nucleus (orc_sample_top_p) */
} orc_spec_params;

/* Does this token close a paragraph? */
static int is_delimiter(const orc_spec_params *P, int32_t tok)
{
    if (P->n_delimiters <= 0) return tok == P->delimiter_id;
    for (int i = 0; i < P->n_delimiters; ++i)
        if (P->delimiter_ids[i] == tok) return 1;
    return 0;
}

typedef struct { int32_t seg_start, step, catchup_len; } orc_handoff;

typedef struct {
    int32_t *tokens;            /* [cap_tokens] tokens written after the prompt */
    uint8_t *source;            /* [cap_tokens] 0 = speculative (small), 1 = target (large) */
    int32_t cap_tokens, n_tokens;
    orc_handoff *handoffs;
    int32_t cap_handoffs, n_handoffs;
    int32_t *emission_tokens;   /* [cap_steps] every token sampled or forced, discarded probes included */
    uint8_t *emission_source;   /* [cap_steps] */
    int32_t *emission_fed;      /* [cap_steps] how many tokens the emitting model ingested at this step */
    int32_t *emission_argmax;   /* [cap_steps] the greedy choice before forcing */
    double *emission_margin;    /* [cap_steps] top-1 minus top-2 logit */
    int32_t cap_steps, n_steps;
    int32_t kv_len_small, kv_len_large;
    double *logits_trace;       /* optional [trace_n_steps][vocab_limit] */
    int32_t trace_first_step, trace_n_steps;
    uint8_t *handoff_kinds;     /* optional [cap_handoffs]: 1 reflection/affirmation, 2 verification, 3 excessive reflection */
} orc_spec_result;

/* The speculative model writes until it samples a reflection keyword right
 * after a delimiter; the target then writes n1 tokens and control returns.
 * Each model ingests the tokens it has not seen yet (its catch-up prefill)
 * the next time it is asked for a token.  force[t] >= 0 replaces the token
 * sampled at emission step t.  large may be NULL (plain decode). */
int orc_generate_spec(const orc_model *small, const orc_model *large, const orc_spec_params *P,
                      const int32_t *prompt, int32_t prompt_len, const int32_t *force, int32_t n_force,
                      orc_spec_result *R)
{
    if (prompt_len < 1 || P->max_new_tokens < 0) return -1;
    if ((P->n_verification > 0 && P->n2 < 1) || (P->neg_threshold >= 0 && P->n3 < 1)) return -1;
    int64_t cap = (int64_t)prompt_len + P->max_new_tokens + 1;
    const orc_model *M[2] = {small, large};
    orc_kv *kv[2] = {orc_kv_create(small, cap), large ? orc_kv_create(large, cap) : NULL};
    int32_t *tokens = (int32_t *)malloc((size_t)cap * sizeof(int32_t));
    memcpy(tokens, prompt, (size_t)prompt_len * sizeof(int32_t));
    int vmax = small->c.vocab;
    if (large && large->c.vocab > vmax) vmax = large->c.vocab;
    double *z = (double *)malloc((size_t)vmax * sizeof(double));
    int active = 0, remaining = 0, rc = 0, neg_count = 0;
    int probing = 0, probe_n = 0, n_refl = 0, n_aff = 0, n_ver = 0;
    int32_t probe_start = 0;
    int32_t pos = prompt_len, t = 0, generated = 0;
    R->n_tokens = R->n_handoffs = R->n_steps = 0;
    if (large && P->target_first_n > 0) {   /* the target opens the answer */
        active = 1;
        remaining = P->target_first_n;
    }
    while (generated < P->max_new_tokens) {
        int a = active;
        int32_t fed = pos - (int32_t)kv[a]->len;
        if (orc_forward(M[a], kv[a], tokens + kv[a]->len, fed, 0, z) != 0) { rc = -2; break; }
        double margin;
        int32_t greedy = orc_sample_top_p(z, P->vocab_limit, P->temperature, P->top_p, P->sample_seed, (uint32_t)t, &margin, NULL);
        int32_t tok = (force && t < n_force && force[t] >= 0) ? force[t] : greedy;
        if (t >= R->cap_steps) { rc = -3; break; }
        R->emission_tokens[t] = tok;
        R->emission_source[t] = (uint8_t)a;
        if (R->emission_fed) R->emission_fed[t] = fed;
        if (R->emission_argmax) R->emission_argmax[t] = greedy;
        if (R->emission_margin) R->emission_margin[t] = margin;
        if (R->logits_trace && t >= R->trace_first_step && t < R->trace_first_step + R->trace_n_steps)
            memcpy(R->logits_trace + (size_t)(t - R->trace_first_step) * P->vocab_limit, z, (size_t)P->vocab_limit * sizeof(double));
        ++t;
        R->n_steps = t;
        int is_kw = 0, is_aff = 0, is_ver = 0;
        for (int i = 0; i < P->n_keywords; ++i) is_kw |= (P->keyword_ids[i] == tok);
        for (int i = 0; i < P->n_affirmation; ++i) is_aff |= (P->affirmation_ids[i] == tok);
        for (int i = 0; i < P->n_verification; ++i) is_ver |= (P->verification_ids[i] == tok);
        const int after_delim = is_delimiter(P, tokens[pos - 1]);
        if (large && a == 0 && !P->takeover_every_delimiter && !probing && after_delim) {
            /* the speculative model opens a sentence: its next probe_len tokens are classified by cue counts */
            probing = 1;
            probe_start = pos;
            probe_n = n_refl = n_aff = n_ver = 0;
        }
        if (probing) {
            n_refl += is_kw; n_aff += is_aff; n_ver += is_ver;
            ++probe_n;
        }
        if (probing && probe_n >= (P->probe_len > 1 ? P->probe_len : 1)) {
            probing = 0;
            /* Affirmation and Reflection cues in one sentence: the majority decides, a tie is a Reflection */
            const int reflection = n_refl > 0 && n_refl >= n_aff;
            if (reflection && P->neg_threshold >= 0) ++neg_count;
            int kind = 0, len = 0;
            if (P->neg_threshold >= 0 && neg_count > P->neg_threshold) { kind = 3; len = P->n3; }   /* (3) */
            else if (n_ver > 0) { kind = 2; len = P->n2; }                                          /* (2) */
            else if (n_refl + n_aff > 0) { kind = 1; len = P->n1; }                                 /* (1) */
            if (kind) {
                int stop = 0;
                if (P->keep_probe) {
                    if (generated >= R->cap_tokens) { rc = -3; break; }
                    tokens[pos] = tok;
                    R->tokens[generated] = tok;
                    R->source[generated] = 0;
                    ++pos; ++generated;
                    R->n_tokens = generated;
                    if (tok == P->eos_id) stop = 1;
                } else {
                    /* the target's segment replaces the whole probe sentence: the speculative model's cache
                     * and the output go back to where the sentence began */
                    generated -= pos - probe_start;
                    pos = probe_start;
                    kv[0]->len = probe_start;
                    R->n_tokens = generated;
                }
                if (kind == 3) {   /* the auxiliary sentence goes into the output, then the target continues */
                    for (int i = 0; i < P->n_aux && generated < P->max_new_tokens && !stop; ++i) {
                        if (generated >= R->cap_tokens) { rc = -3; break; }
                        tokens[pos] = P->aux_ids[i];
                        R->tokens[generated] = P->aux_ids[i];
                        R->source[generated] = 2;
                        ++pos; ++generated;
                        R->n_tokens = generated;
                    }
                    if (rc) break;
                    neg_count = 0;
                }
                if (R->n_handoffs >= R->cap_handoffs) { rc = -3; break; }
                R->handoffs[R->n_handoffs].seg_start = pos;
                R->handoffs[R->n_handoffs].step = t - 1;
                R->handoffs[R->n_handoffs].catchup_len = pos - (int32_t)kv[1]->len;
                if (R->handoff_kinds) R->handoff_kinds[R->n_handoffs] = (uint8_t)kind;
                R->n_handoffs++;
                active = 1;
                remaining = len;
                if (stop) break;
                continue;
            }
        }
        if (large && a == 1 && after_delim && is_ver && remaining < P->n2) {
            /* (2) applies to the target's own sentences too: from this token on it writes n2 tokens */
            if (R->n_handoffs >= R->cap_handoffs) { rc = -3; break; }
            R->handoffs[R->n_handoffs].seg_start = pos;
            R->handoffs[R->n_handoffs].step = t - 1;
            R->handoffs[R->n_handoffs].catchup_len = 0;
            if (R->handoff_kinds) R->handoff_kinds[R->n_handoffs] = 2;
            R->n_handoffs++;
            remaining = P->n2;
        }
        if (generated >= R->cap_tokens) { rc = -3; break; }
        tokens[pos] = tok;
        R->tokens[generated] = tok;
        R->source[generated] = (uint8_t)a;
        ++pos; ++generated;
        R->n_tokens = generated;
        if (tok == P->eos_id) break;
        if (a == 1 && --remaining == 0) active = 0;
        if (large && a == 0 && P->takeover_every_delimiter && is_delimiter(P, tok) && generated < P->max_new_tokens) {
            /* the speculative model closed a paragraph: the target writes the next n1 tokens */
            if (R->n_handoffs >= R->cap_handoffs) { rc = -3; break; }
            R->handoffs[R->n_handoffs].seg_start = pos;
            R->handoffs[R->n_handoffs].step = t - 1;
            R->handoffs[R->n_handoffs].catchup_len = pos - (int32_t)kv[1]->len;
            if (R->handoff_kinds) R->handoff_kinds[R->n_handoffs] = 1;
            R->n_handoffs++;
            active = 1;
            remaining = P->n1;
        }
    }
    R->kv_len_small = (int32_t)kv[0]->len;
    R->kv_len_large = kv[1] ? (int32_t)kv[1]->len : 0;
    orc_kv_destroy(kv[0]);
    orc_kv_destroy(kv[1]);
    free(tokens);
    free(z);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* Greedy speculative decoding: the comparison system of the paper's section  */
/* "Comparisons between Speculative Decoding and Speculative Thinking"        */
/* ------------------------------------------------------------------------- */

/* The speculative model drafts gamma tokens one by one (the paper sets 20 "to match the number of intervention
 * tokens"), the target model scores the drafts in one pass and keeps the longest prefix it would have written
 * itself; the first draft it disagrees with is replaced by its own token, and when it agrees with all of them its
 * next token comes for free (Leviathan et al., "Fast inference from transformers via speculative decoding", the
 * greedy case).  Every round therefore writes (accepted drafts + 1) tokens, and the whole output equals the target
 * model's own greedy continuation.  Both caches are cut back to the accepted length after a round.
 *
 * force_draft[k] >= 0 replaces the k-th drafted token (k counts drafts over all rounds); force_target[i] >= 0
 * replaces the target's choice for the i-th generated position.  With both given the acceptance pattern is a pure
 * function of the two arrays, which is how the hand-traced pins work. */
typedef struct {
    int32_t gamma;          /* drafts per round (paper: 20) */
    int32_t eos_id;         /* -1: none */
    int32_t vocab_limit;
    int32_t max_new_tokens;
} orc_specdec_params;

typedef struct {
    int32_t *tokens;        /* [cap_tokens] */
    uint8_t *source;        /* [cap_tokens] 0 = accepted draft, 1 = written by the target */
    int32_t cap_tokens, n_tokens;
    int32_t *round_drafted, *round_accepted;   /* [cap_rounds] */
    int32_t cap_rounds, n_rounds;
    int32_t kv_len_small, kv_len_large;
    int32_t n_drafted, n_accepted;             /* totals */
    double *choice_margin;  /* optional [cap_tokens]: top-2 margin of the target's logits row that decided generated position i */
    double *draft_margin;   /* optional [cap_drafts]: top-2 margin of the speculative model's logits behind draft k */
    int32_t cap_drafts;
} orc_specdec_result;

int orc_generate_specdec(const orc_model *small, const orc_model *large, const orc_specdec_params *P,
                         const int32_t *prompt, int32_t prompt_len, const int32_t *force_draft, int32_t n_force_draft,
                         const int32_t *force_target, int32_t n_force_target, orc_specdec_result *R)
{
    if (prompt_len < 1 || P->max_new_tokens < 0 || P->gamma < 1) return -1;
    int64_t cap = (int64_t)prompt_len + P->max_new_tokens + P->gamma + 2;
    orc_kv *kvs = orc_kv_create(small, cap), *kvl = orc_kv_create(large, cap);
    int32_t *tokens = (int32_t *)malloc((size_t)cap * sizeof(int32_t));
    memcpy(tokens, prompt, (size_t)prompt_len * sizeof(int32_t));
    int vmax = small->c.vocab > large->c.vocab ? small->c.vocab : large->c.vocab;
    double *z = (double *)malloc((size_t)vmax * sizeof(double));
    double *zrows = (double *)malloc((size_t)(P->gamma + 1) * (size_t)large->c.vocab * sizeof(double));
    int32_t *draft = (int32_t *)malloc((size_t)P->gamma * sizeof(int32_t));
    int32_t pos = prompt_len, generated = 0, k_draft = 0;
    int rc = 0, stop = 0;
    R->n_tokens = R->n_rounds = R->n_drafted = R->n_accepted = 0;
    while (generated < P->max_new_tokens && !stop) {
        /* drafts: as many as the round can still use (it always ends with one token of the target) */
        int g = P->max_new_tokens - generated - 1;
        if (g > P->gamma) g = P->gamma;
        for (int i = 0; i < g; ++i) {
            /* the speculative model ingests what it lacks (the prompt, the target's last token, its previous draft) */
            int32_t fed = pos + i - (int32_t)kvs->len;
            if (orc_forward(small, kvs, tokens + kvs->len, fed, 0, z) != 0) { rc = -2; break; }
            double dm;
            int32_t d = orc_argmax(z, P->vocab_limit, &dm);
            if (force_draft && k_draft < n_force_draft && force_draft[k_draft] >= 0) d = force_draft[k_draft];
            if (R->draft_margin && k_draft < R->cap_drafts) R->draft_margin[k_draft] = dm;
            ++k_draft;
            draft[i] = d;
            tokens[pos + i] = d;   /* provisional: fed to both models, kept only if accepted */
        }
        if (rc) break;
        /* the target scores the pending tokens and all drafts in one pass; the last g + 1 rows are its choices for
         * positions pos .. pos + g */
        int32_t fed_l = pos + g - (int32_t)kvl->len;
        double *all = (double *)malloc((size_t)fed_l * (size_t)large->c.vocab * sizeof(double));
        if (orc_forward(large, kvl, tokens + kvl->len, fed_l, 1, all) != 0) { free(all); rc = -2; break; }
        memcpy(zrows, all + (size_t)(fed_l - (g + 1)) * large->c.vocab, (size_t)(g + 1) * large->c.vocab * sizeof(double));
        free(all);
        int n = 0;
        int32_t choice = 0;
        for (;;) {
            double cm;
            choice = orc_argmax(zrows + (size_t)n * large->c.vocab, P->vocab_limit, &cm);
            if (R->choice_margin && generated + n < R->cap_tokens) R->choice_margin[generated + n] = cm;
            if (force_target && generated + n < n_force_target && force_target[generated + n] >= 0) choice = force_target[generated + n];
            if (n < g && draft[n] == choice) ++n; else break;
        }
        if (R->n_rounds >= R->cap_rounds) { rc = -3; break; }
        R->round_drafted[R->n_rounds] = g;
        R->round_accepted[R->n_rounds] = n;
        R->n_rounds++;
        R->n_drafted += g;
        R->n_accepted += n;
        /* write the accepted drafts and the target's token; an end-of-sequence id ends the output where it stands */
        for (int i = 0; i <= n && !stop; ++i) {
            int32_t tok = i < n ? draft[i] : choice;
            if (generated >= R->cap_tokens) { rc = -3; stop = 1; break; }
            tokens[pos] = tok;
            R->tokens[generated] = tok;
            R->source[generated] = (uint8_t)(i < n ? 0 : 1);
            ++pos; ++generated;
            if (tok == P->eos_id) stop = 1;
        }
        R->n_tokens = generated;
        /* both caches keep the accepted prefix only (the target's own token has not been fed to anyone) */
        int32_t keep = pos - 1;
        if (kvl->len > keep) kvl->len = keep;
        if (kvs->len > keep) kvs->len = keep;
    }
    R->kv_len_small = (int32_t)kvs->len;
    R->kv_len_large = (int32_t)kvl->len;
    orc_kv_destroy(kvs);
    orc_kv_destroy(kvl);
    free(tokens); free(z); free(zrows); free(draft);
    return rc;
}
