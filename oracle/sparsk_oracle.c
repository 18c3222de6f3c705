/*
 * sparsk_oracle.c -- plain CPU decoder for SPAR-K (scheduled periodic alternating
 * early exit with deferred parallel decoding).
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be checked
 * against something written straight from the paper.  Only the test-suite, the
 * smoke check and the CPU-baseline leg of the benchmark may load it; the product
 * never does.  It shares no code, header, table or constant with the CUDA path.
 *
 * What it follows:
 *   - Sec. III: a stack of L transformer layers; h_t^(l) is the hidden state of
 *     position t after layer l; the token is read from a head applied to a hidden
 *     state (Eq. 1 for the last layer, Eq. 2 for a layer-specific head g_l).
 *   - Sec. IV-B.1: the exit schedule.  A speech chunk is cut into subgroups of K
 *     positions; one fixed position of every subgroup runs all L layers, the
 *     others leave at layer l_EE.  Text positions always run all L layers.
 *   - Sec. IV-B.3 and Algorithm 1: an early-exit step computes layers 1..l_EE,
 *     caches their K/V, keeps h^(l_EE) and marks the position as pending; the next
 *     full-depth step pushes the pending positions together with its own position
 *     through layers l_EE+1..L in one causal block, which fills their K/V, and
 *     then empties the pending set.  The token emitted at an early-exit step is
 *     never revised.
 *
 * The paper says nothing about the inside of a layer.  The layer used here is the
 * usual pre-norm decoder block: RMSNorm, bias-free q/k/v projections, rotary
 * position embedding in the rotate-half form over the whole head, grouped-query
 * causal softmax attention, output projection with residual, RMSNorm, SwiGLU MLP
 * with residual.  A head is RMSNorm followed by a bias-free projection to the
 * vocabulary.  Token ids [0, Vt) are text, [Vt, Vt+Vs) are speech, and the argmax
 * is taken over the id range of the modality being emitted (lowest id on ties).
 *
 * Arithmetic: every value is a double.  Weights arrive as bfloat16 bit patterns
 * (the values the GPU also gets) and are widened exactly.  Nothing is blocked,
 * fused or reordered beyond the loops written here.
 *
 * Pinned (see tests, "not gpu"): schedule against the exit layers the paper prints
 * in Table II and against enumeration; whole decoder against a cache-free
 * recomputation in NumPy and against a library Llama forward; rope / softmax /
 * rmsnorm against textbook identities; the KV invariant of Sec. IV-B.3.
 * Parity unpinned: nothing about the *quality* of early-exit tokens (heads are
 * random), which is outside what this decoder computes.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn;
    int32_t vocab_text, vocab_speech;
    double rms_eps, rope_base;
    int32_t exit_layer;     /* l_EE, 1..L; equal to L means no early exit        */
    int32_t refresh_period; /* K >= 1                                             */
    int32_t refresh_phase;  /* r in [0,K): in-chunk index c is full iff c%K == r  */
    int32_t text_exit;      /* 0: text always full depth (paper's main rows);
                               1: text follows the same schedule as speech;
                               2: only text follows it, speech always runs L
                                  layers (Sec. V-E, row G10: text Even, speech --) */
    int32_t max_len;        /* positions a sequence can hold                      */
    int32_t text_period;    /* K of text positions when they follow the schedule
                               (text_exit 1 or 2); 0: the same K and r as speech:
                               the modalities may need different policies (Sec. V-E) */
    int32_t text_phase;     /* r of text positions, in [0, text_period)           */
    /* Confidence-based early exit (Sec. V-B, compared method 3; thresholds in Sec. VI):
     * positions of the modalities in conf_modalities (bit 0 text, bit 1 speech) ignore the
     * schedule; from layer conf_start on, the head of each layer is applied to the position's
     * hidden state, and the position exits at the first layer whose prediction has an
     * entropy below conf_threshold (natural logarithm, over the ids of the modality being
     * emitted); if none does, it runs all L layers. */
    int32_t conf_modalities;
    int32_t conf_start;     /* first layer whose head is consulted, 1..L-1        */
    double conf_threshold;
} ora_dims;

typedef struct {
    const uint16_t *embed;            /* [Vt+Vs, d]                               */
    const uint16_t *const *attn_norm; /* [L] -> [d]                               */
    const uint16_t *const *wq;        /* [L] -> [Hq*hd, d]                        */
    const uint16_t *const *wk;        /* [L] -> [Hkv*hd, d]                       */
    const uint16_t *const *wv;        /* [L] -> [Hkv*hd, d]                       */
    const uint16_t *const *wo;        /* [L] -> [d, Hq*hd]                        */
    const uint16_t *const *mlp_norm;  /* [L] -> [d]                               */
    const uint16_t *const *w_gate;    /* [L] -> [F, d]                            */
    const uint16_t *const *w_up;      /* [L] -> [F, d]                            */
    const uint16_t *const *w_down;    /* [L] -> [d, F]                            */
    const uint16_t *const *head_norm; /* [L] -> [d]   (entry l-1: head of layer l; may be NULL) */
    const uint16_t *const *head_proj; /* [L] -> [Vt+Vs, d]                        */
} ora_weights;

typedef struct {
    ora_dims dm;
    ora_weights w;
} ora_model;

typedef struct {
    const ora_model *m;
    int32_t len;       /* positions ingested so far                               */
    int32_t n_pending; /* |P|                                                     */
    int32_t *pend_pos; /* positions in P, ascending                               */
    double *pend_h;    /* h^(l_EE) of each pending position, [max_pending][d]     */
    int32_t *pend_fill; /* layers whose K/V the pending position already has (the
                           layer it left at, or a later one it was carried to); the
                           scheduled decoder only ever stores l_EE here           */
    int32_t max_pending;
    double *K, *V;     /* [L][max_len][Hkv*hd], keys stored after rotation        */
} ora_seq;

/* ---------------------------------------------------------------- helpers */

static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Sec. IV-B.1.  modality 0 = text, 1 = speech.  c = index of the position inside
 * its chunk (0-based).  Returns the number of layers the step runs. */
int32_t ora_depth(int32_t modality, int32_t c, int32_t K, int32_t r, int32_t e, int32_t L,
                  int32_t text_exit)
{
    if (modality == 0 && text_exit == 0) return L;
    if (modality == 1 && text_exit == 2) return L;
    return (c % K == r) ? L : e;
}

/* The same rule with a period and a phase of its own for each modality (Sec. V-E: text and
 * speech positions may need different policies): speech positions use (K_s, r_s), text
 * positions that follow the schedule use (K_t, r_t). */
int32_t ora_depth_mod(int32_t modality, int32_t c, int32_t K_s, int32_t r_s, int32_t K_t,
                      int32_t r_t, int32_t e, int32_t L, int32_t text_exit)
{
    if (modality == 0) return ora_depth(0, c, K_t, r_t, e, L, text_exit);
    return ora_depth(1, c, K_s, r_s, e, L, text_exit);
}

/* y = x / sqrt(mean(x^2) + eps) * g */
void ora_rmsnorm(const double *x, const uint16_t *g, int32_t d, double eps, double *y)
{
    double ss = 0.0;
    for (int i = 0; i < d; i++) ss += x[i] * x[i];
    double inv = 1.0 / sqrt(ss / d + eps);
    for (int i = 0; i < d; i++) y[i] = x[i] * inv * bf16_to_double(g[i]);
}

/* Rotary embedding of one head at absolute position pos, rotate-half pairing:
 * element i is paired with element i + hd/2, angle pos * base^(-2i/hd). */
void ora_rope(double *x, int32_t hd, int32_t pos, double base)
{
    int half = hd / 2;
    for (int i = 0; i < half; i++) {
        double theta = (double)pos * pow(base, -2.0 * i / hd);
        double c = cos(theta), s = sin(theta);
        double a = x[i], b = x[i + half];
        x[i] = a * c - b * s;
        x[i + half] = b * c + a * s;
    }
}

/* One query against n keys/values of one head: out = sum_u softmax_u(q.K[u]/sqrt(hd)) V[u].
 * K and V rows are `stride` doubles apart.  w (length n) receives the softmax weights. */
void ora_attend(const double *q, const double *K, const double *V, int32_t n, int32_t hd,
                int32_t stride, double *w, double *out)
{
    double mx = -INFINITY;
    for (int u = 0; u < n; u++) {
        double s = 0.0;
        for (int i = 0; i < hd; i++) s += q[i] * K[(size_t)u * stride + i];
        w[u] = s / sqrt((double)hd);
        if (w[u] > mx) mx = w[u];
    }
    double z = 0.0;
    for (int u = 0; u < n; u++) {
        w[u] = exp(w[u] - mx);
        z += w[u];
    }
    for (int u = 0; u < n; u++) w[u] /= z;
    for (int i = 0; i < hd; i++) out[i] = 0.0;
    for (int u = 0; u < n; u++)
        for (int i = 0; i < hd; i++) out[i] += w[u] * V[(size_t)u * stride + i];
}

/* Y[r][o] = sum_i W[o][i] X[r][i]   (W bf16 [n_out][n_in], X [n_rows][n_in]) */
static void matmul_rows(const uint16_t *W, int n_out, int n_in, const double *X, int n_rows,
                        double *Y)
{
#pragma omp parallel
    {
        double *wrow = (double *)malloc(sizeof(double) * (size_t)n_in);
#pragma omp for schedule(static)
        for (int o = 0; o < n_out; o++) {
            const uint16_t *src = W + (size_t)o * n_in;
            for (int i = 0; i < n_in; i++) wrow[i] = bf16_to_double(src[i]);
            for (int r = 0; r < n_rows; r++) {
                const double *x = X + (size_t)r * n_in;
                double s = 0.0;
                for (int i = 0; i < n_in; i++) s += wrow[i] * x[i];
                Y[(size_t)r * n_out + o] = s;
            }
        }
        free(wrow);
    }
}

static double silu(double x) { return x / (1.0 + exp(-x)); }

/* ---------------------------------------------------------------- model / sequence */

ora_model *ora_model_new(const ora_dims *dm, const ora_weights *w)
{
    if (!dm || !w) return NULL;
    if (dm->n_layers < 1 || dm->exit_layer < 1 || dm->exit_layer > dm->n_layers) return NULL;
    if (dm->refresh_period < 1 || dm->refresh_phase < 0 || dm->refresh_phase >= dm->refresh_period)
        return NULL;
    if (dm->n_q_heads % dm->n_kv_heads != 0 || dm->head_dim % 2 != 0) return NULL;
    if (dm->text_period < 0 || (dm->text_period > 0 && (dm->text_phase < 0 || dm->text_phase >= dm->text_period)))
        return NULL;
    ora_model *m = (ora_model *)calloc(1, sizeof *m);
    m->dm = *dm;
    m->w = *w;
    return m;
}

void ora_model_free(ora_model *m) { free(m); }

ora_seq *ora_seq_new(const ora_model *m, int32_t max_pending)
{
    const ora_dims *dm = &m->dm;
    ora_seq *s = (ora_seq *)calloc(1, sizeof *s);
    s->m = m;
    s->max_pending = max_pending < 1 ? 1 : max_pending;
    s->pend_pos = (int32_t *)calloc((size_t)s->max_pending, sizeof(int32_t));
    s->pend_h = (double *)calloc((size_t)s->max_pending * dm->d_model, sizeof(double));
    s->pend_fill = (int32_t *)calloc((size_t)s->max_pending, sizeof(int32_t));
    size_t kv = (size_t)dm->n_layers * dm->max_len * dm->n_kv_heads * dm->head_dim;
    s->K = (double *)calloc(kv, sizeof(double));
    s->V = (double *)calloc(kv, sizeof(double));
    if (!s->pend_pos || !s->pend_h || !s->pend_fill || !s->K || !s->V) return NULL;
    return s;
}

void ora_seq_free(ora_seq *s)
{
    if (!s) return;
    free(s->pend_pos);
    free(s->pend_h);
    free(s->pend_fill);
    free(s->K);
    free(s->V);
    free(s);
}

int32_t ora_seq_len(const ora_seq *s) { return s->len; }
int32_t ora_seq_pending(const ora_seq *s) { return s->n_pending; }
int32_t ora_seq_pending_pos(const ora_seq *s, int32_t j) { return s->pend_pos[j]; }
int32_t ora_seq_pending_fill(const ora_seq *s, int32_t j) { return s->pend_fill[j]; }

static double *kv_at(double *base, const ora_dims *dm, int layer /*1-based*/, int pos)
{
    size_t row = (size_t)dm->n_kv_heads * dm->head_dim;
    return base + ((size_t)(layer - 1) * dm->max_len + pos) * row;
}

/* Read or overwrite the cached key/value of one (layer, position): Hkv*hd doubles each. */
void ora_get_kv(ora_seq *s, int32_t layer, int32_t pos, double *k, double *v)
{
    const ora_dims *dm = &s->m->dm;
    size_t row = (size_t)dm->n_kv_heads * dm->head_dim;
    memcpy(k, kv_at(s->K, dm, layer, pos), row * sizeof(double));
    memcpy(v, kv_at(s->V, dm, layer, pos), row * sizeof(double));
}
void ora_set_kv(ora_seq *s, int32_t layer, int32_t pos, const double *k, const double *v)
{
    const ora_dims *dm = &s->m->dm;
    size_t row = (size_t)dm->n_kv_heads * dm->head_dim;
    memcpy(kv_at(s->K, dm, layer, pos), k, row * sizeof(double));
    memcpy(kv_at(s->V, dm, layer, pos), v, row * sizeof(double));
}
/* Declare that positions [0, len) already have K/V at every layer (set through ora_set_kv). */
void ora_set_len(ora_seq *s, int32_t len)
{
    s->len = len;
    s->n_pending = 0;
}

/*
 * One transformer layer applied to a block of rows of ONE sequence.
 * pos[i] is the absolute position of row i (ascending), H[i] its hidden state,
 * updated in place from h^(layer-1) to h^(layer).  All rows first write their
 * K/V into the cache, then every row attends to positions 0..pos[i]: that is
 * the causal mask over the block plus the whole earlier cache (Algorithm 1,
 * full-depth branch: pending positions and the current one pass the upper layers together).
 */
static void layer_block(ora_seq *s, int layer, const int32_t *pos, int n_rows, double *H)
{
    const ora_dims *dm = &s->m->dm;
    const ora_weights *w = &s->m->w;
    const int d = dm->d_model, hd = dm->head_dim, Hq = dm->n_q_heads, Hkv = dm->n_kv_heads;
    const int F = dm->d_ffn, G = Hq / Hkv, li = layer - 1;
    const int qd = Hq * hd, kd = Hkv * hd;

    double *A = (double *)malloc(sizeof(double) * (size_t)n_rows * d);
    double *Q = (double *)malloc(sizeof(double) * (size_t)n_rows * qd);
    double *Kn = (double *)malloc(sizeof(double) * (size_t)n_rows * kd);
    double *Vn = (double *)malloc(sizeof(double) * (size_t)n_rows * kd);
    double *O = (double *)malloc(sizeof(double) * (size_t)n_rows * qd);
    double *T = (double *)malloc(sizeof(double) * (size_t)n_rows * d);
    double *Gt = (double *)malloc(sizeof(double) * (size_t)n_rows * F);
    double *Up = (double *)malloc(sizeof(double) * (size_t)n_rows * F);

    for (int i = 0; i < n_rows; i++)
        ora_rmsnorm(H + (size_t)i * d, w->attn_norm[li], d, dm->rms_eps, A + (size_t)i * d);
    matmul_rows(w->wq[li], qd, d, A, n_rows, Q);
    matmul_rows(w->wk[li], kd, d, A, n_rows, Kn);
    matmul_rows(w->wv[li], kd, d, A, n_rows, Vn);
    for (int i = 0; i < n_rows; i++) {
        for (int j = 0; j < Hq; j++) ora_rope(Q + (size_t)i * qd + j * hd, hd, pos[i], dm->rope_base);
        for (int j = 0; j < Hkv; j++) ora_rope(Kn + (size_t)i * kd + j * hd, hd, pos[i], dm->rope_base);
        memcpy(kv_at(s->K, dm, layer, pos[i]), Kn + (size_t)i * kd, sizeof(double) * kd);
        memcpy(kv_at(s->V, dm, layer, pos[i]), Vn + (size_t)i * kd, sizeof(double) * kd);
    }
    /* every (row, head) pair is one independent call of ora_attend; the pairs are only dealt to
     * threads, each with its own buffer for the softmax weights */
#pragma omp parallel
    {
        double *wts = (double *)malloc(sizeof(double) * (size_t)dm->max_len);
#pragma omp for collapse(2) schedule(static)
        for (int i = 0; i < n_rows; i++)
            for (int j = 0; j < Hq; j++) {
                int kvh = j / G;
                ora_attend(Q + (size_t)i * qd + j * hd, kv_at(s->K, dm, layer, 0) + kvh * hd,
                           kv_at(s->V, dm, layer, 0) + kvh * hd, pos[i] + 1, hd, kd, wts,
                           O + (size_t)i * qd + j * hd);
            }
        free(wts);
    }
    matmul_rows(w->wo[li], d, qd, O, n_rows, T);
    for (size_t i = 0; i < (size_t)n_rows * d; i++) H[i] += T[i];

    for (int i = 0; i < n_rows; i++)
        ora_rmsnorm(H + (size_t)i * d, w->mlp_norm[li], d, dm->rms_eps, A + (size_t)i * d);
    matmul_rows(w->w_gate[li], F, d, A, n_rows, Gt);
    matmul_rows(w->w_up[li], F, d, A, n_rows, Up);
    for (size_t i = 0; i < (size_t)n_rows * F; i++) Gt[i] = silu(Gt[i]) * Up[i];
    matmul_rows(w->w_down[li], d, F, Gt, n_rows, T);
    for (size_t i = 0; i < (size_t)n_rows * d; i++) H[i] += T[i];

    free(A); free(Q); free(Kn); free(Vn); free(O); free(T); free(Gt); free(Up);
}

static void embed_row(const ora_model *m, int32_t token, double *h)
{
    const int d = m->dm.d_model;
    for (int i = 0; i < d; i++) h[i] = bf16_to_double(m->w.embed[(size_t)token * d + i]);
}

/* Ingest n prompt tokens at full depth; nothing is emitted.  Returns 0, or -1 when
 * the sequence would overflow or has pending positions. */
int32_t ora_prefill(ora_seq *s, const int32_t *tokens, int32_t n)
{
    const ora_dims *dm = &s->m->dm;
    if (n < 0 || s->len + n > dm->max_len || s->n_pending) return -1;
    if (n == 0) return 0;
    const int d = dm->d_model;
    double *H = (double *)malloc(sizeof(double) * (size_t)n * d);
    int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    for (int i = 0; i < n; i++) {
        pos[i] = s->len + i;
        embed_row(s->m, tokens[i], H + (size_t)i * d);
    }
    for (int l = 1; l <= dm->n_layers; l++) layer_block(s, l, pos, n, H);
    s->len += n;
    free(H);
    free(pos);
    return 0;
}

/*
 * Head of layer `layer` on hidden state h, restricted to the id range of `modality`.
 * logits (length Vt+Vs, may be NULL) gets -inf outside the range.  Returns the
 * argmax id (lowest id on ties); *margin = best - second best inside the range.
 */
static int32_t head_argmax(const ora_model *m, int layer, const double *h, int modality,
                           double *logits, double *margin)
{
    const ora_dims *dm = &m->dm;
    const int d = dm->d_model, V = dm->vocab_text + dm->vocab_speech;
    const int lo = modality == 0 ? 0 : dm->vocab_text;
    const int hi = modality == 0 ? dm->vocab_text : V;
    double *a = (double *)malloc(sizeof(double) * (size_t)d);
    double *z = (double *)malloc(sizeof(double) * (size_t)(hi - lo));
    ora_rmsnorm(h, m->w.head_norm[layer - 1], d, dm->rms_eps, a);
    matmul_rows(m->w.head_proj[layer - 1] + (size_t)lo * d, hi - lo, d, a, 1, z);
    int best = 0;
    for (int i = 1; i < hi - lo; i++)
        if (z[i] > z[best]) best = i;
    double second = -INFINITY;
    for (int i = 0; i < hi - lo; i++)
        if (i != best && z[i] > second) second = z[i];
    if (margin) *margin = z[best] - second;
    if (logits) {
        for (int i = 0; i < V; i++) logits[i] = -INFINITY;
        for (int i = lo; i < hi; i++) logits[i] = z[i - lo];
    }
    free(a);
    free(z);
    return lo + best;
}

/*
 * One decoding step (Algorithm 1, one iteration of its loop, for text and speech
 * alike).  `token` is the input token of this step (the last emitted or last
 * prompt token); `modality` is the modality of the token this step emits and
 * `counter` its index inside its chunk.
 * Outputs: *next_token, *depth (layers run), *margin (top-2 gap of the restricted
 * logits), hidden (d doubles, the hidden state the head read; may be NULL), logits
 * (Vt+Vs doubles; may be NULL).
 * Returns 0; -1 if the cache or the pending store is full; -2 if a needed head is
 * missing.
 */
int32_t ora_decode_step(ora_seq *s, int32_t token, int32_t modality, int32_t counter,
                        int32_t *next_token, int32_t *depth, double *margin, double *hidden,
                        double *logits)
{
    const ora_model *m = s->m;
    const ora_dims *dm = &m->dm;
    const int d = dm->d_model, L = dm->n_layers, e = dm->exit_layer;
    if (s->len >= dm->max_len) return -1;
    const int K_t = dm->text_period > 0 ? dm->text_period : dm->refresh_period;
    const int r_t = dm->text_period > 0 ? dm->text_phase : dm->refresh_phase;
    const int dep = ora_depth_mod(modality, counter, dm->refresh_period, dm->refresh_phase, K_t, r_t,
                                  e, L, dm->text_exit);
    if (dep < L && s->n_pending >= s->max_pending) return -1;
    if (!m->w.head_norm[dep - 1] || !m->w.head_proj[dep - 1]) return -2;

    const int32_t p = s->len;
    double *h = (double *)malloc(sizeof(double) * (size_t)d);
    embed_row(m, token, h);
    /* layers 1..l_EE on the new position; their K/V go into the cache */
    for (int l = 1; l <= e; l++) layer_block(s, l, &p, 1, h);

    if (dep < L) {
        /* early exit: keep h^(l_EE), defer the upper K/V, read the token from g_{l_EE} */
        s->pend_pos[s->n_pending] = p;
        s->pend_fill[s->n_pending] = e;
        memcpy(s->pend_h + (size_t)s->n_pending * d, h, sizeof(double) * d);
        s->n_pending++;
        *next_token = head_argmax(m, e, h, modality, logits, margin);
        if (hidden) memcpy(hidden, h, sizeof(double) * d);
    } else {
        /* full depth: pending positions and the new one go through l_EE+1..L together */
        const int n = s->n_pending + 1;
        double *H = (double *)malloc(sizeof(double) * (size_t)n * d);
        int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        for (int j = 0; j < s->n_pending; j++) {
            pos[j] = s->pend_pos[j];
            memcpy(H + (size_t)j * d, s->pend_h + (size_t)j * d, sizeof(double) * d);
        }
        pos[n - 1] = p;
        memcpy(H + (size_t)(n - 1) * d, h, sizeof(double) * d);
        for (int l = e + 1; l <= L; l++) layer_block(s, l, pos, n, H);
        /* only the new position's h^(L) is read; pending positions keep their emitted token */
        *next_token = head_argmax(m, L, H + (size_t)(n - 1) * d, modality, logits, margin);
        if (hidden) memcpy(hidden, H + (size_t)(n - 1) * d, sizeof(double) * d);
        s->n_pending = 0;
        free(H);
        free(pos);
    }
    *depth = dep;
    s->len = p + 1;
    free(h);
    return 0;
}

/* ---------------------------------------------------------------- exits at any layer */

/* Entropy (natural logarithm) of softmax(z[0..n)).  Sec. V-B: the confidence signal of the
 * compared method is the entropy of the layer's next-token distribution. */
double ora_entropy(const double *z, int32_t n)
{
    double mx = -INFINITY;
    for (int i = 0; i < n; i++)
        if (z[i] > mx) mx = z[i];
    double sum = 0.0;
    for (int i = 0; i < n; i++) sum += exp(z[i] - mx);
    double h = 0.0;
    for (int i = 0; i < n; i++) {
        double p = exp(z[i] - mx) / sum;
        if (p > 0.0) h -= p * log(p);
    }
    return h;
}

/*
 * One decoding step whose depth is not known beforehand: either dictated by the caller
 * (forced_depth in 1..L: any layer that has a head) or decided on the way by the confidence
 * rule of the dims (forced_depth = 0; positions of a modality outside conf_modalities follow
 * the schedule as in ora_decode_step).
 *
 * Deferred filling, stated for exits at arbitrary layers (Sec. IV-B.3 states it for one exit
 * layer; the rule is the same): a position that left at layer f lacks K/V above f.  Whenever a
 * later position is about to run a layer l > f, the earlier one is taken along through l in
 * the same causal block, so that every position attends to complete K/V at every layer it
 * runs.  A pending position therefore records how far it has been carried (pend_fill) and the
 * hidden state at that layer; a step that runs all L layers completes and drops them all.
 * With a single exit layer this is exactly Algorithm 1.
 *
 * entropies (may be NULL) receives, for layer l = 1..L-1, the entropy computed at that layer
 * or -1 where no head was consulted.  With a dictated depth the rule decides nothing, but for a
 * position of a confidence modality the entropies of the layers conf_start .. depth are still
 * reported (a checker can then judge a depth chosen elsewhere against them).
 */
int32_t ora_decode_step_dyn(ora_seq *s, int32_t token, int32_t modality, int32_t counter,
                            int32_t forced_depth, int32_t *next_token, int32_t *depth,
                            double *margin, double *hidden, double *logits, double *entropies)
{
    const ora_model *m = s->m;
    const ora_dims *dm = &m->dm;
    const int d = dm->d_model, L = dm->n_layers;
    const int V = dm->vocab_text + dm->vocab_speech;
    if (s->len >= dm->max_len) return -1;
    if (forced_depth < 0 || forced_depth > L) return -3;
    const int conf_mod = (dm->conf_modalities >> (modality ? 1 : 0)) & 1;
    const int by_conf = forced_depth == 0 && conf_mod;
    int target = forced_depth;   /* 0: decided by confidence */
    if (forced_depth == 0 && !by_conf) {
        const int K_t = dm->text_period > 0 ? dm->text_period : dm->refresh_period;
        const int r_t = dm->text_period > 0 ? dm->text_phase : dm->refresh_phase;
        target = ora_depth_mod(modality, counter, dm->refresh_period, dm->refresh_phase, K_t, r_t,
                               dm->exit_layer, L, dm->text_exit);
    }
    if (target && (!m->w.head_norm[target - 1] || !m->w.head_proj[target - 1])) return -2;
    if (by_conf && (dm->conf_start < 1 || dm->conf_start >= L)) return -3;
    if (s->n_pending >= s->max_pending) return -1;   /* the step may add one */
    if (entropies)
        for (int l = 1; l < L; l++) entropies[l - 1] = -1.0;

    const int32_t p = s->len;
    const int n_max = s->n_pending + 1;
    double *H = (double *)malloc(sizeof(double) * (size_t)n_max * d);
    double *Hb = (double *)malloc(sizeof(double) * (size_t)n_max * d);
    int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_max);
    int32_t *who = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_max);
    double *z = (double *)malloc(sizeof(double) * (size_t)V);
    /* row j < n_pending: pending position j at the layer it has been carried to; last row: the
     * new position */
    for (int j = 0; j < s->n_pending; j++) memcpy(H + (size_t)j * d, s->pend_h + (size_t)j * d, sizeof(double) * d);
    double *hc = H + (size_t)s->n_pending * d;
    embed_row(m, token, hc);

    int dep = 0;
    for (int l = 1; l <= L; l++) {
        /* the block of this layer: pending positions not yet carried through l, then the new one */
        int n = 0;
        for (int j = 0; j < s->n_pending; j++)
            if (s->pend_fill[j] < l) {
                pos[n] = s->pend_pos[j];
                who[n] = j;
                memcpy(Hb + (size_t)n * d, H + (size_t)j * d, sizeof(double) * d);
                n++;
            }
        pos[n] = p;
        who[n] = s->n_pending;
        memcpy(Hb + (size_t)n * d, hc, sizeof(double) * d);
        n++;
        layer_block(s, l, pos, n, Hb);
        for (int i = 0; i < n; i++) memcpy(H + (size_t)who[i] * d, Hb + (size_t)i * d, sizeof(double) * d);
        for (int j = 0; j < s->n_pending; j++)
            if (s->pend_fill[j] < l) s->pend_fill[j] = l;
        dep = l;
        if (conf_mod && dm->conf_start >= 1 && l >= dm->conf_start && l < L && (by_conf || entropies)) {
            if (!m->w.head_norm[l - 1] || !m->w.head_proj[l - 1]) {
                if (by_conf) {
                    free(H); free(Hb); free(pos); free(who); free(z);
                    return -2;
                }
            } else {
                head_argmax(m, l, hc, modality, z, NULL);
                const int lo = modality == 0 ? 0 : dm->vocab_text;
                const int hi = modality == 0 ? dm->vocab_text : V;
                const double ent = ora_entropy(z + lo, hi - lo);
                if (entropies) entropies[l - 1] = ent;
                if (by_conf && ent < dm->conf_threshold) break;
            }
        }
        if (target && l == target) break;
    }
    *next_token = head_argmax(m, dep, hc, modality, logits, margin);
    if (hidden) memcpy(hidden, hc, sizeof(double) * d);
    if (dep == L) {
        s->n_pending = 0;
    } else {
        /* every pending position has been carried to layer dep (or was beyond it already) */
        for (int j = 0; j < s->n_pending; j++) memcpy(s->pend_h + (size_t)j * d, H + (size_t)j * d, sizeof(double) * d);
        s->pend_pos[s->n_pending] = p;
        s->pend_fill[s->n_pending] = dep;
        memcpy(s->pend_h + (size_t)s->n_pending * d, hc, sizeof(double) * d);
        s->n_pending++;
    }
    *depth = dep;
    s->len = p + 1;
    free(H); free(Hb); free(pos); free(who); free(z);
    return 0;
}
