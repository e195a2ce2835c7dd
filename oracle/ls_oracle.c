/*
 * ls_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, obviously-correct CPU statement of what the batch-1
 * self-speculative greedy decode loop of LayerSkip computes on a Llama-style
 * decoder.  Arithmetic is IEEE double throughout; the model "is" its bf16
 * weights, which are widened exactly (bf16 -> double) on use.  Nothing here is
 * blocked, fused or reordered: every function is the textbook definition, or
 * the paper's algorithm taken step by step.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call into this file; the CUDA library shares
 * no code with it.
 *
 * Passages followed (LayerSkip, arXiv 2404.16710):
 *   Sec. 4.1 notation     residual decoder x_{l+1} = x_l + f_l(x_l), logits g(x_L)
 *   Sec. 2.1 / Sec. 4.2   the LM head g = final normalisation + linear layer is
 *                         shared by every exit; early exit outputs g(x_E)
 *   Sec. 4.3.1            self-drafting: d tokens, autoregressively, exiting at layer E
 *   Sec. 4.3.2            self-verification: the remaining L-E layers score all draft
 *                         positions; accept up to the first disagreement, plus the
 *                         verified token there
 *   Sec. 4.3.3            one KV cache for both stages + the exit-layer activations
 *   Appendix A.4          the loop: draft, verify, match, extend output, crop the cache
 *
 * Llama internals (RMSNorm, rotary embedding in the half-split pairing, causal
 * softmax attention with grouped KV heads, SwiGLU) are the standard published
 * definitions; the paper does not restate them.
 *
 * Pins (tests/test_oracle_*.py): closed forms for RMSNorm / RoPE / softmax /
 * SiLU, a double-precision numpy recomputation WITHOUT any cache using full
 * [T,T] attention matrices (oracle/ls_bruteforce.py), GQA <-> replicated-MHA
 * equivalence, the losslessness invariant for every (E, d), the zero-scale
 * case where every draft must be accepted, and hand-built match cases.
 * The accepted-per-step values on synthetic weights have no value in the paper
 * to compare with: "parity unpinned" for those numbers themselves (their
 * invariants are pinned).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t max_seq;
    int32_t eos_id; /* -1: never stop early */
    double rms_eps, rope_theta;
} lso_config;

/* bf16 bit patterns, row-major [out, in]; arrays of n_layers pointers */
typedef struct {
    const uint16_t *tok_embed, *final_norm, *lm_head;
    const uint16_t *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
    const uint16_t *const *ffn_norm, *const *w_gate, *const *w_up, *const *w_down;
} lso_weights;

typedef struct {
    lso_config c;
    lso_weights w;
    double *kc, *vc; /* [L][max_seq][Hkv*hd] */
} lso_model;

static double bf16_val(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* ---- elementary operations (exported so that tests can pin each one) ---- */

/* RMSNorm: y_i = x_i / sqrt(mean_j x_j^2 + eps) * g_i */
void lso_rmsnorm(const double *x, const uint16_t *g, int32_t D, double eps, double *y)
{
    double ss = 0.0;
    for (int i = 0; i < D; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / (double)D + eps);
    for (int i = 0; i < D; ++i) y[i] = x[i] * r * bf16_val(g[i]);
}

/* Rotary embedding of one head vector at position pos, half-split pairing:
 * (v_j, v_{j+hd/2}) is rotated by the angle pos * theta^(-2j/hd). */
void lso_rope(double *v, int32_t hd, int32_t pos, double theta)
{
    int half = hd / 2;
    for (int j = 0; j < half; ++j) {
        double ang = (double)pos * pow(theta, -2.0 * (double)j / (double)hd);
        double c = cos(ang), s = sin(ang);
        double a = v[j], b = v[j + half];
        v[j] = a * c - b * s;
        v[j + half] = a * s + b * c;
    }
}

/* y = W h, W is [N, K] row-major bf16 */
void lso_linear(const uint16_t *W, int32_t N, int32_t K, const double *h, double *y)
{
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        const uint16_t *row = W + (size_t)n * (size_t)K;
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += bf16_val(row[k]) * h[k];
        y[n] = acc;
    }
}

/* in-place softmax over n scores, max-subtracted */
void lso_softmax(double *s, int32_t n)
{
    double mx = s[0];
    for (int i = 1; i < n; ++i)
        if (s[i] > mx) mx = s[i];
    double z = 0.0;
    for (int i = 0; i < n; ++i) {
        s[i] = exp(s[i] - mx);
        z += s[i];
    }
    for (int i = 0; i < n; ++i) s[i] /= z;
}

double lso_silu(double z) { return z / (1.0 + exp(-z)); }

/* One query position of causal attention with grouped KV heads.
 * q [Hq*hd]; keys/values k, v are [n_keys][Hkv*hd]; o [Hq*hd].
 * Query head i reads KV head i / (Hq/Hkv). */
void lso_attention(const double *q, const double *k, const double *v, int32_t n_keys,
                   int32_t Hq, int32_t Hkv, int32_t hd, double *o)
{
    int group = Hq / Hkv;
    int kvw = Hkv * hd;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < Hq; ++i) {
        int kh = i / group;
        double *s = (double *)malloc(sizeof(double) * (size_t)n_keys);
        for (int j = 0; j < n_keys; ++j) {
            double acc = 0.0;
            for (int t = 0; t < hd; ++t) acc += q[i * hd + t] * k[(size_t)j * kvw + kh * hd + t];
            s[j] = acc / sqrt((double)hd);
        }
        lso_softmax(s, n_keys);
        for (int t = 0; t < hd; ++t) {
            double acc = 0.0;
            for (int j = 0; j < n_keys; ++j) acc += s[j] * v[(size_t)j * kvw + kh * hd + t];
            o[i * hd + t] = acc;
        }
        free(s);
    }
}

/* argmax, the lowest index wins a tie; also reports the top-1 / top-2 margin
 * and the largest magnitude (either may be NULL) */
int32_t lso_argmax(const double *z, int32_t n, double *margin, double *maxabs)
{
    int best = 0;
    for (int i = 1; i < n; ++i)
        if (z[i] > z[best]) best = i;
    if (margin) {
        double second = -INFINITY;
        for (int i = 0; i < n; ++i)
            if (i != best && z[i] > second) second = z[i];
        *margin = z[best] - second;
    }
    if (maxabs) {
        double m = 0.0;
        for (int i = 0; i < n; ++i)
            if (fabs(z[i]) > m) m = fabs(z[i]);
        *maxabs = m;
    }
    return best;
}

/* match (Appendix A.4): the number of leading drafts the full model agrees with */
int32_t lso_match(const int32_t *draft, const int32_t *verified, int32_t d)
{
    int n = 0;
    while (n < d && draft[n] == verified[n]) ++n;
    return n;
}

/* ---- the model ---- */

lso_model *lso_model_create(const lso_config *c, const lso_weights *w)
{
    if (c->n_heads % c->n_kv_heads != 0 || c->head_dim % 2 != 0) return NULL;
    lso_model *m = (lso_model *)calloc(1, sizeof(lso_model));
    if (!m) return NULL;
    m->c = *c;
    m->w = *w;
    size_t n = (size_t)c->n_layers * (size_t)c->max_seq * (size_t)(c->n_kv_heads * c->head_dim);
    m->kc = (double *)calloc(n, sizeof(double));
    m->vc = (double *)calloc(n, sizeof(double));
    if (!m->kc || !m->vc) {
        free(m->kc);
        free(m->vc);
        free(m);
        return NULL;
    }
    return m;
}

void lso_model_free(lso_model *m)
{
    if (!m) return;
    free(m->kc);
    free(m->vc);
    free(m);
}

static void embed(const lso_model *m, int32_t id, double *x)
{
    int D = m->c.d_model;
    for (int i = 0; i < D; ++i) x[i] = bf16_val(m->w.tok_embed[(size_t)id * D + i]);
}

/* One decoder layer applied to the token at position pos (Sec. 4.1:
 * x_{l+1} = x_l + f_l(x_l)); appends this position's k, v to layer l's cache
 * and attends over positions 0..pos. */
static void layer_token(lso_model *m, int l, double *x, int pos)
{
    const lso_config *c = &m->c;
    int D = c->d_model, Hq = c->n_heads, Hkv = c->n_kv_heads, hd = c->head_dim, F = c->d_ffn;
    int qw = Hq * hd, kvw = Hkv * hd;
    double *h = (double *)malloc(sizeof(double) * (size_t)D);
    double *q = (double *)malloc(sizeof(double) * (size_t)qw);
    double *o = (double *)malloc(sizeof(double) * (size_t)qw);
    double *t = (double *)malloc(sizeof(double) * (size_t)D);
    double *g = (double *)malloc(sizeof(double) * (size_t)F);
    double *u = (double *)malloc(sizeof(double) * (size_t)F);
    double *kl = m->kc + ((size_t)l * c->max_seq) * kvw;
    double *vl = m->vc + ((size_t)l * c->max_seq) * kvw;
    double *kp = kl + (size_t)pos * kvw, *vp = vl + (size_t)pos * kvw;

    lso_rmsnorm(x, m->w.attn_norm[l], D, c->rms_eps, h);
    lso_linear(m->w.wq[l], qw, D, h, q);
    lso_linear(m->w.wk[l], kvw, D, h, kp);
    lso_linear(m->w.wv[l], kvw, D, h, vp);
    for (int i = 0; i < Hq; ++i) lso_rope(q + i * hd, hd, pos, c->rope_theta);
    for (int i = 0; i < Hkv; ++i) lso_rope(kp + i * hd, hd, pos, c->rope_theta);
    lso_attention(q, kl, vl, pos + 1, Hq, Hkv, hd, o);
    lso_linear(m->w.wo[l], D, qw, o, t);
    for (int i = 0; i < D; ++i) x[i] += t[i];

    lso_rmsnorm(x, m->w.ffn_norm[l], D, c->rms_eps, h);
    lso_linear(m->w.w_gate[l], F, D, h, g);
    lso_linear(m->w.w_up[l], F, D, h, u);
    for (int i = 0; i < F; ++i) g[i] = lso_silu(g[i]) * u[i];
    lso_linear(m->w.w_down[l], D, F, g, t);
    for (int i = 0; i < D; ++i) x[i] += t[i];

    free(h); free(q); free(o); free(t); free(g); free(u);
}

/* layers [l0, l1) on one token */
static void layers_token(lso_model *m, int l0, int l1, double *x, int pos)
{
    for (int l = l0; l < l1; ++l) layer_token(m, l, x, pos);
}

/* the shared LM head g(.) = final norm + linear (Sec. 2.1, Sec. 4.2) */
static void lm_head(const lso_model *m, const double *x, double *logits)
{
    int D = m->c.d_model;
    double *h = (double *)malloc(sizeof(double) * (size_t)D);
    lso_rmsnorm(x, m->w.final_norm, D, m->c.rms_eps, h);
    lso_linear(m->w.lm_head, m->c.vocab, D, h, logits);
    free(h);
}

/* Teacher-forced logits: feed ids[0..n-1] at positions 0..n-1; for every
 * position t >= first write g(x_E) to exit_logits[t - first] and g(x_L) to
 * final_logits[t - first] (each [n - first, V], either may be NULL).  Positions
 * below `first` go through all layers exactly as the others do (they fill the
 * cache); only their logits are not asked for.  exit_layer = E counts the
 * early layers. */
int32_t lso_teacher_logits_tail(lso_model *m, const int32_t *ids, int32_t n, int32_t exit_layer,
                                int32_t first, double *exit_logits, double *final_logits)
{
    const lso_config *c = &m->c;
    if (n > c->max_seq || exit_layer < 1 || exit_layer > c->n_layers || first < 0 || first > n) return -1;
    double *x = (double *)malloc(sizeof(double) * (size_t)c->d_model);
    for (int t = 0; t < n; ++t) {
        if (ids[t] < 0 || ids[t] >= c->vocab) { free(x); return -1; }
        embed(m, ids[t], x);
        layers_token(m, 0, exit_layer, x, t);
        if (exit_logits && t >= first) lm_head(m, x, exit_logits + (size_t)(t - first) * c->vocab);
        layers_token(m, exit_layer, c->n_layers, x, t);
        if (final_logits && t >= first) lm_head(m, x, final_logits + (size_t)(t - first) * c->vocab);
    }
    free(x);
    return 0;
}

/* the same for every position */
int32_t lso_teacher_logits(lso_model *m, const int32_t *ids, int32_t n, int32_t exit_layer,
                           double *exit_logits, double *final_logits)
{
    return lso_teacher_logits_tail(m, ids, n, exit_layer, 0, exit_logits, final_logits);
}

/* Autoregressive greedy decoding with the full model (the result every other
 * routine must reproduce).  margins / maxabs ([max_new], may be NULL) receive the
 * top-1/top-2 logit gap and max|logit| at every emitted token. */
int32_t lso_generate_full(lso_model *m, const int32_t *prompt, int32_t P, int32_t max_new,
                          int32_t *out_ids, int32_t *out_n, double *margins, double *maxabs)
{
    const lso_config *c = &m->c;
    if (P < 1 || P + max_new > c->max_seq) return -1;
    double *x = (double *)malloc(sizeof(double) * (size_t)c->d_model);
    double *z = (double *)malloc(sizeof(double) * (size_t)c->vocab);
    int n = 0;
    for (int t = 0; t < P - 1; ++t) {
        embed(m, prompt[t], x);
        layers_token(m, 0, c->n_layers, x, t);
    }
    int32_t cur = prompt[P - 1];
    int pos = P - 1;
    while (n < max_new) {
        embed(m, cur, x);
        layers_token(m, 0, c->n_layers, x, pos);
        lm_head(m, x, z);
        double mg, ma;
        cur = lso_argmax(z, c->vocab, &mg, &ma);
        if (margins) margins[n] = mg;
        if (maxabs) maxabs[n] = ma;
        out_ids[n++] = cur;
        ++pos;
        if (c->eos_id >= 0 && cur == c->eos_id) break;
    }
    *out_n = n;
    free(x); free(z);
    return 0;
}

/* Early-exit greedy decoding (Sec. 4.2): every token is g(x_E). */
int32_t lso_generate_early(lso_model *m, const int32_t *prompt, int32_t P, int32_t exit_layer,
                           int32_t max_new, int32_t *out_ids, int32_t *out_n)
{
    const lso_config *c = &m->c;
    if (P < 1 || P + max_new > c->max_seq || exit_layer < 1 || exit_layer > c->n_layers) return -1;
    double *x = (double *)malloc(sizeof(double) * (size_t)c->d_model);
    double *z = (double *)malloc(sizeof(double) * (size_t)c->vocab);
    int n = 0;
    for (int t = 0; t < P - 1; ++t) {
        embed(m, prompt[t], x);
        layers_token(m, 0, exit_layer, x, t);
    }
    int32_t cur = prompt[P - 1];
    int pos = P - 1;
    while (n < max_new) {
        embed(m, cur, x);
        layers_token(m, 0, exit_layer, x, pos);
        lm_head(m, x, z);
        cur = lso_argmax(z, c->vocab, NULL, NULL);
        out_ids[n++] = cur;
        ++pos;
        if (c->eos_id >= 0 && cur == c->eos_id) break;
    }
    *out_n = n;
    free(x); free(z);
    return 0;
}

/* Self-speculative greedy decoding (Sec. 4.3, Appendix A.4).
 *
 * The prompt except its last token goes through all L layers (cache only); the
 * loop starts with cur = prompt[P-1] at cache length c = P-1.  One step:
 *   draft    for j in 0..d-1: layers 0..E-1 on the current draft input at
 *            position c+j (appending those layers' k, v), keep X_E[j],
 *            draft[j] = argmax g(X_E[j]), next input = draft[j];
 *            then layers 0..E-1 once more on draft[d-1] at position c+d -> X_E[d]
 *   verify   layers E..L-1 on rows 0..d at positions c..c+d, each row attending
 *            over the cache and the rows before it; verified[i] = argmax g(x_L[i])
 *   match    n = leading agreements; emit draft[0..n-1] then verified[n]
 *   crop     cur = verified[n]; c += n+1 (every emitted token but the last has
 *            a cache entry; entries beyond c are stale and get overwritten)
 * The emission is truncated at max_new (and after the first EOS when enabled);
 * accepted[step] records n untruncated.  cache_len_trace ([max_new], may be
 * NULL) receives c after every step.
 */
int32_t lso_generate_spec(lso_model *m, const int32_t *prompt, int32_t P, int32_t exit_layer,
                          int32_t num_draft, int32_t max_new, int32_t *out_ids, int32_t *out_n,
                          int32_t *accepted, int32_t *out_steps, int32_t *cache_len_trace)
{
    const lso_config *c = &m->c;
    int E = exit_layer, d = num_draft, L = c->n_layers, D = c->d_model;
    if (P < 1 || E < 1 || E > L - 1 || d < 1 || P + max_new + d + 1 > c->max_seq) return -1;
    double *x = (double *)malloc(sizeof(double) * (size_t)D);
    double *XE = (double *)malloc(sizeof(double) * (size_t)D * (size_t)(d + 1));
    double *z = (double *)malloc(sizeof(double) * (size_t)c->vocab);
    int32_t *draft = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
    int32_t *verified = (int32_t *)malloc(sizeof(int32_t) * (size_t)(d + 1));

    for (int t = 0; t < P - 1; ++t) {
        embed(m, prompt[t], x);
        layers_token(m, 0, L, x, t);
    }
    int32_t cur = prompt[P - 1];
    int clen = P - 1, n_out = 0, steps = 0, stop = 0;
    while (n_out < max_new && !stop) {
        /* self-drafting */
        int32_t in = cur;
        for (int j = 0; j < d; ++j) {
            embed(m, in, x);
            layers_token(m, 0, E, x, clen + j);
            memcpy(XE + (size_t)j * D, x, sizeof(double) * (size_t)D);
            lm_head(m, x, z);
            draft[j] = lso_argmax(z, c->vocab, NULL, NULL);
            in = draft[j];
        }
        embed(m, draft[d - 1], x);
        layers_token(m, 0, E, x, clen + d);
        memcpy(XE + (size_t)d * D, x, sizeof(double) * (size_t)D);
        /* self-verification, continuing from the exit-layer activations */
        for (int i = 0; i <= d; ++i) {
            memcpy(x, XE + (size_t)i * D, sizeof(double) * (size_t)D);
            layers_token(m, E, L, x, clen + i);
            lm_head(m, x, z);
            verified[i] = lso_argmax(z, c->vocab, NULL, NULL);
        }
        /* match, extend, crop */
        int n = lso_match(draft, verified, d);
        for (int i = 0; i <= n && n_out < max_new && !stop; ++i) {
            int32_t tok = (i < n) ? draft[i] : verified[n];
            out_ids[n_out++] = tok;
            if (c->eos_id >= 0 && tok == c->eos_id) stop = 1;
        }
        cur = verified[n];
        clen += n + 1;
        accepted[steps] = n;
        if (cache_len_trace) cache_len_trace[steps] = clen;
        ++steps;
    }
    *out_n = n_out;
    *out_steps = steps;
    free(x); free(XE); free(z); free(draft); free(verified);
    return 0;
}

/* Self-speculative decoding with an adaptive draft length: an extension (the paper drafts
 * a fixed d per step and leaves dynamic per-token conditions to future work, Sec. 9), stated
 * here so that the library's version of it has something to be compared with.
 *
 * One step, with at most d drafts and a confidence threshold tau > 0 on the exit logits:
 *   draft    for j in 0..d-1: layers 0..E-1 on the current draft input at position c+j,
 *            keep X_E[j]; z = g(X_E[j]); margin = largest - second largest entry of z
 *            (0 on a tie).  If margin < tau: the token is not kept, drafting stops, k = j.
 *            Otherwise draft[j] = argmax z and it becomes the next input.
 *            If no pass stopped: k = d and, as in the fixed-length loop, layers 0..E-1 run
 *            once more on draft[d-1] at position c+d -> X_E[d].
 *   verify   layers E..L-1 on rows 0..k; verified[i] = argmax g(x_L[i])
 *   match    n = leading agreements among the k kept drafts; emit draft[0..n-1], verified[n]
 *   crop     cur = verified[n]; c += n+1
 * Every emitted token is either a draft the full model agreed with or the full model's own
 * token, so the ids are those of lso_generate_full for every tau.  drafted[step] = k,
 * accepted[step] = n.  closest_gap ([max_new], may be NULL) receives, per step, the smallest
 * |margin - tau| over the stop decisions the step took -- what a comparison with an
 * implementation in another precision needs, to know how close to the threshold it came.
 */
int32_t lso_generate_adaptive(lso_model *m, const int32_t *prompt, int32_t P, int32_t exit_layer,
                              int32_t max_draft, double tau, int32_t max_new, int32_t *out_ids,
                              int32_t *out_n, int32_t *accepted, int32_t *drafted, int32_t *out_steps,
                              double *closest_gap)
{
    const lso_config *c = &m->c;
    int E = exit_layer, d = max_draft, L = c->n_layers, D = c->d_model;
    if (P < 1 || E < 1 || E > L - 1 || d < 1 || !(tau > 0.0) || P + max_new + d + 1 > c->max_seq) return -1;
    double *x = (double *)malloc(sizeof(double) * (size_t)D);
    double *XE = (double *)malloc(sizeof(double) * (size_t)D * (size_t)(d + 1));
    double *z = (double *)malloc(sizeof(double) * (size_t)c->vocab);
    int32_t *draft = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
    int32_t *verified = (int32_t *)malloc(sizeof(int32_t) * (size_t)(d + 1));

    for (int t = 0; t < P - 1; ++t) {
        embed(m, prompt[t], x);
        layers_token(m, 0, L, x, t);
    }
    int32_t cur = prompt[P - 1];
    int clen = P - 1, n_out = 0, steps = 0, stop = 0;
    while (n_out < max_new && !stop) {
        int32_t in = cur;
        int k = d;
        double gap = INFINITY; /* smallest |margin - tau| over the decisions taken this step */
        for (int j = 0; j < d; ++j) {
            embed(m, in, x);
            layers_token(m, 0, E, x, clen + j);
            memcpy(XE + (size_t)j * D, x, sizeof(double) * (size_t)D);
            lm_head(m, x, z);
            double margin;
            int32_t tok = lso_argmax(z, c->vocab, &margin, NULL);
            if (fabs(margin - tau) < gap) gap = fabs(margin - tau);
            if (margin < tau) {
                k = j;
                break;
            }
            draft[j] = tok;
            in = tok;
        }
        if (k == d) {
            embed(m, draft[d - 1], x);
            layers_token(m, 0, E, x, clen + d);
            memcpy(XE + (size_t)d * D, x, sizeof(double) * (size_t)D);
        }
        for (int i = 0; i <= k; ++i) {
            memcpy(x, XE + (size_t)i * D, sizeof(double) * (size_t)D);
            layers_token(m, E, L, x, clen + i);
            lm_head(m, x, z);
            verified[i] = lso_argmax(z, c->vocab, NULL, NULL);
        }
        int n = lso_match(draft, verified, k);
        for (int i = 0; i <= n && n_out < max_new && !stop; ++i) {
            int32_t tok = (i < n) ? draft[i] : verified[n];
            out_ids[n_out++] = tok;
            if (c->eos_id >= 0 && tok == c->eos_id) stop = 1;
        }
        cur = verified[n];
        clen += n + 1;
        accepted[steps] = n;
        drafted[steps] = k;
        if (closest_gap) closest_gap[steps] = gap;
        ++steps;
    }
    *out_n = n_out;
    *out_steps = steps;
    free(x); free(XE); free(z); free(draft); free(verified);
    return 0;
}

int32_t lso_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
