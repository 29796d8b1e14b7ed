/*
 * SpecBound CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct implementation of what the bounded
 * self-speculative decode step computes, written from the paper:
 *
 *   - a Llama-style decoder (the model family of the paper's Section 4.1),
 *   - plain greedy autoregressive decoding, which DEFINES the correct output
 *     (the paper's exact-equivalence claim: abstract, Section 3.3, Section 5),
 *   - the Annealed Confidence Threshold exit test (Section 3.2, Eq. 1-2),
 *   - the Bounded Speculation with Cached States round loop (Section 3.3 and
 *     the appendix "Illustration of Long Shallow Chains"),
 *   - the analytic speed-up model (Section 3.4, Eq. 3-5).
 *
 * Arithmetic: weights are read in their storage type (fp32 or bf16, both exact
 * in fp64); every sum, norm, softmax and activation is fp64.  Nothing is
 * blocked, fused or reordered beyond "one output row = one dot product".
 * OpenMP, where used, splits independent output rows only.
 *
 * It shares no code with the CUDA library and is only ever called from tests,
 * the smoke check and the benchmark's CPU-baseline leg.
 *
 * Pins (tests/test_oracle_*.py): closed forms of Eq. 1-5, softmax special
 * cases, torch CPU library routines for each decoder block, no-cache brute
 * force, speculative == autoregressive over a hyper-parameter grid, and the two
 * worked scenarios of Section 3.3 / the appendix with scripted exits.
 * Sampling decoding (Section 4.3 "decoding strategies", Table 2): the paper names
 * temperature sampling but prints no acceptance rule.  The reading taken here:
 * the token at sequence position p is the inverse-CDF sample, in vocabulary
 * order, of softmax(z / T_s) -- restricted to its top-p nucleus when top_p < 1 --
 * at the uniform number u(seed, p) of a counter-based generator; verification recomputes that token for every draft row and accepts
 * a draft iff it equals it.  Autoregressive sampling with the same (seed, T_s)
 * DEFINES the correct output; the speculative loop must reproduce it token for
 * token, which makes it lossless sample by sample and hence in distribution.
 * Pins: published splitmix64 outputs, stratified-u counts against a library
 * softmax, the T_s -> 0 limit (greedy), speculative == autoregressive over a grid.
 * Not pinned by the paper: the confidence VALUES on random weights (the paper
 * prints none) -- "parity unpinned" for those beyond the library cross-check.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_W 8

typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    double rope_base, rms_eps;
    int32_t wdtype;        /* storage of weights: 0 = fp32, 1 = bf16 */
    int32_t max_seq;
    int32_t kv_round_bf16; /* 1: K (after RoPE) and V are rounded to bf16 when cached */
} orc_config;

typedef struct {
    const void *attn_norm, *wq, *wk, *wv, *wo, *mlp_norm, *w_gate, *w_up, *w_down;
} orc_layer;

typedef struct {
    const void *embed, *final_norm, *lm_head;
    const orc_layer* layers; /* [n_layers] */
} orc_weights;

/* One speculation round as the loop of Section 3.3 executed it. */
typedef struct {
    int32_t w;                 /* rows in flight when the unified pass started */
    int32_t D;                 /* depth all rows were aligned to               */
    int32_t emitted;           /* tokens committed by this round               */
    int32_t accepted_drafts;   /* drafts that survived verification            */
    int32_t layer_steps;       /* layer passes issued (any number of rows)     */
    int32_t probes;            /* exit tests issued                            */
    int32_t exit_layer[ORC_MAX_W]; /* 0 = did not exit by d_max (difficult token) */
    int32_t draft[ORC_MAX_W];      /* -1 = none                                */
    int32_t g[ORC_MAX_W];          /* final-layer greedy token of each row     */
    int32_t layers_done[ORC_MAX_W];/* layers each row went through in total    */
    int32_t depth_after[ORC_MAX_W][ORC_MAX_W]; /* [draft step][row] depth after that step */
    double conf[ORC_MAX_W];        /* confidence at the exit layer (or at d_max) */
} orc_round;

typedef struct orc_ctx {
    orc_config c;
    orc_weights w;
    orc_layer* layers;
    double *K, *V; /* [n_layers][max_seq][n_kv_heads*head_dim] */
    /* Section 3.2: the exit test after layer l may use a head of its own ("lightweight LM heads"):
     * exit_head[l-1] / exit_norm[l-1], NULL = the shared LM head / final norm gain */
    const void** exit_head;
    const void** exit_norm;
    /* sampling decoding (Section 4.3, decoding strategies): temperature 0 = greedy */
    double sample_temperature, sample_top_p;
    uint64_t sample_seed;
} orc_ctx;

/* ---------------------------------------------------------------- helpers */

static double wget(const void* base, int dtype, size_t i) {
    if (dtype == 0) return (double)((const float*)base)[i];
    uint32_t u = (uint32_t)((const uint16_t*)base)[i] << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* round-to-nearest-even to bf16 (through fp32), returned as a double */
static double round_bf16(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) != 0x7f800000u) u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* y[r] = sum_c W[r,c] x[c], W row-major [rows, cols] */
static void matvec(const void* W, int dtype, int rows, int cols, const double* x, double* y) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < rows; ++r) {
        double acc = 0.0;
        size_t base = (size_t)r * (size_t)cols;
        for (int c = 0; c < cols; ++c) acc += wget(W, dtype, base + c) * x[c];
        y[r] = acc;
    }
}

/* RMSNorm(x) = x / sqrt(mean(x^2) + eps) * gain */
static void rmsnorm(const double* x, const void* gain, int dtype, int d, double eps, double* out) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    double inv = 1.0 / sqrt(ss / d + eps);
    for (int i = 0; i < d; ++i) out[i] = x[i] * inv * wget(gain, dtype, i);
}

/* rotary embedding, rotate-half pairing (i, i + hd/2), angle = pos * base^(-2i/hd) */
static void rope(double* v, int hd, int pos, double base) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)pos * pow(base, -2.0 * i / hd);
        double c = cos(ang), s = sin(ang), a = v[i], b = v[i + half];
        v[i] = a * c - b * s;
        v[i + half] = b * c + a * s;
    }
}

static double* kv_at(double* base, const orc_config* c, int layer0, int pos) {
    size_t kvd = (size_t)c->n_kv_heads * c->head_dim;
    return base + ((size_t)layer0 * c->max_seq + pos) * kvd;
}

/* One decoder layer (1-based index `layer`) for ONE row at position `pos`.
 * Writes K,V of this layer at `pos`, attends over positions 0..pos. */
static void layer_row(orc_ctx* o, int layer, double* h, int pos) {
    const orc_config* c = &o->c;
    const orc_layer* L = &o->layers[layer - 1];
    int d = c->d_model, H = c->n_heads, Hkv = c->n_kv_heads, hd = c->head_dim, F = c->d_ffn;
    int qd = H * hd, kvd = Hkv * hd, dt = c->wdtype;
    double* a = malloc(sizeof(double) * d);
    double* q = malloc(sizeof(double) * qd);
    double* att = malloc(sizeof(double) * qd);
    double* proj = malloc(sizeof(double) * d);
    double* gate = malloc(sizeof(double) * F);
    double* up = malloc(sizeof(double) * F);
    double* sc = malloc(sizeof(double) * (pos + 1));
    double* kk = kv_at(o->K, c, layer - 1, pos);
    double* vv = kv_at(o->V, c, layer - 1, pos);

    rmsnorm(h, L->attn_norm, dt, d, c->rms_eps, a);
    matvec(L->wq, dt, qd, d, a, q);
    matvec(L->wk, dt, kvd, d, a, kk);
    matvec(L->wv, dt, kvd, d, a, vv);
    for (int i = 0; i < H; ++i) rope(q + i * hd, hd, pos, c->rope_base);
    for (int i = 0; i < Hkv; ++i) rope(kk + i * hd, hd, pos, c->rope_base);
    if (c->kv_round_bf16)
        for (int i = 0; i < kvd; ++i) { kk[i] = round_bf16(kk[i]); vv[i] = round_bf16(vv[i]); }

    int group = H / Hkv;
    for (int i = 0; i < H; ++i) {
        int kh = i / group;
        double mx = -INFINITY;
        for (int t = 0; t <= pos; ++t) {
            const double* kt = kv_at(o->K, c, layer - 1, t) + kh * hd;
            double s = 0.0;
            for (int e = 0; e < hd; ++e) s += q[i * hd + e] * kt[e];
            s /= sqrt((double)hd);
            sc[t] = s;
            if (s > mx) mx = s;
        }
        double den = 0.0;
        for (int t = 0; t <= pos; ++t) { sc[t] = exp(sc[t] - mx); den += sc[t]; }
        for (int e = 0; e < hd; ++e) att[i * hd + e] = 0.0;
        for (int t = 0; t <= pos; ++t) {
            const double* vt = kv_at(o->V, c, layer - 1, t) + kh * hd;
            double p = sc[t] / den;
            for (int e = 0; e < hd; ++e) att[i * hd + e] += p * vt[e];
        }
    }
    matvec(L->wo, dt, d, qd, att, proj);
    for (int i = 0; i < d; ++i) h[i] += proj[i];

    rmsnorm(h, L->mlp_norm, dt, d, c->rms_eps, a);
    matvec(L->w_gate, dt, F, d, a, gate);
    matvec(L->w_up, dt, F, d, a, up);
    for (int i = 0; i < F; ++i) gate[i] = gate[i] / (1.0 + exp(-gate[i])) * up[i]; /* silu(g) * u */
    matvec(L->w_down, dt, d, F, gate, proj);
    for (int i = 0; i < d; ++i) h[i] += proj[i];

    free(a); free(q); free(att); free(proj); free(gate); free(up); free(sc);
}

static void embed_row(const orc_ctx* o, int tok, double* h) {
    for (int i = 0; i < o->c.d_model; ++i) h[i] = wget(o->w.embed, o->c.wdtype, (size_t)tok * o->c.d_model + i);
}

/* logits of the shared LM head on the final-RMSNorm of h */
static void head_logits(const orc_ctx* o, const double* h, double* z) {
    int d = o->c.d_model;
    double* x = malloc(sizeof(double) * d);
    rmsnorm(h, o->w.final_norm, o->c.wdtype, d, o->c.rms_eps, x);
    matvec(o->w.lm_head, o->c.wdtype, o->c.vocab, d, x, z);
    free(x);
}

/* logits of the exit test after layer `layer` (1-based): that layer's own head if one was set */
static void exit_logits(const orc_ctx* o, int layer, const double* h, double* z) {
    int d = o->c.d_model;
    const void* head = o->exit_head[layer - 1] ? o->exit_head[layer - 1] : o->w.lm_head;
    const void* gain = o->exit_norm[layer - 1] ? o->exit_norm[layer - 1] : o->w.final_norm;
    double* x = malloc(sizeof(double) * d);
    rmsnorm(h, gain, o->c.wdtype, d, o->c.rms_eps, x);
    matvec(head, o->c.wdtype, o->c.vocab, d, x, z);
    free(x);
}

static int argmax_first(const double* z, int n) {
    int t = 0;
    for (int v = 1; v < n; ++v) if (z[v] > z[t]) t = v; /* ties: lowest index */
    return t;
}

/* ---- sampling decoding (Section 4.3, decoding strategies; Table 2) ---- */

/* Counter-based uniform number in (0,1): the splitmix64 output function applied to
 * seed + (pos+1) * golden-ratio increment, i.e. for seed 0 the (pos+1)-th output of
 * the published splitmix64 stream; top 53 bits, centred in their cell. */
uint64_t orc_mix64(uint64_t seed, int64_t pos) {
    uint64_t x = seed + 0x9E3779B97F4A7C15ull * (uint64_t)(pos + 1);
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}
double orc_uniform(uint64_t seed, int64_t pos) {
    return ((double)(orc_mix64(seed, pos) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

/* Nucleus of top-p sampling, as a logit threshold: the largest logit value z* such that the tokens
 * with z_v >= z* hold at least top_p of the mass of softmax(z / temperature).  The nucleus is
 * {v : z_v >= z*}: tokens in descending order of probability until top_p is reached, equal logits
 * entering together.  top_p >= 1: -infinity (every token). */
static const double* g_sort_key;
static int by_logit_desc(const void* a, const void* b) {
    double x = g_sort_key[*(const int*)a], y = g_sort_key[*(const int*)b];
    if (x != y) return x > y ? -1 : 1;
    return *(const int*)a - *(const int*)b;
}
double orc_nucleus_threshold(const double* z, int V, double temperature, double top_p) {
    if (!(top_p < 1.0)) return -INFINITY;
    double m = z[0];
    for (int v = 1; v < V; ++v) if (z[v] > m) m = z[v];
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += exp((z[v] - m) / temperature);
    int* idx = malloc(sizeof(int) * V);
    for (int v = 0; v < V; ++v) idx[v] = v;
    g_sort_key = z;
    qsort(idx, V, sizeof(int), by_logit_desc);
    double acc = 0.0, zstar = z[idx[V - 1]];
    for (int k = 0; k < V; ++k) {
        acc += exp((z[idx[k]] - m) / temperature);
        int group_ends = k == V - 1 || z[idx[k + 1]] != z[idx[k]];
        if (group_ends && acc >= top_p * total) { zstar = z[idx[k]]; break; }
    }
    free(idx);
    return zstar;
}

/* Inverse-CDF sample, in vocabulary order, of softmax(z / temperature) restricted to the top-p
 * nucleus (top_p >= 1: all tokens) and renormalised: the first nucleus token whose cumulative
 * un-normalised mass reaches u * (mass of the nucleus).  slack (nullable) receives the distance
 * from u to the nearer edge of the chosen token's CDF interval. */
int orc_sample_token(const double* z, int V, double temperature, double top_p, double u, double* slack) {
    double m = z[0];
    for (int v = 1; v < V; ++v) if (z[v] > m) m = z[v];
    double zstar = orc_nucleus_threshold(z, V, temperature, top_p);
    double total = 0.0;
    for (int v = 0; v < V; ++v) if (z[v] >= zstar) total += exp((z[v] - m) / temperature);
    double target = u * total, run = 0.0;
    int pick = -1;
    double lo = 0.0;
    for (int v = 0; v < V; ++v) {
        if (!(z[v] >= zstar)) continue;
        double e = exp((z[v] - m) / temperature);
        if (e > 0.0) pick = v;                      /* rounding guard: last token with mass */
        if (run + e >= target) { pick = v; lo = run; run += e; break; }
        run += e;
        lo = run;
    }
    if (slack) {
        double a = target - lo, b = run - target;
        *slack = (a < b ? a : b) / total;
    }
    return pick;
}


/* The decoding rule at the last layer: greedy top-1, or (temperature > 0) the inverse-CDF
 * sample at u(seed, pos), pos = sequence position of the token being produced. */
static int next_token(const orc_ctx* o, const double* z, int pos, double* slack) {
    if (o->sample_temperature > 0.0)
        return orc_sample_token(z, o->c.vocab, o->sample_temperature, o->sample_top_p, orc_uniform(o->sample_seed, pos), slack);
    return argmax_first(z, o->c.vocab);
}
void orc_set_sampling(orc_ctx* o, double temperature, double top_p, uint64_t seed) {
    o->sample_temperature = temperature > 0.0 ? temperature : 0.0;
    o->sample_top_p = top_p > 0.0 && top_p < 1.0 ? top_p : 1.0;
    o->sample_seed = seed;
}

/* Eq. 2: p = max softmax(z / T) = 1 / sum_v exp((z_v - z_max)/T); token = argmax z */
static void confidence_from_logits(const double* z, int V, double T, double* conf, int* token) {
    int t = argmax_first(z, V);
    double s = 0.0;
    for (int v = 0; v < V; ++v) s += exp((z[v] - z[t]) / T);
    *conf = 1.0 / s;
    *token = t;
}

/* ---------------------------------------------------------------- public */

orc_ctx* orc_create(const orc_config* cfg, const orc_weights* w) {
    orc_ctx* o = calloc(1, sizeof(orc_ctx));
    o->c = *cfg;
    o->w = *w;
    o->layers = malloc(sizeof(orc_layer) * cfg->n_layers);
    memcpy(o->layers, w->layers, sizeof(orc_layer) * cfg->n_layers);
    size_t n = (size_t)cfg->n_layers * cfg->max_seq * cfg->n_kv_heads * cfg->head_dim;
    o->K = calloc(n, sizeof(double));
    o->V = calloc(n, sizeof(double));
    o->exit_head = calloc(cfg->n_layers, sizeof(void*));
    o->exit_norm = calloc(cfg->n_layers, sizeof(void*));
    if (!o->K || !o->V) { free(o->K); free(o->V); free(o->layers); free(o->exit_head); free(o->exit_norm); free(o); return NULL; }
    return o;
}

void orc_destroy(orc_ctx* o) {
    if (!o) return;
    free(o->K); free(o->V); free(o->layers); free(o->exit_head); free(o->exit_norm); free(o);
}

/* Head ([vocab, d_model], storage dtype) and norm gain ([d_model]) of the exit test after `layer`; NULL = shared. */
void orc_set_exit_head(orc_ctx* o, int layer, const void* head, const void* norm) {
    o->exit_head[layer - 1] = head;
    o->exit_norm[layer - 1] = norm;
}

/* Exit test of Section 3.2 after layer `layer` on one hidden state, with that layer's head. */
void orc_exit_confidence_at(orc_ctx* o, int layer, const double* h, double T, double* conf, int32_t* token) {
    double* z = malloc(sizeof(double) * o->c.vocab);
    int t;
    exit_logits(o, layer, h, z);
    confidence_from_logits(z, o->c.vocab, T, conf, &t);
    *token = t;
    free(z);
}

/* Section 3.2, Eq. 1: T_l = 1 + alpha (1 - l/L), l = 1..L, out[l-1] */
void orc_tau_schedule(double alpha, int L, double* out) {
    for (int l = 1; l <= L; ++l) out[l - 1] = 1.0 + alpha * (1.0 - (double)l / L);
}

/* Section 3.4, Eq. 3: T_round / T_AR */
double orc_round_cost(int L, int w, int d_max) { return ((double)w * d_max + L - d_max) / L; }

/* Section 3.4, Eq. 4 (left side, the sum as printed) */
double orc_expected_accepted(double a, int w) {
    double s = 0.0;
    for (int k = 0; k < w; ++k) s += k * pow(a, k) * (1.0 - a);
    return s + w * pow(a, w);
}

/* Section 3.4, Eq. 5 */
double orc_speedup(int L, double a, int w, int d_max) {
    return L * a * (1.0 - pow(a, w)) / ((1.0 - a) * ((double)w * d_max + L - d_max));
}

/* Exit test of Section 3.2 on one hidden state. logits_out may be NULL. */
void orc_exit_confidence(orc_ctx* o, const double* h, double T, double* conf, int32_t* token, double* logits_out) {
    double* z = malloc(sizeof(double) * o->c.vocab);
    int t;
    head_logits(o, h, z);
    confidence_from_logits(z, o->c.vocab, T, conf, &t);
    *token = t;
    if (logits_out) memcpy(logits_out, z, sizeof(double) * o->c.vocab);
    free(z);
}

/* Confidence of a given logit vector (Eq. 2 alone). */
void orc_confidence(const double* z, int V, double T, double* conf, int32_t* token) {
    int t;
    confidence_from_logits(z, V, T, conf, &t);
    *token = t;
}

/* Load cache contents for one layer and position (kernel-level parity cases). */
void orc_set_kv(orc_ctx* o, int layer, int pos, const double* k, const double* v) {
    size_t kvd = (size_t)o->c.n_kv_heads * o->c.head_dim;
    memcpy(kv_at(o->K, &o->c, layer - 1, pos), k, kvd * sizeof(double));
    memcpy(kv_at(o->V, &o->c, layer - 1, pos), v, kvd * sizeof(double));
}

void orc_get_kv(orc_ctx* o, int layer, int pos, double* k, double* v) {
    size_t kvd = (size_t)o->c.n_kv_heads * o->c.head_dim;
    memcpy(k, kv_at(o->K, &o->c, layer - 1, pos), kvd * sizeof(double));
    memcpy(v, kv_at(o->V, &o->c, layer - 1, pos), kvd * sizeof(double));
}

/* One layer for m rows at consecutive positions first_pos.., h is [m][d] in/out.
 * Rows go in position order, so each sees the K,V of the rows before it. */
void orc_layer_forward(orc_ctx* o, int layer, double* h, int m, int first_pos) {
    for (int i = 0; i < m; ++i) layer_row(o, layer, h + (size_t)i * o->c.d_model, first_pos + i);
}

void orc_embed(orc_ctx* o, int tok, double* h) { embed_row(o, tok, h); }

void orc_final_logits(orc_ctx* o, const double* h, double* z) { head_logits(o, h, z); }

/* Full-depth forward of one token at `pos` using the cache; returns the token the decoding
 * rule produces for position pos + 1 (greedy unless sampling is set), optionally the logits. */
static int full_step(orc_ctx* o, int tok, int pos, double* z_out) {
    int d = o->c.d_model, V = o->c.vocab;
    double* h = malloc(sizeof(double) * d);
    double* z = z_out ? z_out : malloc(sizeof(double) * V);
    embed_row(o, tok, h);
    for (int l = 1; l <= o->c.n_layers; ++l) layer_row(o, l, h, pos);
    head_logits(o, h, z);
    int t = next_token(o, z, pos + 1, NULL);
    if (!z_out) free(z);
    free(h);
    return t;
}

/* Prefill: every prompt token through all layers; returns the first generated token. */
int orc_prefill(orc_ctx* o, const int32_t* prompt, int n_prompt) {
    int t = -1;
    for (int p = 0; p < n_prompt; ++p) t = full_step(o, prompt[p], p, NULL);
    return t;
}

/* Plain autoregressive decoding (greedy, or sampling when set): the definition of the correct
 * output.  margins (nullable) receives top1 - top2 of the final logits behind each token; under
 * sampling, the distance from u to the nearer edge of the chosen token's CDF interval. */
int orc_ar_generate(orc_ctx* o, const int32_t* prompt, int n_prompt, int n_gen, int32_t* out, double* margins) {
    if (n_prompt < 1 || n_prompt + n_gen > o->c.max_seq) return -1;
    int V = o->c.vocab;
    double* z = malloc(sizeof(double) * V);
    int tok = -1;
    for (int p = 0; p < n_prompt + n_gen - 1; ++p) {
        int in = p < n_prompt ? prompt[p] : out[p - n_prompt];
        tok = full_step(o, in, p, z);
        if (p >= n_prompt - 1) {
            out[p - n_prompt + 1] = tok;
            if (margins && o->sample_temperature > 0.0) {
                next_token(o, z, p + 1, &margins[p - n_prompt + 1]);   /* CDF slack instead of a logit margin */
            } else if (margins) {
                double second = -INFINITY;
                for (int v = 0; v < V; ++v) if (v != tok && z[v] > second) second = z[v];
                margins[p - n_prompt + 1] = z[tok] - second;
            }
        }
    }
    free(z);
    return n_gen;
}

/* Brute force: no cache is carried between tokens.  For every generated token the
 * whole prefix is recomputed from the embeddings, as a sequence-level forward with
 * its own local K/V arrays (a different organisation of the same mathematics). */
int orc_bruteforce_generate(orc_ctx* o, const int32_t* prompt, int n_prompt, int n_gen, int32_t* out) {
    const orc_config* c = &o->c;
    int d = c->d_model, H = c->n_heads, Hkv = c->n_kv_heads, hd = c->head_dim, F = c->d_ffn, V = c->vocab;
    int qd = H * hd, kvd = Hkv * hd, dt = c->wdtype, group = H / Hkv;
    int maxn = n_prompt + n_gen;
    int32_t* toks = malloc(sizeof(int32_t) * maxn);
    memcpy(toks, prompt, sizeof(int32_t) * n_prompt);
    double* X = malloc(sizeof(double) * maxn * d);
    double* A = malloc(sizeof(double) * maxn * d);
    double* Q = malloc(sizeof(double) * maxn * qd);
    double* Kl = malloc(sizeof(double) * maxn * kvd);
    double* Vl = malloc(sizeof(double) * maxn * kvd);
    double* O = malloc(sizeof(double) * maxn * qd);
    double* G = malloc(sizeof(double) * F);
    double* U = malloc(sizeof(double) * F);
    double* P = malloc(sizeof(double) * d);
    double* sc = malloc(sizeof(double) * maxn);
    double* z = malloc(sizeof(double) * V);
    for (int gi = 0; gi < n_gen; ++gi) {
        int n = n_prompt + gi;
        for (int p = 0; p < n; ++p) embed_row(o, toks[p], X + (size_t)p * d);
        for (int l = 0; l < c->n_layers; ++l) {
            const orc_layer* L = &o->layers[l];
            for (int p = 0; p < n; ++p) {
                rmsnorm(X + (size_t)p * d, L->attn_norm, dt, d, c->rms_eps, A + (size_t)p * d);
                matvec(L->wq, dt, qd, d, A + (size_t)p * d, Q + (size_t)p * qd);
                matvec(L->wk, dt, kvd, d, A + (size_t)p * d, Kl + (size_t)p * kvd);
                matvec(L->wv, dt, kvd, d, A + (size_t)p * d, Vl + (size_t)p * kvd);
                for (int i = 0; i < H; ++i) rope(Q + (size_t)p * qd + i * hd, hd, p, c->rope_base);
                for (int i = 0; i < Hkv; ++i) rope(Kl + (size_t)p * kvd + i * hd, hd, p, c->rope_base);
                if (c->kv_round_bf16)
                    for (int i = 0; i < kvd; ++i) {
                        Kl[(size_t)p * kvd + i] = round_bf16(Kl[(size_t)p * kvd + i]);
                        Vl[(size_t)p * kvd + i] = round_bf16(Vl[(size_t)p * kvd + i]);
                    }
            }
            for (int p = 0; p < n; ++p)
                for (int i = 0; i < H; ++i) {
                    int kh = i / group;
                    double mx = -INFINITY, den = 0.0;
                    for (int t = 0; t <= p; ++t) {
                        double s = 0.0;
                        for (int e = 0; e < hd; ++e) s += Q[(size_t)p * qd + i * hd + e] * Kl[(size_t)t * kvd + kh * hd + e];
                        sc[t] = s / sqrt((double)hd);
                        if (sc[t] > mx) mx = sc[t];
                    }
                    for (int t = 0; t <= p; ++t) { sc[t] = exp(sc[t] - mx); den += sc[t]; }
                    for (int e = 0; e < hd; ++e) {
                        double acc = 0.0;
                        for (int t = 0; t <= p; ++t) acc += sc[t] / den * Vl[(size_t)t * kvd + kh * hd + e];
                        O[(size_t)p * qd + i * hd + e] = acc;
                    }
                }
            for (int p = 0; p < n; ++p) {
                double* x = X + (size_t)p * d;
                matvec(L->wo, dt, d, qd, O + (size_t)p * qd, P);
                for (int i = 0; i < d; ++i) x[i] += P[i];
                rmsnorm(x, L->mlp_norm, dt, d, c->rms_eps, A);
                matvec(L->w_gate, dt, F, d, A, G);
                matvec(L->w_up, dt, F, d, A, U);
                for (int i = 0; i < F; ++i) G[i] = G[i] / (1.0 + exp(-G[i])) * U[i];
                matvec(L->w_down, dt, d, F, G, P);
                for (int i = 0; i < d; ++i) x[i] += P[i];
            }
        }
        head_logits(o, X + (size_t)(n - 1) * d, z);
        toks[n] = out[gi] = next_token(o, z, n, NULL);
    }
    free(toks); free(X); free(A); free(Q); free(Kl); free(Vl); free(O); free(G); free(U); free(P); free(sc); free(z);
    return n_gen;
}

/* Teacher-forced check: one causal pass over tokens[0..n_total); for each position
 * p in [from-1, n_total-1) reports about the prediction of token p+1:
 * top1, top2, margin = z[top1]-z[top2], and z[tokens[p+1]] - z[top1] (0 when equal). */
int orc_teacher_forced(orc_ctx* o, const int32_t* tokens, int n_total, int from,
                       int32_t* top1, int32_t* top2, double* margin, double* deficit) {
    if (n_total > o->c.max_seq || from < 1) return -1;
    int V = o->c.vocab;
    double* z = malloc(sizeof(double) * V);
    for (int p = 0; p < n_total - 1; ++p) {
        if (p < from - 1) { full_step(o, tokens[p], p, z); continue; }
        full_step(o, tokens[p], p, z);
        int t1 = argmax_first(z, V);
        int t2 = -1;
        for (int v = 0; v < V; ++v) if (v != t1 && (t2 < 0 || z[v] > z[t2])) t2 = v;
        int k = p - (from - 1);
        top1[k] = t1; top2[k] = t2; margin[k] = z[t1] - z[t2];
        deficit[k] = z[tokens[p + 1]] - z[t1];
    }
    free(z);
    return n_total - from;
}

/* The round loop of Section 3.3 (bounded speculation with cached states).
 *
 * script / script_len: optional scripted exit decisions replacing the test
 *   p >= threshold for the first script_len drafted rows (in drafting order):
 *   script[k] = e >= 1 -> row k exits at layer e with that layer's greedy token;
 *   script[k] = 0      -> row k does not exit (difficult token).
 * tau[l-1] <= 0: layer l is not tested for an exit (probe-layer mask); scripted or not, no row exits there.
 * rounds / max_rounds: optional trace. Returns the number of rounds, or -1. */
int orc_specbound_generate(orc_ctx* o, const int32_t* prompt, int n_prompt, int n_gen,
                           int d_max, int w_max, const double* tau, double threshold,
                           const int32_t* script, int script_len,
                           int32_t* out, orc_round* rounds, int max_rounds) {
    const orc_config* c = &o->c;
    int d = c->d_model, L = c->n_layers, V = c->vocab;
    if (n_prompt < 1 || d_max < 1 || d_max > L || w_max < 1 || w_max > ORC_MAX_W) return -1;
    if (n_prompt + n_gen + w_max > c->max_seq) return -1;
    double* h = malloc(sizeof(double) * ORC_MAX_W * d); /* hidden-state cache: one vector per row */
    double* z = malloc(sizeof(double) * V);
    int depth[ORC_MAX_W];
    int n_rounds = 0, n_out = 0, drafted = 0;

    int pending = orc_prefill(o, prompt, n_prompt); /* first generated token, full depth */
    int n = n_prompt;                               /* positions complete in every layer */
    if (n_gen > 0) out[n_out++] = pending;

    while (n_out < n_gen) {
        orc_round R;
        memset(&R, 0, sizeof(R));
        int w = 0, cur = pending;
        for (;;) {                                  /* draft phase: one new row per iteration */
            int r = w++;
            embed_row(o, cur, h + (size_t)r * d);
            depth[r] = 0; R.draft[r] = -1; R.exit_layer[r] = 0;
            int exited = 0;
            int scripted = script && drafted < script_len;
            int scripted_exit = scripted ? script[drafted] : 0;
            ++drafted;
            for (int l = 1; l <= d_max; ++l) {
                /* rows whose depth is l-1 form a suffix ending in the new row: run layer l on them */
                int r0 = r;
                while (r0 > 0 && depth[r0 - 1] == l - 1) --r0;
                orc_layer_forward(o, l, h + (size_t)r0 * d, r + 1 - r0, n + r0);
                for (int i = r0; i <= r; ++i) { depth[i] = l; R.layers_done[i]++; }
                R.layer_steps++;
                /* probe-layer mask (a reading of Section 3.2's "first layer where p >= threshold" for callers that
                 * do not want every layer tested): a layer whose temperature is <= 0 is walked but not tested,
                 * so no exit can happen there */
                if (!(tau[l - 1] > 0.0)) continue;
                double p; int t;
                exit_logits(o, l, h + (size_t)r * d, z);
                confidence_from_logits(z, V, tau[l - 1], &p, &t);
                R.probes++;
                R.conf[r] = p;
                int take = scripted ? (scripted_exit == l) : (p >= threshold);
                if (take) { R.draft[r] = t; R.exit_layer[r] = l; exited = 1; break; }
            }
            for (int i = 0; i < w; ++i) R.depth_after[r][i] = depth[i];
            if (!exited) break;                     /* depth bound: difficult token ends the round */
            if (w == w_max) break;                  /* width bound: long shallow chain ends the round */
            cur = R.draft[r];
        }
        int D = 0;
        for (int i = 0; i < w; ++i) if (depth[i] > D) D = depth[i];
        for (int l = 1; l <= D; ++l) {              /* alignment to the deepest row */
            int r0 = w;
            while (r0 > 0 && depth[r0 - 1] == l - 1) --r0;
            if (r0 == w) continue;
            orc_layer_forward(o, l, h + (size_t)r0 * d, w - r0, n + r0);
            for (int i = r0; i < w; ++i) { depth[i] = l; R.layers_done[i]++; }
            R.layer_steps++;
        }
        for (int l = D + 1; l <= L; ++l) {          /* unified parallel pass */
            orc_layer_forward(o, l, h, w, n);
            for (int i = 0; i < w; ++i) R.layers_done[i]++;
            R.layer_steps++;
        }
        for (int i = 0; i < w; ++i) {
            head_logits(o, h + (size_t)i * d, z);
            R.g[i] = next_token(o, z, n + i + 1, NULL);   /* row i holds position n+i and predicts n+i+1 */
        }
        /* greedy acceptance: the longest prefix of drafts the full model reproduces, then the
         * model's own token at the first row that had no draft or a wrong one */
        int acc = 0;
        while (acc < w && R.draft[acc] >= 0 && R.g[acc] == R.draft[acc]) ++acc;
        int emit = acc < w ? acc + 1 : w;
        if (emit > n_gen - n_out) emit = n_gen - n_out; /* truncate an overshooting round */
        for (int i = 0; i < emit; ++i) out[n_out++] = R.g[i];
        n += emit;                                   /* rollback: positions >= n are dead */
        pending = R.g[emit - 1];
        R.w = w; R.D = D; R.emitted = emit;
        R.accepted_drafts = acc;                     /* rows 0..acc-1 had their draft confirmed */
        if (rounds && n_rounds < max_rounds) rounds[n_rounds] = R;
        ++n_rounds;
    }
    free(h); free(z);
    return n_rounds;
}
