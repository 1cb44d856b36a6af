/*
 * dbt_oracle.c -- CPU oracle for the Decode-Branch Transformer forward pass.
 *
 * TEST INFRASTRUCTURE ONLY (see dbt_oracle.h).  Plain loops, fp32 storage, double
 * accumulators, no blocking, no fusion, no SIMD intrinsics; OpenMP only on the outermost
 * loop of a routine.  Each routine names the passage of the paper it restates.
 *
 * Notation follows the paper: S_1/S_2 primary and branch residual states, N_i normalised
 * states, Q_1,K_1,V_1 primary projections, Q_2 and Q~_2 the branch query before and after
 * the a coupling, H_i the activated MLP intermediate, M_i the MLP output, z_1/z_2 logits,
 * p/q their softmaxes.  Stacked rows are path-major: rows 0..n-1 primary, then n rows per
 * decode branch (one branch in the main text; K-1 of them in Appendix C.1, "More decode
 * branches": own embedding each, shared coupling vectors, branch distributions averaged).
 */
#include "dbt_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

struct orc_model {
    orc_config cfg;
    orc_weights w;
    orc_layer_weights *layers; /* owned copy of the per-layer pointer table */
    float *kc, *vc;            /* [L][max_batch][max_seq][kv_dim]           */
    int32_t *len;              /* [max_batch] tokens already cached         */
    float *rlog;               /* MoE: router logits of the last step, [L][K][max_batch][E] */
};

static inline int paths_of(const orc_config *c) { return c->n_paths >= 2 ? c->n_paths : 2; }

/* ------------------------------------------------------------------------------------ */
/* storage helpers                                                                       */

static inline float bf16_bits_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* round-to-nearest-even fp32 -> bf16 -> fp32 (used only by the kv_round_bf16 switch) */
static inline float round_through_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return f; /* NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    u &= 0xffff0000u;
    memcpy(&f, &u, sizeof f);
    return f;
}

static inline size_t q_dim_of(const orc_config *c) { return (size_t)c->n_q_heads * c->head_dim; }
static inline size_t kv_dim_of(const orc_config *c) { return (size_t)c->n_kv_heads * c->head_dim; }

/* row `row` of matrix W [.,n_in] (dtype dt) dotted with x, accumulated in double */
static double dot_row(const void *W, int dt, size_t row, int n_in, const float *x) {
    double acc = 0.0;
    if (dt == 0) {
        const float *w = (const float *)W + row * (size_t)n_in;
        for (int k = 0; k < n_in; k++) acc += (double)w[k] * (double)x[k];
    } else {
        const uint16_t *w = (const uint16_t *)W + row * (size_t)n_in;
        for (int k = 0; k < n_in; k++) acc += (double)bf16_bits_to_f32(w[k]) * (double)x[k];
    }
    return acc;
}

/* copy row `row` of a [.,n] table (dtype dt) into fp32 */
static void fetch_row(const void *W, int dt, size_t row, int n, float *out) {
    if (dt == 0) {
        memcpy(out, (const float *)W + row * (size_t)n, sizeof(float) * (size_t)n);
    } else {
        const uint16_t *w = (const uint16_t *)W + row * (size_t)n;
        for (int k = 0; k < n; k++) out[k] = bf16_bits_to_f32(w[k]);
    }
}

static const void *mat_offset(const void *W, int dt, size_t elems) {
    return (const char *)W + elems * (dt == 0 ? 4u : 2u);
}

/* ------------------------------------------------------------------------------------ */
/* unit operations                                                                       */

/* RMSNorm(v; g) = g * v / sqrt(mean(v^2) + eps)   (Eq. embeddings and every "RMSNorm") */
void orc_rmsnorm(const float *x, const float *g, int n, float eps, float *y) {
    double ss = 0.0;
    for (int i = 0; i < n; i++) ss += (double)x[i] * (double)x[i];
    double inv = 1.0 / sqrt(ss / (double)n + (double)eps);
    for (int i = 0; i < n; i++) y[i] = (float)((double)g[i] * (double)x[i] * inv);
}

/* The paper's H W with W stored transposed: Y[r][i] = sum_k W[i][k] X[r][k]. */
void orc_linear(const void *W, int dt, int n_out, int n_in, const float *X, int R, float *Y) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < n_out; i++)
        for (int r = 0; r < R; r++)
            Y[(size_t)r * n_out + i] = (float)dot_row(W, dt, (size_t)i, n_in, X + (size_t)r * n_in);
}

/* RoPE with half-split pairs (i, i + d_h/2), angle t * base^(-2i/d_h), 0-based t. */
void orc_rope(float *x, int n_heads, int head_dim, int t, float base) {
    int half = head_dim / 2;
    for (int h = 0; h < n_heads; h++) {
        float *v = x + (size_t)h * head_dim;
        for (int i = 0; i < half; i++) {
            double theta = (double)t * pow((double)base, -2.0 * (double)i / (double)head_dim);
            double c = cos(theta), s = sin(theta);
            double x0 = v[i], x1 = v[i + half];
            v[i] = (float)(x0 * c - x1 * s);
            v[i + half] = (float)(x1 * c + x0 * s);
        }
    }
}

/* softmax(u.K_j / sqrt(d_h)) V over the n_keys visible positions (Background, attention Eq.) */
void orc_attend(const float *u, const float *K, const float *V, int n_keys, int stride,
                int head_dim, float *o) {
    double *sc = (double *)malloc(sizeof(double) * (size_t)n_keys);
    double scale = 1.0 / sqrt((double)head_dim);
    double mx = -INFINITY;
    for (int j = 0; j < n_keys; j++) {
        const float *kj = K + (size_t)j * stride;
        double acc = 0.0;
        for (int i = 0; i < head_dim; i++) acc += (double)u[i] * (double)kj[i];
        sc[j] = acc * scale;
        if (sc[j] > mx) mx = sc[j];
    }
    double den = 0.0;
    for (int j = 0; j < n_keys; j++) {
        sc[j] = exp(sc[j] - mx);
        den += sc[j];
    }
    for (int i = 0; i < head_dim; i++) {
        double acc = 0.0;
        for (int j = 0; j < n_keys; j++) acc += sc[j] * (double)V[(size_t)j * stride + i];
        o[i] = (float)(acc / den);
    }
    free(sc);
}

/* gated MLP activation: H = SiLU(gate) * up */
void orc_swiglu(const float *g, const float *u, int n, float *h) {
    for (int i = 0; i < n; i++) {
        double x = g[i];
        h[i] = (float)(x / (1.0 + exp(-x)) * (double)u[i]);
    }
}

/* I = TopK(r, k); w = softmax(r)[I] / sum(softmax(r)[I])   (Eq. moe_layer; Section 4.3) */
void orc_route(const float *logits, int E, int k, const int32_t *forced, int32_t *idx, float *wts) {
    double *p = (double *)malloc(sizeof(double) * (size_t)E);
    double mx = -INFINITY, den = 0.0;
    for (int e = 0; e < E; e++)
        if ((double)logits[e] > mx) mx = logits[e];
    for (int e = 0; e < E; e++) {
        p[e] = exp((double)logits[e] - mx);
        den += p[e];
    }
    for (int e = 0; e < E; e++) p[e] /= den;
    if (forced) {
        for (int j = 0; j < k; j++) idx[j] = forced[j];
    } else {
        char *taken = (char *)calloc((size_t)E, 1);
        for (int j = 0; j < k; j++) { /* k passes of "largest not yet taken, lowest index first" */
            int best = -1;
            for (int e = 0; e < E; e++)
                if (!taken[e] && (best < 0 || p[e] > p[best])) best = e;
            taken[best] = 1;
            idx[j] = best;
        }
        free(taken);
    }
    double sel = 0.0;
    for (int j = 0; j < k; j++) sel += p[idx[j]];
    for (int j = 0; j < k; j++) wts[j] = (float)(p[idx[j]] / sel);
    free(p);
}

/* p = softmax(z1), q_j = softmax(zb_j) for the nb decode branches, qbar = mean_j q_j
 * (Appendix C.1; nb = 1 is the main text's single q), alpha = clip_[0.5,1](sum_v p_v^2),
 * mix = alpha p + (1-alpha) qbar, greedy token = argmax mix (lowest index on ties).
 * zb is [nb][V]. */
int orc_readout_multi(const float *z1, const float *zb, int nb, int V, float *alpha, float *mix) {
    double m1 = -INFINITY, d1 = 0.0;
    double *mb = (double *)malloc(sizeof(double) * (size_t)nb);
    double *db = (double *)malloc(sizeof(double) * (size_t)nb);
    for (int v = 0; v < V; v++)
        if ((double)z1[v] > m1) m1 = z1[v];
    for (int v = 0; v < V; v++) d1 += exp((double)z1[v] - m1);
    for (int j = 0; j < nb; j++) {
        const float *z = zb + (size_t)j * V;
        mb[j] = -INFINITY;
        db[j] = 0.0;
        for (int v = 0; v < V; v++)
            if ((double)z[v] > mb[j]) mb[j] = z[v];
        for (int v = 0; v < V; v++) db[j] += exp((double)z[v] - mb[j]);
    }
    double coll = 0.0;
    for (int v = 0; v < V; v++) {
        double p = exp((double)z1[v] - m1) / d1;
        coll += p * p;
    }
    double a = coll;
    if (a < 0.5) a = 0.5;
    if (a > 1.0) a = 1.0;
    int best = 0;
    double bestv = -1.0;
    for (int v = 0; v < V; v++) {
        double p = exp((double)z1[v] - m1) / d1;
        double qbar = 0.0;
        for (int j = 0; j < nb; j++) qbar += exp((double)zb[(size_t)j * V + v] - mb[j]) / db[j];
        qbar /= (double)nb;
        double mv = a * p + (1.0 - a) * qbar;
        if (mix) mix[v] = (float)mv;
        if (mv > bestv) {
            bestv = mv;
            best = v;
        }
    }
    if (alpha) *alpha = (float)a;
    free(mb); free(db);
    return best;
}

/* The main text's two-path readout (Eq. alpha, Eq. mixloss): one decode branch. */
int orc_readout(const float *z1, const float *z2, int V, float *alpha, float *mix) {
    return orc_readout_multi(z1, z2, 1, V, alpha, mix);
}

static int argmax_f32(const float *z, int n) {
    int best = 0;
    for (int i = 1; i < n; i++)
        if (z[i] > z[best]) best = i;
    return best;
}

void orc_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
int orc_get_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------ */
/* MLP sub-layers on `paths` stacked groups of n rows: m = [N_1; N_2; ...] (group 0 primary) */

/* Eq. mlp: M_1 = H_1 W_D ; H~_j = H_j + b*H_1 ; M_j = H~_j W_D + c*M_1 for every branch j
 * (b, c shared by the branches: Appendix C.1). */
static void mlp_dense(const orc_config *c, const orc_layer_weights *lw, const float *m, int paths,
                      int n, float *M) {
    int d = c->d_model, F = c->d_ff, dt = c->weight_dtype;
    float *g = (float *)malloc(sizeof(float) * (size_t)n * F);
    float *u = (float *)malloc(sizeof(float) * (size_t)n * F);
    float *H1 = (float *)malloc(sizeof(float) * (size_t)n * F);
    float *Hj = (float *)malloc(sizeof(float) * (size_t)n * F);
    orc_linear(lw->w_gate, dt, F, d, m, n, g);
    orc_linear(lw->w_up, dt, F, d, m, n, u);
    orc_swiglu(g, u, n * F, H1);
    orc_linear(lw->w_down, dt, d, F, H1, n, M);
    for (int p = 1; p < paths; p++) {
        const float *mj = m + (size_t)p * n * d;
        float *Mj = M + (size_t)p * n * d;
        orc_linear(lw->w_gate, dt, F, d, mj, n, g);
        orc_linear(lw->w_up, dt, F, d, mj, n, u);
        orc_swiglu(g, u, n * F, Hj);
        for (int r = 0; r < n; r++)
            for (int i = 0; i < F; i++)
                Hj[(size_t)r * F + i] += lw->coup_b[i] * H1[(size_t)r * F + i];
        orc_linear(lw->w_down, dt, d, F, Hj, n, Mj);
        for (int r = 0; r < n; r++)
            for (int i = 0; i < d; i++)
                Mj[(size_t)r * d + i] += lw->coup_c[i] * M[(size_t)r * d + i];
    }
    free(g); free(u); free(H1); free(Hj);
}

/* Eq. moe_layer with per-path fan-out (Eq. moe_budget), un-gated shared experts
 * (M_i = R_i + G(N_i), Appendix B.3) and the c coupling on the total primary output.
 * Compute-matched allocation (Appendix B.3, Eq. matched_shared_expert): the shared expert
 * is evaluated on the primary state only, M_j = R_j(N_j;k_2) + g_G * G(N_1), no b, no c.
 * Every decode branch routes for itself with fan-out k_2 (router replay: with the primary's
 * expert set).  forced / chosen: [paths][n][kmax] slices for this layer (nullable);
 * logits_out: [paths][ld_logits][E] router logits of this layer (nullable). */
static void mlp_moe(const orc_config *c, const orc_layer_weights *lw, const float *m, int paths,
                    int n, const int32_t *forced, int32_t *chosen, float *logits_out, int ld_logits,
                    float *Mout) {
    int d = c->d_model, E = c->n_experts, Fe = c->d_expert, dt = c->weight_dtype;
    int Fs = c->n_shared_experts * Fe;
    int kmax = c->k_primary > c->k_branch ? c->k_primary : c->k_branch;
    float *logits = (float *)malloc(sizeof(float) * (size_t)E);
    float *g = (float *)malloc(sizeof(float) * (size_t)(Fe > Fs ? Fe : Fs));
    float *u = (float *)malloc(sizeof(float) * (size_t)(Fe > Fs ? Fe : Fs));
    float *h = (float *)malloc(sizeof(float) * (size_t)(Fe > Fs ? Fe : Fs));
    float *y = (float *)malloc(sizeof(float) * (size_t)d);
    double *acc = (double *)malloc(sizeof(double) * (size_t)d);
    float *Hs1 = (float *)malloc(sizeof(float) * (size_t)n * (Fs > 0 ? Fs : 1));
    float *G1 = (float *)calloc((size_t)n * d, sizeof(float)); /* G(N_1), zero without shared experts */
    int matched = c->compute_matched;
    int32_t idx[64];
    float wts[64];
    int32_t *idx1 = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * kmax);
    const float *M1 = Mout;

    for (int p = 0; p < paths; p++) {
        for (int r = 0; r < n; r++) {
            const float *mr = m + ((size_t)p * n + r) * d;
            float *M = Mout + ((size_t)p * n + r) * d;
            int k = p ? c->k_branch : c->k_primary;
            const int32_t *f = forced ? forced + ((size_t)p * n + r) * kmax : NULL;
            orc_linear(lw->router, dt, E, d, mr, 1, logits);
            if (logits_out) memcpy(logits_out + ((size_t)p * ld_logits + r) * E, logits, sizeof(float) * (size_t)E);
            if (p >= 1 && c->router_mode == 1) { /* router replay: I_j := I_1, own weights */
                k = c->k_primary;
                f = idx1 + (size_t)r * kmax;
            }
            orc_route(logits, E, k, f, idx, wts);
            if (p == 0) memcpy(idx1 + (size_t)r * kmax, idx, sizeof(int32_t) * (size_t)k);
            if (chosen) {
                int32_t *co = chosen + ((size_t)p * n + r) * kmax;
                for (int j = 0; j < kmax; j++) co[j] = j < k ? idx[j] : -1;
            }
            for (int i = 0; i < d; i++) acc[i] = 0.0;
            for (int j = 0; j < k; j++) { /* routed experts, weighted */
                size_t e = (size_t)idx[j];
                orc_linear(mat_offset(lw->exp_gate, dt, e * Fe * d), dt, Fe, d, mr, 1, g);
                orc_linear(mat_offset(lw->exp_up, dt, e * Fe * d), dt, Fe, d, mr, 1, u);
                orc_swiglu(g, u, Fe, h);
                orc_linear(mat_offset(lw->exp_down, dt, e * (size_t)d * Fe), dt, d, Fe, h, 1, y);
                for (int i = 0; i < d; i++) acc[i] += (double)wts[j] * (double)y[i];
            }
            if (p >= 1 && matched) { /* the branch receives the gated primary shared-expert output */
                for (int i = 0; i < d; i++) acc[i] += (double)lw->gate_g[i] * (double)G1[(size_t)r * d + i];
            } else if (Fs > 0) { /* shared expert(s): every token, weight one */
                orc_linear(lw->sh_gate, dt, Fs, d, mr, 1, g);
                orc_linear(lw->sh_up, dt, Fs, d, mr, 1, u);
                orc_swiglu(g, u, Fs, h);
                if (p == 0) memcpy(Hs1 + (size_t)r * Fs, h, sizeof(float) * (size_t)Fs);
                if (p >= 1 && c->moe_b_coupling)
                    for (int i = 0; i < Fs; i++) h[i] += lw->coup_b[i] * Hs1[(size_t)r * Fs + i];
                orc_linear(lw->sh_down, dt, d, Fs, h, 1, y);
                if (p == 0) memcpy(G1 + (size_t)r * d, y, sizeof(float) * (size_t)d);
                for (int i = 0; i < d; i++) acc[i] += (double)y[i];
            }
            if (p >= 1 && !matched)
                for (int i = 0; i < d; i++) acc[i] += (double)lw->coup_c[i] * (double)M1[(size_t)r * d + i];
            for (int i = 0; i < d; i++) M[i] = (float)acc[i];
        }
    }
    free(logits); free(g); free(u); free(h); free(y); free(acc); free(Hs1); free(G1); free(idx1);
}

static void mlp_any(const orc_config *c, const orc_layer_weights *lw, const float *m, int paths, int n,
                    const int32_t *forced, int32_t *chosen, float *logits_out, int ld_logits, float *M) {
    if (c->n_experts > 0)
        mlp_moe(c, lw, m, paths, n, forced, chosen, logits_out, ld_logits, M);
    else
        mlp_dense(c, lw, m, paths, n, M);
}

/* ------------------------------------------------------------------------------------ */
/* model handle                                                                          */

static int config_ok(const orc_config *c) {
    if (c->d_model <= 0 || c->n_layers <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0) return 0;
    if (c->head_dim <= 0 || (c->head_dim & 1) || c->vocab <= 0) return 0;
    if (c->n_q_heads % c->n_kv_heads) return 0;
    if (c->weight_dtype != 0 && c->weight_dtype != 1) return 0;
    if (c->n_paths != 0 && (c->n_paths < 2 || c->n_paths > 16)) return 0;
    if (c->n_experts > 0) {
        if (c->d_expert <= 0 || c->k_primary <= 0 || c->k_branch <= 0) return 0;
        if (c->k_primary > c->n_experts || c->k_branch > c->n_experts) return 0;
        if (c->k_primary > 64 || c->k_branch > 64 || c->n_shared_experts < 0) return 0;
    } else if (c->d_ff <= 0 || c->compute_matched) {
        return 0;
    }
    return 1;
}

orc_model *orc_create(const orc_config *cfg, const orc_weights *w) {
    if (!cfg || !w || !config_ok(cfg) || cfg->max_batch <= 0 || cfg->max_seq <= 0) return NULL;
    orc_model *m = (orc_model *)calloc(1, sizeof *m);
    m->cfg = *cfg;
    m->w = *w;
    m->layers = (orc_layer_weights *)malloc(sizeof(orc_layer_weights) * (size_t)cfg->n_layers);
    memcpy(m->layers, w->layers, sizeof(orc_layer_weights) * (size_t)cfg->n_layers);
    m->w.layers = m->layers;
    size_t n = (size_t)cfg->n_layers * cfg->max_batch * cfg->max_seq * kv_dim_of(cfg);
    m->kc = (float *)calloc(n, sizeof(float));
    m->vc = (float *)calloc(n, sizeof(float));
    m->len = (int32_t *)calloc((size_t)cfg->max_batch, sizeof(int32_t));
    if (cfg->n_experts > 0)
        m->rlog = (float *)calloc((size_t)cfg->n_layers * paths_of(cfg) * cfg->max_batch * cfg->n_experts, sizeof(float));
    if (!m->kc || !m->vc || (cfg->n_experts > 0 && !m->rlog)) {
        orc_destroy(m);
        return NULL;
    }
    return m;
}

void orc_destroy(orc_model *m) {
    if (!m) return;
    free(m->layers); free(m->kc); free(m->vc); free(m->len); free(m->rlog); free(m);
}
void orc_reset(orc_model *m) { memset(m->len, 0, sizeof(int32_t) * (size_t)m->cfg.max_batch); }
int orc_seq_len(const orc_model *m, int b) { return m->len[b]; }
float *orc_k_cache(orc_model *m) { return m->kc; }
float *orc_v_cache(orc_model *m) { return m->vc; }
void orc_set_seq_len(orc_model *m, int b, int len) { m->len[b] = len; }
const float *orc_router_logits(const orc_model *m) { return m->rlog; }

static size_t cache_index(const orc_config *c, int l, int b, int t) {
    return (((size_t)l * c->max_batch + b) * c->max_seq + t) * kv_dim_of(c);
}

/* ------------------------------------------------------------------------------------ */
/* one incremental step (Section 4.4, items 2-3; primary-only is the standard decode)    */

static int step(orc_model *m, const int32_t *tokens, int B, int grouped, int want_logits,
                const int32_t *forced, int32_t *chosen, int32_t *next, float *z1, float *z2,
                float *alpha, float *mix) {
    const orc_config *c = &m->cfg;
    int d = c->d_model, dh = c->head_dim, nq = c->n_q_heads, nkv = c->n_kv_heads, V = c->vocab;
    int G = nq / nkv, dt = c->weight_dtype;
    size_t qd = q_dim_of(c), kvd = kv_dim_of(c);
    int K = paths_of(c);            /* residual paths: the primary and K-1 decode branches */
    int P = grouped ? K : 1;        /* paths evaluated in this step                        */
    int R = P * B;
    /* rows that evaluate attention: the compute-matched branch has none (Eq. matched_attention) */
    int Pa = (grouped && !c->compute_matched) ? K : 1, Ra = Pa * B;
    int kmax = c->k_primary > c->k_branch ? c->k_primary : c->k_branch;
    if (B <= 0 || B > c->max_batch) return -1;
    for (int b = 0; b < B; b++) {
        if (m->len[b] >= c->max_seq) return -1;
        if (tokens[b] < 0 || tokens[b] >= V) return -1;
    }

    float *S = (float *)malloc(sizeof(float) * (size_t)R * d);    /* residual states   */
    float *N = (float *)malloc(sizeof(float) * (size_t)R * d);    /* normalised states */
    float *Q = (float *)malloc(sizeof(float) * (size_t)R * qd);
    float *Kn = (float *)malloc(sizeof(float) * (size_t)B * kvd);
    float *Vn = (float *)malloc(sizeof(float) * (size_t)B * kvd);
    float *O = (float *)malloc(sizeof(float) * (size_t)R * qd);
    float *A = (float *)malloc(sizeof(float) * (size_t)R * d);
    float *M = (float *)malloc(sizeof(float) * (size_t)R * d);
    float *row = (float *)malloc(sizeof(float) * (size_t)d);

    /* Eq. embeddings: S_1^0 = RMSNorm(E_1[x]), S_j^0 = RMSNorm(E_j[x]); every decode branch has
     * its own table (Appendix C.1), stored one after another in embed_branch */
    for (int b = 0; b < B; b++) {
        fetch_row(m->w.embed_primary, dt, (size_t)tokens[b], d, row);
        orc_rmsnorm(row, m->w.embed_norm_g, d, c->rms_eps, S + (size_t)b * d);
        for (int j = 1; j < P; j++) {
            fetch_row(m->w.embed_branch, dt, (size_t)(j - 1) * V + (size_t)tokens[b], d, row);
            orc_rmsnorm(row, m->w.embed_norm_g, d, c->rms_eps, S + ((size_t)j * B + b) * d);
        }
    }

    for (int l = 0; l < c->n_layers; l++) {
        const orc_layer_weights *lw = &m->layers[l];
        /* N_i = RMSNorm(S_i) */
        for (int r = 0; r < R; r++)
            orc_rmsnorm(S + (size_t)r * d, lw->attn_norm_g, d, c->rms_eps, N + (size_t)r * d);
        /* Q_i = RoPE(N_i W_Q) for all paths; K_1 = RoPE(N_1 W_K), V_1 = N_1 W_V: primary only */
        orc_linear(lw->wq, dt, (int)qd, d, N, Ra, Q);
        orc_linear(lw->wk, dt, (int)kvd, d, N, B, Kn);
        orc_linear(lw->wv, dt, (int)kvd, d, N, B, Vn);
        for (int r = 0; r < Ra; r++) orc_rope(Q + (size_t)r * qd, nq, dh, m->len[r % B], c->rope_base);
        for (int b = 0; b < B; b++) orc_rope(Kn + (size_t)b * kvd, nkv, dh, m->len[b], c->rope_base);
        /* Q~_j = Q_j + a * Q_1 (the same a for every branch) */
        for (int j = 1; j < Pa; j++)
            for (int b = 0; b < B; b++)
                for (size_t i = 0; i < qd; i++)
                    Q[((size_t)j * B + b) * qd + i] += lw->coup_a[i] * Q[(size_t)b * qd + i];
        /* the primary path appends its key and value; the branches have none */
        for (int b = 0; b < B; b++) {
            float *kd = m->kc + cache_index(c, l, b, m->len[b]);
            float *vd = m->vc + cache_index(c, l, b, m->len[b]);
            for (size_t i = 0; i < kvd; i++) {
                kd[i] = c->kv_round_bf16 ? round_through_bf16(Kn[(size_t)b * kvd + i]) : Kn[(size_t)b * kvd + i];
                vd[i] = c->kv_round_bf16 ? round_through_bf16(Vn[(size_t)b * kvd + i]) : Vn[(size_t)b * kvd + i];
            }
        }
        /* every query attends to primary positions 0..t inclusive */
#pragma omp parallel for schedule(static)
        for (int rh = 0; rh < Ra * nq; rh++) {
            int r = rh / nq, h = rh % nq, b = r % B, g = h / G;
            orc_attend(Q + (size_t)r * qd + (size_t)h * dh, m->kc + cache_index(c, l, b, 0) + (size_t)g * dh,
                       m->vc + cache_index(c, l, b, 0) + (size_t)g * dh, m->len[b] + 1, (int)kvd, dh,
                       O + (size_t)r * qd + (size_t)h * dh);
        }
        /* S-bar_i = S_i + Attn_i W_O */
        orc_linear(lw->wo, dt, d, (int)qd, O, Ra, A);
        if (grouped && c->compute_matched) /* A_j = g_A * A_1 (Eq. matched_attention) */
            for (int j = 1; j < P; j++)
                for (int b = 0; b < B; b++)
                    for (int i = 0; i < d; i++)
                        A[((size_t)j * B + b) * d + i] = lw->gate_a[i] * A[(size_t)b * d + i];
        for (size_t i = 0; i < (size_t)R * d; i++) S[i] += A[i];
        /* MLP / MoE on RMSNorm(S-bar_i), then S_i^{l+1} = S-bar_i + M_i */
        for (int r = 0; r < R; r++)
            orc_rmsnorm(S + (size_t)r * d, lw->mlp_norm_g, d, c->rms_eps, N + (size_t)r * d);
        const int32_t *f = forced ? forced + (size_t)l * K * B * kmax : NULL;
        int32_t *ch = chosen ? chosen + (size_t)l * K * B * kmax : NULL;
        if (ch && !grouped)
            for (int i = 0; i < (K - 1) * B * kmax; i++) ch[(size_t)B * kmax + i] = -1;
        float *lg = m->rlog ? m->rlog + (size_t)l * K * c->max_batch * c->n_experts : NULL;
        mlp_any(c, lw, N, P, B, f, ch, lg, c->max_batch, M);
        for (size_t i = 0; i < (size_t)R * d; i++) S[i] += M[i];
    }
    for (int b = 0; b < B; b++) m->len[b] += 1;

    if (want_logits) {
        float *Z = (float *)malloc(sizeof(float) * (size_t)R * V);
        float *zb = (float *)malloc(sizeof(float) * (size_t)(P > 1 ? P - 1 : 1) * V);
        for (int r = 0; r < R; r++) {
            if (c->final_norm)
                orc_rmsnorm(S + (size_t)r * d, m->w.final_norm_g, d, c->rms_eps, N + (size_t)r * d);
            else
                memcpy(N + (size_t)r * d, S + (size_t)r * d, sizeof(float) * (size_t)d);
        }
        orc_linear(m->w.lm_head, dt, V, d, N, R, Z);
        for (int b = 0; b < B; b++) {
            const float *zb1 = Z + (size_t)b * V;
            if (z1) memcpy(z1 + (size_t)b * V, zb1, sizeof(float) * (size_t)V);
            if (grouped) {
                for (int j = 1; j < P; j++) { /* branch logits, branch-major: z2 [K-1][B][V] */
                    memcpy(zb + (size_t)(j - 1) * V, Z + ((size_t)j * B + b) * V, sizeof(float) * (size_t)V);
                    if (z2) memcpy(z2 + ((size_t)(j - 1) * B + b) * V, Z + ((size_t)j * B + b) * V, sizeof(float) * (size_t)V);
                }
                float al;
                int tok = orc_readout_multi(zb1, zb, P - 1, V, &al, mix ? mix + (size_t)b * V : NULL);
                if (alpha) alpha[b] = al;
                if (next) next[b] = tok;
            } else if (next) {
                next[b] = argmax_f32(zb1, V);
            }
        }
        free(Z); free(zb);
    }
    free(S); free(N); free(Q); free(Kn); free(Vn); free(O); free(A); free(M); free(row);
    return 0;
}

int orc_decode_step(orc_model *m, const int32_t *tokens, int B, int grouped,
                    const int32_t *forced_experts, int32_t *chosen_experts, int32_t *next,
                    float *z1, float *z2, float *alpha, float *mix) {
    if (!m || !tokens) return -1;
    return step(m, tokens, B, grouped, 1, forced_experts, chosen_experts, next, z1, z2, alpha, mix);
}

/* Section 4.4 item 1: the primary path alone walks the prompt and fills the cache. */
int orc_prefill(orc_model *m, const int32_t *tokens, int B, int n, float *last_logits) {
    if (!m || !tokens || B <= 0 || B > m->cfg.max_batch || n <= 0) return -1;
    int32_t *col = (int32_t *)malloc(sizeof(int32_t) * (size_t)B);
    int rc = 0;
    for (int t = 0; t < n && rc == 0; t++) {
        for (int b = 0; b < B; b++) col[b] = tokens[(size_t)b * n + t];
        int last = (t == n - 1);
        rc = step(m, col, B, 0, last && last_logits != NULL, NULL, NULL, NULL, last ? last_logits : NULL,
                  NULL, NULL, NULL);
    }
    free(col);
    return rc;
}

/* ------------------------------------------------------------------------------------ */
/* Non-incremental forward over whole sequences (the training-time graph of Section 4:   */
/* every path at every position, ordinary causal mask, the branches read K_1,V_1).       */
/* z2 is [K-1][B][T][V].                                                                 */

int orc_full_forward(const orc_config *c, const orc_weights *w, const int32_t *tokens, int B, int T,
                     float *z1, float *z2, float *k_out, float *v_out) {
    if (!c || !w || !tokens || !config_ok(c) || B <= 0 || T <= 0) return -1;
    int d = c->d_model, dh = c->head_dim, nq = c->n_q_heads, nkv = c->n_kv_heads, V = c->vocab;
    int G = nq / nkv, dt = c->weight_dtype;
    int K = paths_of(c), Pa = c->compute_matched ? 1 : K;
    size_t qd = q_dim_of(c), kvd = kv_dim_of(c);
    double scale = 1.0 / sqrt((double)dh);
    for (size_t i = 0; i < (size_t)B * T; i++)
        if (tokens[i] < 0 || tokens[i] >= V) return -1;

    /* path-major stacks of T rows each: S = [S_1; S_2; ...] */
    float *S = (float *)malloc(sizeof(float) * (size_t)K * T * d);
    float *N = (float *)malloc(sizeof(float) * (size_t)K * T * d);
    float *Q = (float *)malloc(sizeof(float) * (size_t)K * T * qd);
    float *K1 = (float *)malloc(sizeof(float) * (size_t)T * kvd), *V1 = (float *)malloc(sizeof(float) * (size_t)T * kvd);
    float *O = (float *)malloc(sizeof(float) * (size_t)K * T * qd);
    float *A = (float *)malloc(sizeof(float) * (size_t)K * T * d);
    float *M = (float *)malloc(sizeof(float) * (size_t)K * T * d);
    float *row = (float *)malloc(sizeof(float) * (size_t)d);

    for (int b = 0; b < B; b++) {
        const int32_t *x = tokens + (size_t)b * T;
        for (int t = 0; t < T; t++) {
            fetch_row(w->embed_primary, dt, (size_t)x[t], d, row);
            orc_rmsnorm(row, w->embed_norm_g, d, c->rms_eps, S + (size_t)t * d);
            for (int j = 1; j < K; j++) {
                fetch_row(w->embed_branch, dt, (size_t)(j - 1) * V + (size_t)x[t], d, row);
                orc_rmsnorm(row, w->embed_norm_g, d, c->rms_eps, S + ((size_t)j * T + t) * d);
            }
        }
        for (int l = 0; l < c->n_layers; l++) {
            const orc_layer_weights *lw = &w->layers[l];
            for (int r = 0; r < K * T; r++)
                orc_rmsnorm(S + (size_t)r * d, lw->attn_norm_g, d, c->rms_eps, N + (size_t)r * d);
            orc_linear(lw->wq, dt, (int)qd, d, N, Pa * T, Q);
            orc_linear(lw->wk, dt, (int)kvd, d, N, T, K1);
            orc_linear(lw->wv, dt, (int)kvd, d, N, T, V1);
            for (int t = 0; t < T; t++) {
                orc_rope(Q + (size_t)t * qd, nq, dh, t, c->rope_base);
                orc_rope(K1 + (size_t)t * kvd, nkv, dh, t, c->rope_base);
                for (int j = 1; j < Pa; j++) {
                    float *Qj = Q + ((size_t)j * T + t) * qd;
                    orc_rope(Qj, nq, dh, t, c->rope_base);
                    for (size_t i = 0; i < qd; i++) Qj[i] += lw->coup_a[i] * Q[(size_t)t * qd + i];
                }
            }
            if (k_out) memcpy(k_out + (((size_t)l * B + b) * T) * kvd, K1, sizeof(float) * (size_t)T * kvd);
            if (v_out) memcpy(v_out + (((size_t)l * B + b) * T) * kvd, V1, sizeof(float) * (size_t)T * kvd);
            /* softmax(Q K^T / sqrt(d_h) + M_causal) V, the T x T form with an explicit mask */
#pragma omp parallel for schedule(static)
            for (int ph = 0; ph < Pa * nq; ph++) {
                int p = ph / nq, h = ph % nq, g = h / G;
                const float *Qp = Q + (size_t)p * T * qd;
                float *Op = O + (size_t)p * T * qd;
                double *Pr = (double *)malloc(sizeof(double) * (size_t)T);
                for (int i = 0; i < T; i++) {
                    double mx = -INFINITY, den = 0.0;
                    for (int j = 0; j < T; j++) {
                        double acc = 0.0;
                        for (int e = 0; e < dh; e++)
                            acc += (double)Qp[(size_t)i * qd + (size_t)h * dh + e] *
                                   (double)K1[(size_t)j * kvd + (size_t)g * dh + e];
                        double mask = (j <= i) ? 0.0 : -INFINITY;
                        Pr[j] = acc * scale + mask;
                        if (Pr[j] > mx) mx = Pr[j];
                    }
                    for (int j = 0; j < T; j++) {
                        Pr[j] = exp(Pr[j] - mx);
                        den += Pr[j];
                    }
                    for (int e = 0; e < dh; e++) {
                        double acc = 0.0;
                        for (int j = 0; j < T; j++) acc += Pr[j] * (double)V1[(size_t)j * kvd + (size_t)g * dh + e];
                        Op[(size_t)i * qd + (size_t)h * dh + e] = (float)(acc / den);
                    }
                }
                free(Pr);
            }
            orc_linear(lw->wo, dt, d, (int)qd, O, Pa * T, A);
            if (c->compute_matched) /* A_j = g_A * A_1 (Eq. matched_attention) */
                for (int j = 1; j < K; j++)
                    for (int t = 0; t < T; t++)
                        for (int i = 0; i < d; i++)
                            A[((size_t)j * T + t) * d + i] = lw->gate_a[i] * A[(size_t)t * d + i];
            for (size_t i = 0; i < (size_t)K * T * d; i++) S[i] += A[i];
            for (int r = 0; r < K * T; r++)
                orc_rmsnorm(S + (size_t)r * d, lw->mlp_norm_g, d, c->rms_eps, N + (size_t)r * d);
            mlp_any(c, lw, N, K, T, NULL, NULL, NULL, 0, M);
            for (size_t i = 0; i < (size_t)K * T * d; i++) S[i] += M[i];
        }
        for (int r = 0; r < K * T; r++) {
            if (c->final_norm)
                orc_rmsnorm(S + (size_t)r * d, w->final_norm_g, d, c->rms_eps, N + (size_t)r * d);
            else
                memcpy(N + (size_t)r * d, S + (size_t)r * d, sizeof(float) * (size_t)d);
        }
        if (z1) orc_linear(w->lm_head, dt, V, d, N, T, z1 + (size_t)b * T * V);
        if (z2)
            for (int j = 1; j < K; j++)
                orc_linear(w->lm_head, dt, V, d, N + (size_t)j * T * d, T, z2 + (((size_t)(j - 1) * B + b) * T) * V);
    }
    free(S); free(N); free(Q); free(K1); free(V1); free(O); free(A); free(M); free(row);
    return 0;
}
