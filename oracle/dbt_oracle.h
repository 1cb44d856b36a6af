/*
 * dbt_oracle.h -- CPU oracle for the Decode-Branch Transformer forward pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct restatement of
 * the paper's Section 4 (two-path layer stack, asymmetric shared-KV attention, coupled
 * MLP / MoE, mixture readout) and of the inference procedure of Section 4.4.  It shares
 * no code, table or constant with the CUDA library and must never be linked, imported or
 * called from the product path.  Only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg may use it.
 *
 * Precision: vectors are stored in fp32; every dot product, norm and softmax sum is
 * accumulated in double, so the result does not depend on loop scheduling.  Weights are
 * read in their storage type (fp32, or bf16 widened exactly to fp32).
 *
 * Parity with the authors' own implementation is unpinned: the paper prints no numeric
 * forward-pass example.  The functions here are pinned instead by the invariants and
 * closed forms the paper and the mathematics fix (see tests/test_oracle_*.py).  The one
 * convention nothing in the paper fixes -- where the b coupling acts inside an MoE layer
 * -- is flagged "parity unpinned" at orc_config.moe_b_coupling.
 */
#ifndef DBT_ORACLE_H
#define DBT_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int32_t d_model, n_layers, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    int32_t weight_dtype;      /* 0 = fp32, 1 = bf16 (uint16 payload)                       */
    int32_t kv_round_bf16;     /* 1: round stored K/V to bf16 (error attribution only)      */
    float   rope_base;         /* RoPE frequency base                                       */
    float   rms_eps;           /* epsilon inside every RMSNorm                              */
    int32_t final_norm;        /* 1: RMSNorm before the shared output matrix                */
    int32_t n_experts;         /* 0 = dense MLP (Eq. mlp); >0 = MoE layer (Eq. moe_layer)   */
    int32_t d_expert;          /* hidden width of one routed expert                         */
    int32_t n_shared_experts;  /* shared experts, applied to every token, un-gated          */
    int32_t k_primary;         /* k_1 of Eq. moe_budget                                     */
    int32_t k_branch;          /* k_2 of Eq. moe_budget                                     */
    int32_t router_mode;       /* 0 independent routing (Section 5), 1 router replay (4.3)  */
    int32_t moe_b_coupling;    /* 1: b couples the shared expert's hidden state; 0: none.
                                  The paper defines b for a single MLP only -- parity
                                  unpinned for MoE layers.                                  */
    int32_t compute_matched;   /* 1: compute-matched MoE allocation (Appendix B.3): the branch
                                  evaluates no attention and no shared expert of its own,
                                  A_2 = g_A * A_1 and M_2 = R_2(N_2;k_2) + g_G * G(N_1);
                                  the a/b/c couplings do not appear in those equations and
                                  are not applied.  MoE layers only.                       */
    int32_t n_paths;           /* K of Appendix C.1 ("More decode branches"): residual paths in
                                  all, the primary plus K-1 decode branches; each branch has
                                  its own embedding table and same-position state, reads the
                                  primary cache, shares a/b/c with the other branches, and the
                                  readout uses the mean of the branch distributions.  2 (or 0)
                                  is the main text's model.                                 */
    int32_t max_batch, max_seq;
} orc_config;

/* Matrices are [out_features, in_features], in-features contiguous, in weight_dtype.
 * Gains and coupling vectors are always fp32. */
typedef struct {
    const float *attn_norm_g;                 /* [d]                                 */
    const void  *wq, *wk, *wv, *wo;           /* [q_dim,d] [kv_dim,d] [kv_dim,d] [d,q_dim] */
    const float *coup_a;                      /* [q_dim]   a^l of Eq. asymattn       */
    const float *mlp_norm_g;                  /* [d]                                 */
    const void  *w_gate, *w_up, *w_down;      /* dense: [F,d] [F,d] [d,F]            */
    const float *coup_b;                      /* [F] dense / [n_shared*d_expert] MoE */
    const float *coup_c;                      /* [d]       c^l of Eq. mlp            */
    const void  *router;                      /* [E,d]                               */
    const void  *exp_gate, *exp_up, *exp_down;/* [E,Fe,d] [E,Fe,d] [E,d,Fe]          */
    const void  *sh_gate, *sh_up, *sh_down;   /* [Fs,d] [Fs,d] [d,Fs], Fs=n_shared*Fe*/
    const float *gate_a, *gate_g;             /* [d] [d]   g_A, g_G of Appendix B.3 (compute_matched) */
} orc_layer_weights;

typedef struct {
    const void  *embed_primary, *embed_branch;   /* E_1 [V,d]; E_2..E_K one after another:
                                                    [K-1][V,d]                        */
    const float *embed_norm_g, *final_norm_g;    /* [d]                              */
    const void  *lm_head;                        /* shared output matrix [V,d]       */
    const orc_layer_weights *layers;             /* [n_layers]                       */
} orc_weights;

typedef struct orc_model orc_model;

/* ---- model-level calls (Section 4.4: prefill, boundary, continuation) ---------------- */

/* Borrow the weight pointers (they must outlive the handle); allocate an fp32 KV cache
 * [L][max_batch][max_seq][kv_dim] for K and V.  Returns NULL on a bad config. */
orc_model *orc_create(const orc_config *cfg, const orc_weights *w);
void orc_destroy(orc_model *m);
void orc_reset(orc_model *m);                      /* all sequence lengths := 0 */
int  orc_seq_len(const orc_model *m, int b);
/* Direct access to the cache (tests inject / inspect it): [L][max_batch][max_seq][kv_dim]. */
float *orc_k_cache(orc_model *m);
float *orc_v_cache(orc_model *m);
void orc_set_seq_len(orc_model *m, int b, int len);
/* MoE models: the router logits r_i = N_i W_r the last step computed, [L][K][max_batch][E]
 * (rows of paths the step did not evaluate keep older contents); NULL for dense models.
 * Tests use them to check that an expert set chosen elsewhere is a valid top-k. */
const float *orc_router_logits(const orc_model *m);

/* Primary-only pass over n prompt positions of sequences 0..B-1 (tokens [B][n]),
 * position by position; appends K/V; logits of the last position to last_logits [B][V]
 * when non-NULL.  Returns 0, or -1 on capacity / argument errors. */
int orc_prefill(orc_model *m, const int32_t *tokens, int B, int n, float *last_logits);

/* One step at position t_b = seq_len[b] for every sequence, token tokens[b].
 * grouped != 0: all K paths; z2 ([K-1][B][V], branch-major), alpha, mix are written; next =
 * argmax of the mixture.  grouped == 0: the primary path alone; next = argmax z1.
 * forced_experts (nullable, MoE): [L][K][B][kmax] expert ids to use instead of top-k
 * selection (weights are still computed from this run's router probabilities), where
 * kmax = max(k_primary,k_branch); chosen_experts (nullable) receives the ids used,
 * same layout, -1 padded.  Any output pointer may be NULL. */
int orc_decode_step(orc_model *m, const int32_t *tokens, int B, int grouped,
                    const int32_t *forced_experts, int32_t *chosen_experts,
                    int32_t *next, float *z1, float *z2, float *alpha, float *mix);

/* Non-incremental definition: every path at every position of tokens [B][T] with an
 * explicit causal mask (the training-time forward).  Touches no cache.  Outputs
 * z1 [B][T][V], z2 [K-1][B][T][V] (nullable), k_out,v_out [L][B][T][kv_dim] (nullable). */
int orc_full_forward(const orc_config *cfg, const orc_weights *w, const int32_t *tokens,
                     int B, int T, float *z1, float *z2, float *k_out, float *v_out);

/* ---- unit operations (the same routines the calls above are built from) --------------- */

void orc_rmsnorm(const float *x, const float *g, int n, float eps, float *y);
/* Y[r][i] = sum_k W[i][k] X[r][k]; W [n_out][n_in] in dtype dt. */
void orc_linear(const void *W, int dt, int n_out, int n_in, const float *X, int R, float *Y);
/* Rotate n_heads heads of width head_dim in place, position t, half-split pairs. */
void orc_rope(float *x, int n_heads, int head_dim, int t, float base);
/* One query head u[head_dim] against n_keys keys/values with row stride `stride`. */
void orc_attend(const float *u, const float *K, const float *V, int n_keys, int stride,
                int head_dim, float *o);
/* SwiGLU: h[i] = silu(g[i]) * u[i]. */
void orc_swiglu(const float *g, const float *u, int n, float *h);
/* Router: softmax over E logits, top-k (ties: lower index), renormalised weights.
 * forced (nullable): ids to use instead of the top-k choice. */
void orc_route(const float *logits, int E, int k, const int32_t *forced, int32_t *idx, float *wts);
/* Readout of Eq. alpha / mixloss: p,q softmax; alpha; mix (nullable, [V]); returns argmax mix. */
int orc_readout(const float *z1, const float *z2, int V, float *alpha, float *mix);
/* The same with nb decode branches (Appendix C.1): zb [nb][V], q replaced by the mean of the
 * branch distributions. */
int orc_readout_multi(const float *z1, const float *zb, int nb, int V, float *alpha, float *mix);

void orc_set_threads(int n);
int  orc_get_threads(void);

#ifdef __cplusplus
}
#endif
#endif /* DBT_ORACLE_H */
