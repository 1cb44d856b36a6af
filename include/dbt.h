/*
 * dbt.h -- C ABI of the grouped decode step of the Decode-Branch Transformer on B200.
 *
 * What the library computes (paper Section 4).  Two residual trajectories share every
 * large matrix: the primary path S_1 is a standard causal Transformer and is the only
 * writer of the persistent KV cache; the decode branch S_2 starts from its own token
 * embedding (Eq. embeddings), forms only a query (Eq. asymattn: Q~_2 = Q_2 + a*Q_1, read
 * against the primary K_1,V_1), is coupled in the MLP by b and c (Eq. mlp) and writes no
 * persistent state.  Logits of both paths go through one output matrix and are mixed with
 * alpha = clip_[0.5,1](sum_v p_v^2) (Eq. alpha, Eq. mixloss).  Inference follows Section
 * 4.4: a primary-only prefill over the prompt, then grouped steps -- both paths' rows
 * stacked through the shared matrices and one read of the primary cache serving both
 * queries ("Decode" paragraph; Section 4.5, Eq. decode_traffic).
 *
 * Conventions.
 *  - Every pointer is marked HOST or DEVICE.  All device memory (weights, KV pool,
 *    workspace, token / logit buffers) belongs to the caller; the library borrows it,
 *    never frees it and never writes the weights.  It must outlive the handle.
 *  - Matrices are row-major [out_features, in_features] (the paper's H W with W stored
 *    transposed), in `weight_dtype`.  Norm gains and the coupling vectors a, b, c are fp32.
 *  - Stacked activations are path-major: rows 0..B-1 primary, then B rows per decode branch.
 *  - KV pool layout: [n_layers][2 (K,V)][num_pages][n_kv_heads][page_size][head_dim] in
 *    `weight_dtype`; K is stored after RoPE.  Logical position t of sequence b lives in
 *    physical page page_table[b][t / page_size], slot t % page_size.
 *  - Calls enqueue work on the CUDA stream given at creation and return without waiting
 *    (the *_host variants wait).  Errors the host can see (bad arguments, capacity) are
 *    returned at once and enqueue nothing.  Errors only the device can see (a token id out
 *    of range) are recorded in a status word read by dbt_sync_status; the offending value is
 *    clamped so that no access leaves its buffer.  Nothing traps or aborts.
 *  - Not thread-safe per handle.
 */
#ifndef DBT_H
#define DBT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dbt_model dbt_model; /* opaque; owned by the library */

typedef enum {
    DBT_OK = 0,
    DBT_ERR_INVALID_ARG = 1,
    DBT_ERR_UNSUPPORTED = 2, /* shape / option outside what the kernels cover        */
    DBT_ERR_CAPACITY = 3,    /* max_batch, max_seq or the page pool would be exceeded */
    DBT_ERR_STATE = 4,
    DBT_ERR_CUDA = 5,
    DBT_ERR_DEVICE = 6,      /* the device status word is non-zero (dbt_sync_status)  */
    DBT_ERR_TIMEOUT = 7      /* a bounded wait inside a kernel ran out (dbt_sync_status) */
} dbt_status;

enum { DBT_DTYPE_F32 = 0, DBT_DTYPE_BF16 = 1 };
enum { DBT_ROUTER_INDEPENDENT = 0, DBT_ROUTER_REPLAY = 1 };

typedef struct {
    uint32_t struct_size; /* sizeof(dbt_config), for versioning */
    int32_t d_model, n_layers, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    int32_t weight_dtype; /* DBT_DTYPE_*; the KV cache uses the same storage type */
    float rope_base;      /* RoPE base; half-split pairs (i, i+head_dim/2), 0-based positions,
                             the same position for both paths */
    float rms_eps;
    int32_t final_norm;       /* 1: RMSNorm before the shared output matrix */
    int32_t n_experts;        /* 0 = dense MLP (Eq. mlp); >0 = MoE (Eq. moe_layer) */
    int32_t d_expert;         /* hidden width of one routed expert */
    int32_t n_shared_experts; /* applied to every token of both paths, un-gated */
    int32_t k_primary;        /* k_1 of Eq. moe_budget */
    int32_t k_branch;         /* k_2 of Eq. moe_budget */
    int32_t router_mode;      /* DBT_ROUTER_* (replay: Section 4.3) */
    int32_t moe_b_coupling;   /* 1: b couples the shared expert's hidden state; 0: b unused in MoE */
    int32_t compute_matched;  /* 1: compute-matched MoE allocation (Appendix B.3): the branch evaluates no
                                 attention and no shared expert; A_2 = g_A*A_1 (Eq. matched_attention),
                                 M_2 = R_2(N_2;k_2) + g_G*G(N_1) (Eq. matched_shared_expert); a, b, c are
                                 not applied.  MoE models only (DBT_ERR_UNSUPPORTED otherwise). */
    int32_t n_paths;          /* K of Appendix C.1 ("More decode branches"): residual paths in all, the primary plus
                                 K-1 decode branches.  Each branch has its own embedding table and same-position
                                 state, reads the primary cache, shares a, b, c (and g_A, g_G) with the other
                                 branches, routes for itself in MoE layers; the readout mixes p with the mean of
                                 the branch distributions.  2 (or 0) is the main text's model; at most 8, and
                                 n_paths * n_q_heads / n_kv_heads <= 16 (DBT_ERR_UNSUPPORTED otherwise). */
    int32_t max_batch, max_seq;
    int32_t page_size; /* tokens per KV page; 16 */
    int32_t num_pages; /* pages in the pool, per layer and per K/V */
} dbt_config;

/* DEVICE pointers.  Unused entries (MoE fields of a dense model and vice versa) may be NULL. */
typedef struct {
    const float *attn_norm_g;                  /* [d]                                         */
    const void *wq, *wk, *wv, *wo;             /* [q_dim,d] [kv_dim,d] [kv_dim,d] [d,q_dim]   */
    const float *coup_a;                       /* [q_dim]                                     */
    const float *mlp_norm_g;                   /* [d]                                         */
    const void *w_gate, *w_up, *w_down;        /* dense: [F,d] [F,d] [d,F]                    */
    const float *coup_b;                       /* dense [F]; MoE [n_shared*d_expert]          */
    const float *coup_c;                       /* [d]                                         */
    const void *router;                        /* [E,d]                                       */
    const void *exp_gate, *exp_up, *exp_down;  /* [E,Fe,d] [E,Fe,d] [E,d,Fe]                  */
    const void *sh_gate, *sh_up, *sh_down;     /* [Fs,d] [Fs,d] [d,Fs], Fs = n_shared*Fe      */
    const float *gate_a, *gate_g;              /* [d] [d]  g_A, g_G (compute_matched only)    */
} dbt_layer_weights;

typedef struct {
    const void *embed_primary, *embed_branch;  /* DEVICE E_1 [V,d]; E_2..E_K one after another
                                                  [n_paths-1][V,d]                            */
    const float *embed_norm_g, *final_norm_g;  /* DEVICE [d]                                  */
    const void *lm_head;                       /* DEVICE shared output matrix [V,d]           */
    const dbt_layer_weights *layers;           /* HOST array [n_layers] of DEVICE pointers    */
} dbt_weights;

/* Bytes the caller must provide for the KV pool and the workspace (both DEVICE, 256-byte
 * aligned).  cfg HOST. */
dbt_status dbt_query_sizes(const dbt_config *cfg, size_t *kv_bytes, size_t *workspace_bytes);

/* Build a handle (Section 4: the model of both paths).  cfg, w HOST; kv_pool_dev,
 * workspace_dev DEVICE; cuda_stream a cudaStream_t (NULL = default stream).  Validates the
 * configuration (DBT_ERR_UNSUPPORTED for head_dim not in {64,128}, page_size != 16,
 * n_q_heads not a multiple of n_kv_heads, more than 16 queries per KV head over both
 * paths, k > n_experts, ...), builds the RoPE table and the default page table
 * (sequence b owns pages b*ceil(max_seq/page_size) ...), and zeroes all sequence lengths.
 * On failure *out is NULL. */
dbt_status dbt_create(const dbt_config *cfg, const dbt_weights *w, void *kv_pool_dev,
                      void *workspace_dev, void *cuda_stream, dbt_model **out);
void dbt_destroy(dbt_model *m);

/* HOST table [B][pages_per_seq] of physical page ids (distinct, < num_pages) for sequences
 * 0..B-1; pages_per_seq <= ceil(max_seq/page_size) bounds each sequence's capacity. */
dbt_status dbt_set_page_table(dbt_model *m, const int32_t *table_host, int32_t B, int32_t pages_per_seq);

/* Sequence lengths := 0 (the cache contents are left as they are). */
dbt_status dbt_reset(dbt_model *m);
/* Declare that sequences 0..B-1 already hold lens_host[b] cached positions (the caller
 * wrote the pool itself, e.g. a synthetic fill for timing).  lens_host HOST. */
dbt_status dbt_set_seq_lens(dbt_model *m, const int32_t *lens_host, int32_t B);
/* Current length of sequence b as the host tracks it (-1 on a bad argument). */
int32_t dbt_seq_len(const dbt_model *m, int32_t b);

/* Section 4.4 item 1, prompt-wide prefill: the primary path alone processes n positions of
 * sequences 0..B-1 (tokens_dev DEVICE int32 [B][n]) starting at their current lengths,
 * writes their K/V and advances the lengths.  No branch computation.
 * last_primary_logits_dev: DEVICE fp32 [B][V] for the last position, or NULL. */
dbt_status dbt_prefill(dbt_model *m, const int32_t *tokens_dev, int32_t B, int32_t n,
                       float *last_primary_logits_dev);

/* Section 4.4 items 1 and 2 in one call: the primary path alone processes the whole prompt x_1..x_S
 * (tokens_dev DEVICE int32 [B][S], sequences 0..B-1 from their current lengths), and the continuation boundary
 * -- one branch evaluation at the final prompt token, coupled to the primary's Q_1, H_1, M_1 of that position
 * and read against the completed cache -- predicts x_{S+1} from the mixture.  Outputs as dbt_decode_step.
 * How it runs: positions 1..S-1 as the prompt-wide prefill, position S as one grouped step.  The boundary
 * evaluation has to stream every shared matrix once for the branch row anyway; letting the primary row of
 * position S ride in that same pass produces the "retained intermediates" where they are consumed, costs no
 * extra memory traffic and needs no per-layer retention buffers.  The values are those of the paper's form
 * (prefill all S positions, then a branch-only evaluation).  Lengths advance by S. */
dbt_status dbt_prefill_boundary(dbt_model *m, const int32_t *tokens_dev, int32_t B, int32_t S, int32_t *next_tokens_dev,
                                float *logits_primary_dev, float *logits_branch_dev, float *alpha_dev);

/* Section 4.4 items 2-3, one grouped step ("Decode" paragraph): for each sequence b the token
 * tokens_dev[b] at position t_b = its length; the primary appends K_1,V_1[t_b]; both paths'
 * queries read positions 0..t_b of the primary cache; the shared matrices are applied to
 * the stacked rows; next_tokens_dev[b] = argmax of alpha*p + (1-alpha)*q (lowest index on
 * ties; with more than one decode branch q is the mean of the branch distributions, Appendix C.1).
 * Lengths advance by one.  All pointers DEVICE; outputs may be NULL: next_tokens_dev int32 [B] (may alias
 * tokens_dev), logits_primary_dev fp32 [B][V], logits_branch_dev fp32 [n_paths-1][B][V], alpha_dev fp32 [B].
 * To start from a prompt x_1..x_S: prefill x_1..x_{S-1}, then pass x_S to the first step
 * (the boundary step of Section 4.4 item 2). */
dbt_status dbt_decode_step(dbt_model *m, const int32_t *tokens_dev, int32_t B, int32_t *next_tokens_dev,
                           float *logits_primary_dev, float *logits_branch_dev, float *alpha_dev);

/* The comparison path: the same step with the branch rows absent (a standard decode step,
 * Background "decode").  Writes the same K/V bits as dbt_decode_step for the same inputs;
 * next token = argmax of the primary logits. */
dbt_status dbt_decode_step_primary_only(dbt_model *m, const int32_t *tokens_dev, int32_t B,
                                        int32_t *next_tokens_dev, float *logits_primary_dev);

/* End-to-end variants with HOST buffers: copy tokens_host [B] to the device, run the step,
 * copy next_tokens_host [B] (and alpha_host [B] when non-NULL) back, wait for the stream.
 * Buffers should be pinned for the copies to be asynchronous. */
dbt_status dbt_decode_step_host(dbt_model *m, const int32_t *tokens_host, int32_t B,
                                int32_t *next_tokens_host, float *alpha_host);
dbt_status dbt_decode_step_primary_only_host(dbt_model *m, const int32_t *tokens_host, int32_t B,
                                             int32_t *next_tokens_host);

/* MoE only: DEVICE int32 [n_layers][n_paths][max_batch][kmax] (kmax = max(k_primary,k_branch)),
 * the expert ids each row used in the last decode step (-1 padded); and the number of
 * distinct experts loaded per layer in the last step, HOST int32 [n_layers] (waits for the
 * stream).  Equation moe_layer leaves near-ties in the router to rounding, so tests read the
 * choice back instead of assuming it. */
dbt_status dbt_last_experts(dbt_model *m, const int32_t **experts_dev, int32_t *kmax);
dbt_status dbt_last_expert_union(dbt_model *m, int32_t *count_per_layer_host);

/* Wait for the stream and read the device status word.  *device_status: 0 = clean; 1 = a token
 * id was out of range, 2 = a page id was out of range (*detail = the offending value; the value was
 * clamped and the step ran on): returns DBT_ERR_DEVICE; 3 = a bounded wait inside a kernel (on a
 * shared-memory barrier that a TMA copy or a tensor-core commit completes) ran out after about two
 * seconds: *detail = the wait site (100 + warp: operand ring of the GEMM, 200 + warp: its accumulator,
 * 300..: the decode attention kernel's page ring, 400..: the prompt attention kernel's, 500..: the
 * persistent per-expert GEMM's rings and accumulators), the CTA skipped its stores, released its tensor memory and
 * returned, so the step's results are invalid but the context stays usable: returns DBT_ERR_TIMEOUT.
 * The first code recorded wins until dbt_reset clears the word.  HOST pointers, may be NULL. */
dbt_status dbt_sync_status(dbt_model *m, int32_t *device_status, int32_t *detail);

/* The persistent state of the method is the primary path's KV cache alone (Background, "KV cache";
 * Section 4.4 "Decode": the branch writes no persistent entries).  These two calls move it between the
 * paged pool and HOST buffers in logical order [n_layers][B][T][kv_dim] (elements of `weight_dtype`, K after
 * RoPE), for sequences seq_ids_host[0..B-1] (HOST; NULL = sequences 0..B-1) and positions 0..T-1, through the
 * page table; they wait for the stream.  Export needs T <= the current length of each sequence
 * (DBT_ERR_STATE otherwise).  Import overwrites those positions and sets the length of each listed
 * sequence to T (the other sequences keep theirs).  T beyond a sequence's capacity: DBT_ERR_CAPACITY.
 * Uses: handing a prefilled cache to another process or a checker, restoring a session, tests. */
dbt_status dbt_kv_export(dbt_model *m, const int32_t *seq_ids_host, int32_t B, int32_t T, void *k_host, void *v_host);
dbt_status dbt_kv_import(dbt_model *m, const int32_t *seq_ids_host, int32_t B, int32_t T, const void *k_host,
                         const void *v_host);

/* Operator-level entry: the grouped skinny GEMM alone (Section 4.4 "Decode": the stacked rows
 * of both paths go through one shared matrix, each weight tile fetched once).
 * Y[r][f] = sum_k W[f][k] X[r][k] with W_dev DEVICE bf16 [n_out][K], X_dev DEVICE bf16 [R][K]
 * (1 <= R <= 256, K a multiple of 8, both 16-byte aligned), Y_dev DEVICE fp32 [R][n_out].
 * scratch_dev: DEVICE fp32 workspace of scratch_floats elements for the split-K partials
 * (at least splits * roundup(R) * n_out with roundup to 16/32/64/128/256); status_dev DEVICE
 * int32[2] (zeroed by the caller; afterwards {3, wait site} when a bounded device wait ran out -- the
 * codes of dbt_sync_status -- else still zero).
 * force_split > 0 asks for that split-K factor (lowered to ceil(K/64) and to a factor whose ranges
 * are all non-empty), 0 lets the library choose; *split_used (HOST, nullable) receives the factor
 * used.  Runs on the tensor cores (TMA + tcgen05); enqueues on cuda_stream. */
dbt_status dbt_op_gemm_tc(const void *W_dev, const void *X_dev, int32_t n_out, int32_t K, int32_t R,
                          int32_t force_split, float *Y_dev, float *scratch_dev, size_t scratch_floats,
                          int32_t *status_dev, void *cuda_stream, int32_t *split_used);

/* The same GEMM for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this entry exists for the integration, not for the method.)  Some hosts of this
 * library run where cudaMalloc is off limits -- inside a region that is being captured into a
 * CUDA graph, in a process whose memory pool is owned and fully handed out by another runtime,
 * or under a policy that forbids allocation after start-up -- and so cannot provide the split-K
 * workspace that dbt_op_gemm_tc asks for.  Here that workspace is a fixed array inside the
 * library's device image: 2^21 floats (8 MiB), resident on every GPU that has loaded the
 * library until the process exits.  The call allocates nothing and frees nothing.
 *   - Arguments as dbt_op_gemm_tc without the scratch pair; inputs, Y_dev and status_dev are
 *     still the caller's.  Results are identical to dbt_op_gemm_tc for the same split factor.
 *   - Limit: roundup(R) * n_out * splits <= 2^21 (roundup to 16/32/64/128/256).  The library
 *     lowers its own split choice to fit; a request that cannot fit even unsplit, or a
 *     force_split that does not fit, returns DBT_ERR_CAPACITY with a message and enqueues
 *     nothing.
 *   - The first call on each device looks up the array's device address (no allocation, but a
 *     runtime query): make that first call outside any stream capture, with the target device
 *     current.
 *   - All calls on a device share the one array and leave their partial sums in it.  Nothing in
 *     it needs to start at zero -- every element that is read has been written by the same
 *     call -- but two calls whose kernels overlap on the GPU (different streams, or a second
 *     process thread) race on it: serialise them. */
dbt_status dbt_op_gemm_tc_static(const void *W_dev, const void *X_dev, int32_t n_out, int32_t K, int32_t R,
                                 int32_t force_split, float *Y_dev, int32_t *status_dev, void *cuda_stream,
                                 int32_t *split_used);

/* Per-kernel timing for the roofline report (paper Eq. roofline, Eq. decode_traffic: time
 * against the bytes that must move).  Between begin and end every kernel launch is bracketed
 * by CUDA events on the handle's stream; end waits for the stream and sums, per kernel family,
 * the launches, the device time and the algorithmic bytes (weights read once, visible K/V read
 * once; 0 for kernels that move neither).  entries_host HOST [max_entries]. */
typedef struct {
    char name[32];
    int64_t launches;
    double total_ms;
    double bytes;
} dbt_profile_entry;
dbt_status dbt_profile_begin(dbt_model *m);
dbt_status dbt_profile_end(dbt_model *m, dbt_profile_entry *entries_host, int32_t max_entries, int32_t *n_entries);

/* Kernels launched by this handle since creation (for benchmark bookkeeping). */
int64_t dbt_launch_count(const dbt_model *m);
/* Last host-side error message of this handle (or of the failed dbt_create when m is NULL). */
const char *dbt_last_error(const dbt_model *m);
/* Library version string. */
const char *dbt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DBT_H */
