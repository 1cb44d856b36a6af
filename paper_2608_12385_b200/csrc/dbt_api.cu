// Host side of the C ABI declared in include/dbt.h: argument checks, workspace carving,
// the per-step launch plan.  Every step of the path runs in this library's kernels.
#include "../../include/dbt.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "dbt_attn_mma.cuh"
#include "dbt_attn_prompt.cuh"
#include "dbt_fused.cuh"
#include "dbt_gemm_tc.cuh"
#include "dbt_gemm_persist.cuh"
#include "dbt_kernels.cuh"

using namespace dbt;

namespace {

thread_local std::string g_create_error;

struct Workspace {
    // fp32 activations, rows = Rmax unless noted
    float *S, *X, *Q, *Kn, *Vn, *O, *G1, *M, *Z, *part, *Zrows;
    float2 *rope;
    int32_t *seq_len, *page_table, *status, *tokens_stage, *next_stage, *att_tickets, *att_tickets2, *gemm_tickets;
    float *alpha_stage;
    char *kv_stage;  // staging for dbt_kv_export / dbt_kv_import (kKvStageBytes)
    int32_t *att_plan;  // a decode step's attention work split (attn_plan_kernel), kAttPlanInts
    // MoE
    float *rlogits, *rwts, *Hexp, *Yexp, *Msh, *Hsh;
    int32_t *ridx, *ecnt, *elist, *last_experts, *union_cnt;
    // bf16 tensor-core path: bf16 GEMM inputs and the fp32 split-K partial buffer
    __nv_bfloat16 *Xb, *Ob, *Hb;
    float *P, *ss;
    // MoE on tensor cores: activation rows sorted by expert
    __nv_bfloat16 *Xs, *Hs;
    float *Pe;
    float *ro_stats;      // readout: per (sequence, vocabulary chunk) softmax records and argmax candidates
    int32_t *ro_tickets;  // readout: arrival counters per sequence
    float *P2;       // split-K partials of the shared expert's GEMMs when they run beside the routed chain
    size_t P2_floats;
    int32_t *epos, *eoff;
    float *rs_sorted;  // 1/rms of each sorted row's source row (norm applied after the per-expert gate|up GEMM)
    size_t P_floats;
};

constexpr size_t kKvStageBytes = (size_t)8 << 20;

struct LayerMaps {
    CUtensorMap wq, wk, wv, wo, wg, wu, wd;  // dense MLP; for MoE wg/wu/wd hold the shared expert
    CUtensorMap eg, eu, ed;                  // all routed experts as [E*Fe, d], [E*Fe, d], [E*d, Fe]
    CUtensorMap rt;                          // router [E, d]
};

}  // namespace

struct dbt_model {
    dbt_config cfg;
    dbt_weights w;
    std::vector<dbt_layer_weights> layers;
    cudaStream_t stream;
    char *kv_pool;
    char *ws_base;
    size_t ws_bytes;
    Workspace ws;
    int Rmax, pages_per_seq_max, pages_per_seq, part_items;
    std::vector<int32_t> len_host;
    int64_t launches;
    std::string err;
    bool pending_union;
    // optional per-launch timing (dbt_profile_begin / dbt_profile_end)
    bool prof_on;
    struct ProfRec { const char *tag; double bytes; cudaEvent_t e0, e1; };
    std::vector<ProfRec> prof;
    std::vector<cudaEvent_t> prof_pool;
    // tensor-core path (bf16 models): TMA descriptors of every weight matrix and GEMM input
    bool tc;
    std::vector<LayerMaps> maps;
    CUtensorMap map_lm, map_Xb, map_Ob, map_Hb, map_kv, map_Xs, map_Hs;
    bool moe_tc;  // MoE experts on the tensor cores
    bool att_fast;  // TMA + mma.sync attention over the bf16 pool
    bool wide;      // dense bf16: RMSNorm factor applied after the GEMM, no row-wide reduction kernel
    // two-plane GEMM inputs: base pointer of each 2-D input map, and the 3-D one-box-per-stage views
    // built from it on first use (key: 2-D map, row-tile width, plane rows)
    struct ActBase { const void *base; };
    std::map<const CUtensorMap *, ActBase> act_base;
    std::map<std::tuple<const CUtensorMap *, int, int>, CUtensorMap> act3d;
    bool evict_first;  // weight tiles and K/V pages carry the evict-first L2 hint (DBT_EVICT_FIRST=0 turns it off)
    int moe_persist;       // per-expert GEMMs as persistent CTAs over the units that have work: -1 by the batch, DBT_MOE_PERSIST=0/1 off/on
    int cur_rows;          // primary rows (sequences x positions) of the launch plan being built
    bool moe_fuse_swiglu;  // the persistent per-expert gate|up launch applies the SwiGLU itself (DBT_MOE_FUSE_SWIGLU=0: a kernel of its own)
    bool prompt_fuse_swiglu;  // prompt chunks: SwiGLU in the gate|up GEMM's epilogue (DBT_PROMPT_FUSE_SWIGLU=0: a kernel of its own)
    bool prompt_attn_off;  // DBT_PROMPT_ATTN=tile: prompt chunks through the 16-row kernel's packed tiles (the earlier form)
    bool fuse_qkv;     // decode steps: the attention kernel does the Q|K|V epilogue itself (DBT_FUSE_QKV=0 keeps the kernel)
    int num_sms;
    int act_parts;  // 2: GEMM inputs carried as hi + lo bf16 terms (the operator-level GEMM entry uses 1: plain bf16)
    // a decode step is captured once per (batch, mode, buffer set) and replayed as a CUDA graph
    struct GraphEntry {
        int B, grouped;
        const void *ptr[5];
        cudaGraph_t graph;
        cudaGraphExec_t exec;
        int64_t launches;
    };
    bool use_graph, use_pdl;
    std::string pdl_off;
    cudaStream_t cap_stream;
    // MoE: the shared expert's three kernels run on a second stream beside the router / routed-expert
    // chain of the same layer (DBT_MOE_OVERLAP=0 keeps one stream)
    cudaStream_t side_stream;
    cudaEvent_t ev_fork, ev_join;
    bool moe_overlap;
    bool readout_row;  // DBT_READOUT=row: the one-CTA-per-row readout kernel
    int moe_row_tile;  // DBT_MOE_ROWTILE: row tile of the per-expert GEMMs (-1: chosen from the batch, 0: one tile of all rows)
    bool moe_wide;  // MoE chain with the RMSNorm factor applied behind the GEMMs (tensor-core MoE path)
    std::vector<GraphEntry> graphs;
    // where a decode step finds sequence b's token: tokens[b * tok_stride + tok_p0] (1, 0 except inside dbt_prefill_boundary)
    int tok_stride = 1, tok_p0 = 0;
    bool att_planned = false;  // inside a decode step whose attention work split has been computed (run_attention_plan)
};

namespace {

size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct Carver {
    char *base;
    size_t off;
    template <typename T>
    T *take(size_t n) {
        off = align_up(off);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

int elem_bytes(const dbt_config &c) { return c.weight_dtype == DBT_DTYPE_F32 ? 4 : 2; }
// Residual paths of the model: the primary and K-1 decode branches (Appendix C.1; 2 in the main text).
int paths_of(const dbt_config &c) { return c.n_paths >= 2 ? c.n_paths : 2; }
// The `grouped` argument of the step functions: 0 = the primary path alone, K >= 2 = all K paths stacked.
int npaths(int grouped) { return grouped > 1 ? grouped : 1; }
// Kernels that pair a primary row with one branch row run a block per branch in grid.z.
unsigned branch_blocks(int grouped) { return grouped > 1 ? (unsigned)(grouped - 1) : 1u; }
int kmax_of(const dbt_config &c) { return c.k_primary > c.k_branch ? c.k_primary : c.k_branch; }
// Rows of the activation buffers: all paths of a full batch in a decode step, or one prompt chunk of the
// prefill (2048 rows for dense bf16 models, whose GEMMs sweep several row tiles per weight tile and whose
// causal attention packs consecutive positions into a query tile; 256 otherwise).
int prefill_rows(const dbt_config &c) {
    // rows of a prompt chunk: bf16 models 2048, everything else 256
    int chunk = c.weight_dtype != DBT_DTYPE_BF16 ? 256 : 2048;
    return paths_of(c) * c.max_batch > chunk ? paths_of(c) * c.max_batch : chunk;
}

const char *check_config(const dbt_config *c, dbt_status *st) {
    *st = DBT_ERR_INVALID_ARG;
    if (!c) return "config is NULL";
    if (c->struct_size != sizeof(dbt_config)) return "dbt_config.struct_size does not match this library";
    if (c->d_model <= 0 || c->n_layers <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->vocab <= 0)
        return "non-positive model dimension";
    if (c->max_batch <= 0 || c->max_seq <= 0 || c->num_pages <= 0) return "non-positive capacity";
    if (c->weight_dtype != DBT_DTYPE_F32 && c->weight_dtype != DBT_DTYPE_BF16) return "unknown weight_dtype";
    *st = DBT_ERR_UNSUPPORTED;
    if (c->head_dim != 64 && c->head_dim != 128) return "head_dim must be 64 or 128";
    if (c->page_size != 16) return "page_size must be 16";
    if (c->n_q_heads % c->n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
    if (c->n_paths != 0 && (c->n_paths < 2 || c->n_paths > 8)) return "n_paths must be 2..8 (0 = 2)";
    if (paths_of(*c) * (c->n_q_heads / c->n_kv_heads) > 16) return "more than 16 queries per KV head over all paths";
    if (c->d_model % 8) return "d_model must be a multiple of 8";
    if (c->router_mode != DBT_ROUTER_INDEPENDENT && c->router_mode != DBT_ROUTER_REPLAY) return "unknown router_mode";
    if (c->compute_matched && c->n_experts <= 0) return "compute_matched is defined for MoE models only";
    if (c->n_experts > 0) {
        if (c->d_expert <= 0 || c->d_expert % 8) return "d_expert must be a positive multiple of 8";
        if (c->k_primary <= 0 || c->k_branch <= 0) return "k_primary and k_branch must be positive";
        if (c->k_primary > c->n_experts || c->k_branch > c->n_experts) return "top-k exceeds n_experts";
        if (kmax_of(*c) > 64 || c->n_experts > 1024) return "at most 64 experts per token and 1024 experts";
        if (c->n_shared_experts < 0) return "negative n_shared_experts";
    } else {
        if (c->d_ff <= 0 || c->d_ff % 8) return "d_ff must be a positive multiple of 8";
    }
    *st = DBT_OK;
    return nullptr;
}

// Rows whose attention may be split into segments: a decode step's, or an unpacked prompt chunk's (<= 256).
int att_rows_of(const dbt_config &c) { return paths_of(c) * c.max_batch > 256 ? paths_of(c) * c.max_batch : 256; }

// One pass over the workspace layout; with base == nullptr it only measures.
size_t carve(const dbt_config &c, char *base, Workspace *ws, int *Rmax_out, int *part_items_out) {
    Carver k{base, 0};
    Workspace w{};
    int Rmax = prefill_rows(c);
    int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
    bool moe = c.n_experts > 0;
    int Fs = moe ? c.n_shared_experts * c.d_expert : 0;
    int F = moe ? (Fs > 0 ? Fs : 8) : c.d_ff;
    int pps = (c.max_seq + c.page_size - 1) / c.page_size;
    int att_rows = att_rows_of(c);
    int part_items = att_rows * c.n_kv_heads + 8 * 148;  // attention partial slots: up to three rounds of 2 x 148 segments plus one per pair
    w.S = k.take<float>((size_t)Rmax * d);
    w.X = k.take<float>((size_t)Rmax * d);
    w.Q = k.take<float>((size_t)Rmax * qd);
    w.Kn = k.take<float>((size_t)Rmax * kvd);
    w.Vn = k.take<float>((size_t)Rmax * kvd);
    w.O = k.take<float>((size_t)Rmax * qd);
    w.G1 = k.take<float>((size_t)Rmax * F);
    w.M = k.take<float>((size_t)Rmax * d);
    w.Z = k.take<float>((size_t)paths_of(c) * c.max_batch * c.vocab);
    w.Zrows = k.take<float>((size_t)paths_of(c) * c.max_batch * d);
    w.part = k.take<float>((size_t)part_items * 16 * (c.head_dim + 2));
    w.rope = k.take<float2>((size_t)c.max_seq * (c.head_dim / 2));
    w.seq_len = k.take<int32_t>(c.max_batch);
    w.page_table = k.take<int32_t>((size_t)c.max_batch * pps);
    w.status = k.take<int32_t>(4);
    w.att_tickets = k.take<int32_t>((size_t)att_rows * c.n_kv_heads);
    w.att_tickets2 = k.take<int32_t>((size_t)att_rows * c.n_kv_heads * kAttMaxGroups);
    w.ro_stats = k.take<float>((size_t)c.max_batch * kRoMaxChunks * kRoRec);
    w.ro_tickets = k.take<int32_t>(c.max_batch);
    w.gemm_tickets = k.take<int32_t>(4096);
    w.tokens_stage = k.take<int32_t>(c.max_batch);
    w.next_stage = k.take<int32_t>(c.max_batch);
    w.alpha_stage = k.take<float>(c.max_batch);
    w.kv_stage = k.take<char>(kKvStageBytes);
    w.att_plan = k.take<int32_t>(kAttPlanInts);
    if (moe) {
        int km = kmax_of(c);
        w.rlogits = k.take<float>((size_t)Rmax * c.n_experts);
        w.rwts = k.take<float>((size_t)Rmax * km);
        w.ridx = k.take<int32_t>((size_t)Rmax * km);
        w.Hexp = k.take<float>((size_t)Rmax * km * c.d_expert);
        w.Yexp = k.take<float>((size_t)Rmax * km * d);
        w.Msh = k.take<float>((size_t)Rmax * d);
        w.Hsh = k.take<float>((size_t)Rmax * (Fs > 0 ? Fs : 8));
        w.ecnt = k.take<int32_t>(c.n_experts);
        w.elist = k.take<int32_t>((size_t)c.n_experts * Rmax);
        w.last_experts = k.take<int32_t>((size_t)c.n_layers * paths_of(c) * c.max_batch * km);
        w.union_cnt = k.take<int32_t>(c.n_layers);
    }
    if (c.weight_dtype == DBT_DTYPE_BF16) {
        // two planes each: rows [0,Rmax) hold hi = bf16(x), rows [Rmax,2Rmax) hold lo = bf16(x - hi)
        w.Xb = k.take<__nv_bfloat16>((size_t)2 * Rmax * d);
        w.Ob = k.take<__nv_bfloat16>((size_t)2 * Rmax * qd);
        w.Hb = k.take<__nv_bfloat16>((size_t)2 * Rmax * F);
        // room for the widest GEMM output at a few splits, capped
        size_t widest = (size_t)(moe ? (qd + 2 * kvd > 2 * F ? qd + 2 * kvd : 2 * F) : (2 * F > qd + 2 * kvd ? 2 * F : qd + 2 * kvd));
        size_t want = (size_t)Rmax * widest * 6;
        size_t cap = (size_t)24 << 20;  // floats (96 MB)
        w.P_floats = want < cap ? want : cap;
        if (w.P_floats < (size_t)Rmax * widest) w.P_floats = (size_t)Rmax * widest;
        w.P = k.take<float>(w.P_floats);
        w.ss = k.take<float>((size_t)((d + 127) / 128) * Rmax);
        if (moe) {
            size_t Rk = (size_t)Rmax * kmax_of(c);
            w.Xs = k.take<__nv_bfloat16>(2 * Rk * d);
            w.Hs = k.take<__nv_bfloat16>(2 * Rk * c.d_expert);
            w.Pe = k.take<float>(Rk * 2 * c.d_expert);
            size_t wide2 = (size_t)(2 * Fs > d ? 2 * Fs : d);
            w.P2_floats = Fs > 0 ? (size_t)Rmax * wide2 * 6 : 0;
            if (w.P2_floats > ((size_t)8 << 20)) w.P2_floats = (size_t)8 << 20;
            if (Fs > 0 && w.P2_floats < (size_t)Rmax * wide2) w.P2_floats = (size_t)Rmax * wide2;
            w.P2 = k.take<float>(w.P2_floats);
            w.epos = k.take<int32_t>(Rk);
            w.eoff = k.take<int32_t>(c.n_experts + 1);
            w.rs_sorted = k.take<float>(Rk);
        }
    }
    if (ws) *ws = w;
    if (Rmax_out) *Rmax_out = Rmax;
    if (part_items_out) *part_items_out = part_items;
    return align_up(k.off);
}

dbt_status fail(dbt_model *m, dbt_status st, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (m)
        m->err = buf;
    else
        g_create_error = buf;
    return st;
}

#define CUDA_TRY(m, call)                                                                            \
    do {                                                                                             \
        cudaError_t e_ = (call);                                                                     \
        if (e_ != cudaSuccess) return fail(m, DBT_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

// Every kernel goes through cudaLaunchKernelEx; with `pdl` the launch carries the programmatic
// stream-serialization attribute, so the kernel may start while its predecessor drains.  Each
// kernel calls griddepcontrol.wait before it touches anything its predecessor produced.
template <typename... Params, typename... Args>
cudaError_t launch_kernel(cudaStream_t stream, bool pdl, dim3 grid, dim3 block, size_t smem,
                          void (*kernel)(Params...), Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    int n = 0;
    if (pdl) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        n++;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, Params(std::forward<Args>(args))...);
}

// Debug aid: DBT_PDL_OFF=tag1,tag2 launches those kernel families fully serialized.
bool pdl_disabled_for(const dbt_model *m, const char *tag) {
    if (m->pdl_off.empty()) return false;
    size_t n = strlen(tag), pos = 0;
    while ((pos = m->pdl_off.find(tag, pos)) != std::string::npos) {
        bool left = pos == 0 || m->pdl_off[pos - 1] == ',';
        bool right = pos + n == m->pdl_off.size() || m->pdl_off[pos + n] == ',';
        if (left && right) return true;
        pos += n;
    }
    return false;
}

cudaEvent_t prof_event(dbt_model *m) {
    cudaEvent_t e = nullptr;
    if (!m->prof_pool.empty()) {
        e = m->prof_pool.back();
        m->prof_pool.pop_back();
    } else {
        cudaEventCreate(&e);
    }
    return e;
}

// tag: kernel family name for the profile; bytes: the algorithmic bytes this launch must move.
#define LAUNCH(m, tag, bytes, kernel, grid, block, smem, ...)                                            \
    do {                                                                                                 \
        cudaEvent_t p0_ = nullptr, p1_ = nullptr;                                                        \
        if ((m)->prof_on) {                                                                              \
            p0_ = prof_event(m);                                                                         \
            p1_ = prof_event(m);                                                                         \
            cudaEventRecord(p0_, (m)->stream);                                                           \
        }                                                                                                \
        cudaError_t e_ = launch_kernel((m)->stream, (m)->use_pdl && !pdl_disabled_for(m, tag), dim3(grid),       \
                                       dim3(block), smem, kernel, __VA_ARGS__);                          \
        (m)->launches++;                                                                                 \
        if ((m)->prof_on) {                                                                              \
            cudaEventRecord(p1_, (m)->stream);                                                           \
            (m)->prof.push_back(dbt_model::ProfRec{tag, (double)(bytes), p0_, p1_});                     \
        }                                                                                                \
        if (e_ != cudaSuccess) return fail(m, DBT_ERR_CUDA, "launch %s: %s", #kernel, cudaGetErrorString(e_)); \
    } while (0)

// Kernels templated on "more than one decode branch" (see resid_wide_kernel).
#define LAUNCH_BR(m, grouped, tag, bytes, kernel, grid, block, smem, ...)                \
    do {                                                                                 \
        if ((grouped) > 2)                                                               \
            LAUNCH(m, tag, bytes, kernel<true>, grid, block, smem, __VA_ARGS__);         \
        else                                                                             \
            LAUNCH(m, tag, bytes, kernel<false>, grid, block, smem, __VA_ARGS__);        \
    } while (0)

// ---- launch helpers -------------------------------------------------------------------

// Mixture readout (Eq. alpha, Eq. mixloss) and greedy token; also advances the sequence lengths.
// Rows cut into chunks of at most 2048 logits, one CTA per (sequence, chunk): two short launches
// instead of one CTA walking a row three times (DBT_READOUT=row keeps that kernel).
dbt_status run_readout(dbt_model *m, int B, int grouped, int32_t *next_dev, float *alpha_dev) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int nc = (c.vocab + kRoChunk - 1) / kRoChunk;
    if (m->readout_row || nc > kRoMaxChunks) {
        LAUNCH(m, "readout", 0, readout_kernel, B, 1024, 0, w.Z, B, c.vocab, grouped, next_dev, alpha_dev, w.seq_len, 1);
        return DBT_OK;
    }
    int chunk = (c.vocab + nc - 1) / nc;
    if (grouped) LAUNCH(m, "readout_stats", 0, readout_stats_kernel, dim3(B, nc), kRoThreads, 0, w.Z, B, c.vocab, grouped, chunk, w.ro_stats);
    LAUNCH(m, "readout", 0, readout_pick_kernel, dim3(B, nc), kRoThreads, 0, w.Z, B, c.vocab, chunk, grouped, w.ro_stats, w.ro_tickets,
           next_dev, alpha_dev, w.seq_len, 1);
    return DBT_OK;
}

template <typename WT>
dbt_status run_linear(dbt_model *m, const char *tag, const LinArgs &a) {
    int total = 0;
    double bytes = 0;
    for (int s = 0; s < a.nseg; s++) bytes += (double)a.n_out[a.epi == EPI_SWIGLU ? 0 : s] * a.K * sizeof(WT);
    if (a.epi == EPI_SWIGLU)
        total = a.n_out[0];
    else
        for (int s = 0; s < a.nseg; s++) total += a.n_out[s];
    int grid = (total + kLinWarps - 1) / kLinWarps;
    LAUNCH(m, tag, bytes, linear_kernel<WT>, grid, kLinWarps * 32, 0, a);
    return DBT_OK;
}

LinArgs lin1(const void *W, float *Y, int n_out, int rows, const float *X, int K, int epi = EPI_STORE) {
    LinArgs a{};
    a.W[0] = W;
    a.Y[0] = Y;
    a.n_out[0] = n_out;
    a.rows[0] = rows;
    a.nseg = 1;
    a.X = X;
    a.K = K;
    a.epi = epi;
    return a;
}

template <typename KT, int DH>
dbt_status run_attention(dbt_model *m, const RowMap &rm, int grouped, const KT *kpool, const KT *vpool, int nsplit,
                         double kv_bytes, bool out_bf16 = false) {
    const dbt_config &c = m->cfg;
    int G = c.n_q_heads / c.n_kv_heads, nq = npaths(grouped) * G;
    dim3 grid(rm.B * rm.cn, c.n_kv_heads, nsplit);
    int NQ = nq <= 1 ? 1 : nq <= 2 ? 2 : nq <= 4 ? 4 : nq <= 8 ? 8 : 16;
    const Workspace &w = m->ws;
#define ATTN_CASE(N)                                                                                          \
    case N:                                                                                                   \
        LAUNCH(m, "attention", kv_bytes, (attn_partial_kernel<KT, N, DH>), grid, 128, 0, w.Q, rm, grouped, G, c.n_kv_heads, kpool,   \
               vpool, w.page_table, m->pages_per_seq_max, c.num_pages, w.seq_len, nsplit, w.part, w.status);  \
        break;
    switch (NQ) {
        ATTN_CASE(1)
        ATTN_CASE(2)
        ATTN_CASE(4)
        ATTN_CASE(8)
        ATTN_CASE(16)
    }
#undef ATTN_CASE
    dim3 mgrid(rm.B * rm.cn, c.n_kv_heads);
    LAUNCH(m, "attn_merge", 0, attn_merge_kernel, mgrid, DH, 0, w.part, nsplit, NQ, DH, rm.B * rm.cn, grouped, G, c.n_kv_heads,
           out_bf16 ? (float *)nullptr : w.O, out_bf16 ? w.Ob : (__nv_bfloat16 *)nullptr,
           (out_bf16 && m->act_parts == 2) ? (size_t)m->Rmax * c.n_q_heads * c.head_dim : (size_t)0);
    return DBT_OK;
}

// MoE sub-layer (Eq. moe_layer, Eq. moe_budget, Section 4.3) on the normalised rows in X:
// router, per-expert row lists, routed experts (each selected expert's matrices streamed once
// for all its rows of both paths), shared expert with the b coupling, weighted combine with
// the c coupling and the residual add into S.
template <typename WT>
dbt_status run_moe(dbt_model *m, int l, const RowMap &rm, int grouped, bool record_experts) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    const dbt_layer_weights &lw = m->layers[l];
    int Bc = rm.B * rm.cn, R = npaths(grouped) * Bc, d = c.d_model;
    dbt_status st;
    int E = c.n_experts, Fe = c.d_expert, km = kmax_of(c), Fs = c.n_shared_experts * Fe;
    LinArgs rl = lin1(lw.router, w.rlogits, E, R, w.X, d);
    if ((st = run_linear<WT>(m, "router", rl)) != DBT_OK) return st;
    int32_t *last = record_experts ? w.last_experts + (size_t)l * paths_of(c) * c.max_batch * km : nullptr;
    if (last && !grouped)
        CUDA_TRY(m, cudaMemsetAsync(last + (size_t)c.max_batch * km, 0xff,
                                    sizeof(int32_t) * (paths_of(c) - 1) * c.max_batch * km, m->stream));
    LAUNCH(m, "route", 0, route_kernel, R, 32, 2 * E * sizeof(float), w.rlogits, 1, (size_t)0, E, Bc, c.k_primary, c.k_branch, km,
           c.router_mode == DBT_ROUTER_REPLAY, w.ridx, w.rwts, last, c.max_batch * km, (const float *)nullptr, 0, 0, d, c.rms_eps);
    int32_t *ucnt = record_experts ? w.union_cnt + l : nullptr;
    if (ucnt) CUDA_TRY(m, cudaMemsetAsync(ucnt, 0, sizeof(int32_t), m->stream));
    LAUNCH(m, "moe_lists", 0, moe_lists_kernel, (E + 127) / 128, 128, 0, w.ridx, R, km, E, m->Rmax, w.ecnt, w.elist, ucnt);
    dim3 g1((Fe + kLinWarps - 1) / kLinWarps, E);
    LAUNCH(m, "expert_gateup", 0, expert_gateup_kernel<WT>, g1, kLinWarps * 32, 0, (const WT *)lw.exp_gate, (const WT *)lw.exp_up,
           Fe, d, w.X, km, w.ecnt, w.elist, m->Rmax, w.Hexp);
    dim3 g2((d + kLinWarps - 1) / kLinWarps, E);
    LAUNCH(m, "expert_down", 0, expert_down_kernel<WT>, g2, kLinWarps * 32, 0, (const WT *)lw.exp_down, Fe, d, w.Hexp, w.ecnt,
           w.elist, m->Rmax, w.Yexp);
    const float *Msh = nullptr;
    // compute-matched allocation (Eq. matched_shared_expert): the shared expert runs on the primary rows only
    const bool matched = grouped && c.compute_matched;
    const int Rs = matched ? Bc : R;
    if (Fs > 0) {  // shared expert(s): every row of both paths; b couples its hidden state
        LinArgs gu{};
        gu.W[0] = lw.sh_gate; gu.W[1] = lw.sh_up; gu.Y[0] = w.Hsh; gu.n_out[0] = Fs; gu.rows[0] = Rs;
        gu.nseg = 2; gu.X = w.X; gu.K = d; gu.epi = EPI_SWIGLU; gu.Bc = Bc; gu.grouped = matched ? 0 : grouped;
        gu.coup = c.moe_b_coupling ? lw.coup_b : nullptr;
        if ((st = run_linear<WT>(m, "shared_gateup", gu)) != DBT_OK) return st;
        LinArgs dn = lin1(lw.sh_down, w.Msh, d, Rs, w.Hsh, Fs, EPI_STORE);
        if ((st = run_linear<WT>(m, "shared_down", dn)) != DBT_OK) return st;
        Msh = w.Msh;
    }
    LAUNCH(m, "moe_combine", 0, moe_combine_kernel, Bc, 256, 0, w.Yexp, Msh, w.ridx, w.rwts, km, Bc, grouped, lw.coup_c,
           matched ? lw.gate_g : (const float *)nullptr, d, w.S);
    return DBT_OK;
}

// The layer stack on `rows` stacked rows (Bc primary rows, then Bc branch rows when grouped).
// Section 4.1 (attention), Eq. mlp / Eq. moe_layer (MLP), in the order the paper gives them.
template <typename WT>
dbt_status run_layers(dbt_model *m, const RowMap &rm, int grouped, bool record_experts) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int Bc = rm.B * rm.cn, R = npaths(grouped) * Bc;
    int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
    size_t pool_layer_elems = (size_t)2 * c.num_pages * c.n_kv_heads * c.page_size * c.head_dim;
    size_t pool_kv_elems = pool_layer_elems / 2;
    int nsplit = (2 * 148 + Bc * c.n_kv_heads - 1) / (Bc * c.n_kv_heads);
    nsplit = nsplit < 1 ? 1 : nsplit > 16 ? 16 : nsplit;
    // compute-matched allocation (Eq. matched_attention): attention is evaluated on the primary rows alone
    const bool matched = grouped && c.compute_matched;
    const int ga = matched ? 0 : grouped, Ra = npaths(ga) * Bc;
    double kv_bytes = 0;  // K and V of every visible position, once per layer
    for (int b = 0; b < rm.B; b++)
        for (int j = 0; j < rm.cn; j++) kv_bytes += (double)(m->len_host[b] + j + 1) * 2 * kvd * sizeof(WT);
    dbt_status st;
    for (int l = 0; l < c.n_layers; l++) {
        const dbt_layer_weights &lw = m->layers[l];
        WT *kpool = reinterpret_cast<WT *>(m->kv_pool) + (size_t)l * pool_layer_elems;
        WT *vpool = kpool + pool_kv_elems;
        // N_i = RMSNorm(S_i)
        LAUNCH(m, "rmsnorm", 0, rmsnorm_kernel, R, 256, 0, w.S, lw.attn_norm_g, c.rms_eps, d, 1, 0, 1, w.X);
        // Q for all rows; K, V for the primary rows only (the branch produces only a query)
        LinArgs a{};
        a.W[0] = lw.wq; a.Y[0] = w.Q; a.n_out[0] = qd; a.rows[0] = Ra;
        a.W[1] = lw.wk; a.Y[1] = w.Kn; a.n_out[1] = kvd; a.rows[1] = Bc;
        a.W[2] = lw.wv; a.Y[2] = w.Vn; a.n_out[2] = kvd; a.rows[2] = Bc;
        a.nseg = 3; a.X = w.X; a.K = d; a.epi = EPI_STORE;
        if ((st = run_linear<WT>(m, "linear_qkv", a)) != DBT_OK) return st;
        LAUNCH(m, "rope_append", 0, rope_couple_append_kernel<WT>, Bc, 256, 0, w.Q, w.Kn, w.Vn, rm, ga, c.n_q_heads, c.n_kv_heads,
               c.head_dim, lw.coup_a, w.rope, w.seq_len, w.page_table, m->pages_per_seq_max, c.num_pages, c.page_size,
               kpool, vpool, w.status);
        if (c.head_dim == 128)
            st = run_attention<WT, 128>(m, rm, ga, kpool, vpool, nsplit, kv_bytes);
        else
            st = run_attention<WT, 64>(m, rm, ga, kpool, vpool, nsplit, kv_bytes);
        if (st != DBT_OK) return st;
        // S-bar_i = S_i + Attn_i W_O  (matched: S-bar_2 = S_2 + g_A * Attn_1 W_O)
        LinArgs o = lin1(lw.wo, nullptr, d, Ra, w.O, qd, matched ? EPI_RESID_GATED : EPI_RESID);
        o.S = w.S; o.Bc = Bc; o.grouped = grouped; o.coup = matched ? lw.gate_a : nullptr;
        if ((st = run_linear<WT>(m, "linear_o", o)) != DBT_OK) return st;
        LAUNCH(m, "rmsnorm", 0, rmsnorm_kernel, R, 256, 0, w.S, lw.mlp_norm_g, c.rms_eps, d, 1, 0, 1, w.X);
        if (c.n_experts == 0) {
            LinArgs gu{};
            gu.W[0] = lw.w_gate; gu.W[1] = lw.w_up; gu.Y[0] = w.G1; gu.n_out[0] = c.d_ff; gu.rows[0] = R;
            gu.nseg = 2; gu.X = w.X; gu.K = d; gu.epi = EPI_SWIGLU; gu.Bc = Bc; gu.grouped = grouped;
            gu.coup = lw.coup_b;
            if ((st = run_linear<WT>(m, "linear_gateup", gu)) != DBT_OK) return st;
            LinArgs dn = lin1(lw.w_down, w.M, d, R, w.G1, c.d_ff, EPI_DOWN);
            dn.Bc = Bc; dn.grouped = grouped; dn.coup = lw.coup_c; dn.S = w.S;
            if ((st = run_linear<WT>(m, "linear_down", dn)) != DBT_OK) return st;
        } else {
            if ((st = run_moe<WT>(m, l, rm, grouped, record_experts)) != DBT_OK) return st;
        }
    }
    return DBT_OK;
}

// Final norm + shared output matrix on `rows` rows taken from S (row r*src_mul+src_add).
template <typename WT>
dbt_status run_head(dbt_model *m, int rows, int src_mul, int src_add) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    LAUNCH(m, "rmsnorm", 0, rmsnorm_kernel, rows, 256, 0, w.S, m->w.final_norm_g, c.rms_eps, c.d_model, src_mul, src_add,
           c.final_norm, w.Zrows);
    LinArgs a = lin1(m->w.lm_head, w.Z, c.vocab, rows, w.Zrows, c.d_model);
    return run_linear<WT>(m, "lm_head", a);
}

// ---- tensor-core path (bf16 weights) -----------------------------------------------------

struct TcCall {
    const CUtensorMap *W[3];
    int n_out[3];
    int rows[3];
    int nseg;
    const CUtensorMap *X;
    int K;
    int R;  // activation rows whose outputs are stored
    float *P;
    size_t P_floats;
    const char *tag;
    int parts;    // 1 or 2 bf16 terms per activation
    int lo_row0;  // row of the lo plane in the activation buffer
    const int *grp_cnt, *grp_off;  // per-expert mode (see TcParams); n_groups experts
    int grp_w_rows, n_groups;
    int grp_row_tiles;  // per-expert mode: row tiles of n_tile rows per expert (0: one tile holds any list)
    int grp_prewait;    // per-expert mode: the lists are final before this launch can be resident (see TcParams)
    int grp_mt2;        // per-expert mode, 64-row tiles: two weight tiles per CTA share each activation box (prompt chunks)
    // per-expert gate|up launch: where it runs as persistent CTAs it may apply the SwiGLU itself (see SwigluEpi);
    // *fused tells the caller whether it did
    const SwigluEpi *swiglu;
    bool *fused;
    // dense gate|up launch over a prompt chunk: gate and up tiles of the same features in one CTA, SwiGLU in the
    // epilogue (see GuEpi); *gu_fused tells the caller whether it was taken
    const GuEpi *gu;
    bool *gu_fused;
};

int norm_threads(int d) { return d >= 1024 ? 1024 : d >= 512 ? 512 : 256; }
int pad_rows(int r) { return r <= 16 ? 16 : r <= 32 ? 32 : r <= 64 ? 64 : r <= 128 ? 128 : 256; }

// Split-K factor from the tile count and K only (never from the mode), so that grouped and
// primary-only steps add the same partials in the same order.
int choose_split(int tiles, int total_kt, int slots) {
    int best = 1;
    double best_cost = 1e30;
    for (int s = 1; s <= total_kt && s <= 16; s++) {
        int kt = (total_kt + s - 1) / s;
        int s_eff = (total_kt + kt - 1) / kt;
        int waves = (tiles * s_eff + slots - 1) / slots;
        double cost = waves * (kt + 3.0);
        if (cost < best_cost - 1e-9) {
            best_cost = cost;
            best = s_eff;
        }
    }
    return best;
}

// CTAs of the GEMM kernel that are resident at once: two per SM up to a row tile of 64 (96 KB of
// ring each), one above.
int split_slots(const dbt_model *m, int n_tile) {
    int sms = m->num_sms > 0 ? m->num_sms : 148;  // the operator-level entry points carry no device query
    return (n_tile <= 64 ? 2 : 1) * sms;
}

template <int N_TILE, int MT = 1>
dbt_status launch_gemm_tc(dbt_model *m, const TcCall &c, const TcParams &p, const LmEpi &e, dim3 grid, double bytes) {
    const CUtensorMap *w1 = c.nseg > 1 ? c.W[1] : c.W[0], *w2 = c.nseg > 2 ? c.W[2] : c.W[0];
    const CUtensorMap *x = c.X;
    TcParams pp = p;
    auto reg = m->act_base.find(c.X);
    if (c.parts == 2 && reg != m->act_base.end()) {
        auto key = std::make_tuple(c.X, N_TILE, c.lo_row0);
        auto hit = m->act3d.find(key);
        if (hit == m->act3d.end()) {
            CUtensorMap t;
            if (make_act_map(&t, reg->second.base, (uint64_t)c.lo_row0, (uint64_t)c.K, N_TILE)) hit = m->act3d.emplace(key, t).first;
        }
        if (hit != m->act3d.end()) {
            x = &hit->second;
            pp.x3d = 1;
            pp.stacked = N_TILE <= 128 ? 1 : 0;
        }
    }
    if constexpr (N_TILE <= 32 && MT == 1) {
        // per-expert launches with short row tiles: persistent CTAs over the units that have work
        // (chosen from the batch and the model only, like every other launch shape: measured 1-3 % faster up to 16
        // stacked rows, within +-2 % of the one-CTA-per-unit launch above that; same bits either way)
        const bool want = m->moe_persist < 0 ? paths_of(m->cfg) * m->cur_rows <= 16 : m->moe_persist > 0;
        if (c.grp_cnt && want && pp.x3d && pp.stacked && c.nseg <= 2 && c.n_groups <= kPersistMaxGroups) {
            if (N_TILE == 16 && c.swiglu && c.fused && c.nseg == 2 && c.n_out[0] == c.n_out[1] && m->moe_fuse_swiglu) {
                const int smem = TcPersistCfg<N_TILE, true>::smem_bytes(c.n_groups);
                if (cudaFuncSetAttribute(gemm_tc_persist_kernel<N_TILE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
                    cudaSuccess)
                    return fail(m, DBT_ERR_CUDA, "shared memory opt-in for the persistent per-expert GEMM");
                LAUNCH(m, c.tag, bytes, (gemm_tc_persist_kernel<N_TILE, true>), dim3(2 * m->num_sms), 192, smem, *c.W[0], *w1, *x, pp,
                       c.n_groups, (int)grid.x / 2, *c.swiglu);
                *c.fused = true;
                return DBT_OK;
            }
            const int smem = TcPersistCfg<N_TILE>::smem_bytes(c.n_groups);
            if (cudaFuncSetAttribute(gemm_tc_persist_kernel<N_TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
                return fail(m, DBT_ERR_CUDA, "shared memory opt-in for the persistent per-expert GEMM");
            LAUNCH(m, c.tag, bytes, gemm_tc_persist_kernel<N_TILE>, dim3(2 * m->num_sms), 192, smem, *c.W[0], *w1, *x, pp, c.n_groups,
                   (int)grid.x, SwigluEpi{});
            return DBT_OK;
        }
    }
    LAUNCH(m, c.tag, bytes, (gemm_tc_kernel<N_TILE, MT>), grid, 128, (TcCfg<N_TILE, MT>::kSmemBytes), *c.W[0], *w1, *w2, *x, pp, e);
    return DBT_OK;
}

// Y partials P[split][R][ldp]; returns the split count and stride the consumer must use.
dbt_status run_gemm_tc(dbt_model *m, const TcCall &c, int n_tile, int *nsplit_out, size_t *split_stride_out,
                       int force_split = 0, LmEpi e = LmEpi{}, int test_skip_load = 0) {
    TcParams p{};
    int tiles = 0, col = 0;
    double bytes = 0;
    // prompt chunks (more rows than the widest tile): two weight tiles per CTA share every activation box where
    // that pays -- such a CTA takes ~1.6x as long as a one-tile CTA, so the choice goes by full waves of CTAs
    int mt = 1;
    if (!c.grp_cnt && c.R > 256) {
        int t1 = 0, t2 = 0;
        for (int s = 0; s < c.nseg; s++) {
            t1 += (c.n_out[s] + kTcM - 1) / kTcM;
            t2 += (c.n_out[s] + 2 * kTcM - 1) / (2 * kTcM);
        }
        const int rt = (c.R + 255) / 256, sms = m->num_sms;
        const int w1 = (t1 * rt + sms - 1) / sms, w2 = (t2 * rt + sms - 1) / sms;
        if (16 * w2 < 10 * w1) mt = 2;
    }
    if (c.grp_cnt && c.grp_mt2 && n_tile == 64) mt = 2;
    const bool gu_pair = !c.grp_cnt && c.R > 256 && c.gu && c.gu_fused && c.nseg == 2 && c.n_out[0] == c.n_out[1] && c.n_out[0] % 8 == 0 &&
                         m->prompt_fuse_swiglu;
    if (gu_pair) mt = 2;
    for (int s = 0; s < c.nseg; s++) {
        p.seg[s] = TcSeg{tiles, c.n_out[s], c.rows[s], col};
        tiles += (c.n_out[s] + kTcM * mt - 1) / (kTcM * mt);
        col += c.n_out[s];
        if (!c.grp_cnt) bytes += (double)c.n_out[s] * c.K * 2;  // per-expert launches: the loaded set is known on the device only
    }
    p.nseg = c.nseg;
    if (gu_pair) {  // tiles of 128 features, each with its gate and its up rows
        p.seg[0] = TcSeg{0, c.n_out[0], c.rows[0], 0};
        p.nseg = 1;
        tiles = (c.n_out[0] + kTcM - 1) / kTcM;
        p.gu = *c.gu;
        p.gu.on = 1;
        *c.gu_fused = true;
    }
    p.K = c.K;
    p.ldp = col;
    p.R = c.R;
    p.parts = c.parts;
    p.lo_row0 = c.lo_row0;
    p.grp_cnt = c.grp_cnt;
    p.grp_off = c.grp_off;
    p.grp_w_rows = c.grp_w_rows;
    p.grp_row_tiles = c.grp_cnt ? c.grp_row_tiles : 0;
    p.grp_prewait = c.grp_cnt ? c.grp_prewait : 0;
    p.P = c.P;
    p.status = m->ws.status;
    p.evict_first = m->evict_first ? 1 : 0;
    p.test_skip_load = test_skip_load;
    // more rows than the widest tile (prompt chunks): several row tiles per weight tile, no split-K
    int row_tiles = 1;
    if (!c.grp_cnt && c.R > 256) {
        if (e.Z) return fail(m, DBT_ERR_UNSUPPORTED, "the output-matrix epilogue takes at most 256 rows");
        n_tile = 256;
        row_tiles = (c.R + 255) / 256;
        force_split = 1;
    }
    p.row_tiles = row_tiles;
    int total_kt = (c.K + kTcK - 1) / kTcK;
    if (c.grp_cnt) force_split = 1;  // enough CTAs already: tiles x selected experts
    int split = force_split > 0 ? (force_split < total_kt ? force_split : total_kt) : choose_split(tiles, total_kt, split_slots(m, n_tile));
    while (split > 1 && (size_t)split * n_tile * col > c.P_floats) split--;
    if ((size_t)c.R * col > c.P_floats) return fail(m, DBT_ERR_CAPACITY, "partial buffer too small for %s", c.tag);
    p.kt_per_split = (total_kt + split - 1) / split;
    split = (total_kt + p.kt_per_split - 1) / p.kt_per_split;
    if (e.Z) {  // the output matrix has tiles enough: unsplit, logits straight from the accumulator
        split = 1;
        p.kt_per_split = total_kt;
    }
    dim3 grid(tiles * row_tiles, c.grp_cnt && c.grp_row_tiles ? c.grp_row_tiles : split, c.grp_cnt ? c.n_groups : 1);
    if (nsplit_out) *nsplit_out = split;
    if (split_stride_out) *split_stride_out = (size_t)c.R * col;
    switch (n_tile) {
        case 16: return launch_gemm_tc<16>(m, c, p, e, grid, bytes);
        case 32: return launch_gemm_tc<32>(m, c, p, e, grid, bytes);
        case 64: return mt == 2 ? launch_gemm_tc<64, 2>(m, c, p, e, grid, bytes) : launch_gemm_tc<64>(m, c, p, e, grid, bytes);
        case 128: return launch_gemm_tc<128>(m, c, p, e, grid, bytes);
        case 256: return mt == 2 ? launch_gemm_tc<256, 2>(m, c, p, e, grid, bytes) : launch_gemm_tc<256>(m, c, p, e, grid, bytes);
    }
    return fail(m, DBT_ERR_UNSUPPORTED, "row tile %d", n_tile);
}

// Inputs of the Q|K|V epilogue when the attention kernel does that work itself (decode steps).
struct QkvFuse {
    const float *P;
    int nsplit;
    size_t stride;
    const float *ss;
    int ss_tiles, ss_ld;
    const float *coup_a;
};

// One deep-ring CTA per SM instead of two CTAs per SM: when the (sequence, KV head) pairs fill one wave of SMs,
// every pair goes to one CTA, so no pair is split and there are no partials to write, no tickets and no merge.
// Chosen from the batch and the model, never from the mode or the lengths (a captured step serves every length).
bool attn_deep(const dbt_model *m, int items) {
    const dbt_config &c = m->cfg;
    const int pairs = items * c.n_kv_heads, G = c.n_q_heads / c.n_kv_heads;
    return paths_of(c) * G <= 8 && 2 * pairs > m->num_sms && pairs <= m->num_sms;
}

// The attention work split of a decode step, once for all its layers.
dbt_status run_attention_plan(dbt_model *m, const RowMap &rm) {
    const dbt_config &c = m->cfg;
    const int items = rm.B * rm.cn;
    if (items > kAttMaxItems) return DBT_OK;  // (the attention launch reports the capacity error)
    LAUNCH(m, "attn_plan", 0, attn_plan_kernel, 1, 32, 0, rm, m->ws.seq_len, c.n_kv_heads,
           attn_deep(m, items) ? m->num_sms : 2 * m->num_sms, m->ws.att_plan);
    m->att_planned = true;  // cleared by the step function when its layers have been enqueued
    return DBT_OK;
}

template <int DH>
dbt_status run_attention_mma(dbt_model *m, const RowMap &rm, int grouped, int layer, double kv_bytes,
                             const QkvFuse *qf = nullptr, bool pack_prompt = false, bool planned = false) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int items = rm.B * rm.cn, G = c.n_q_heads / c.n_kv_heads;
    AttnParams p{};
    p.Q = w.Q;
    p.rm = rm;
    p.grouped = grouped;
    p.G = G;
    p.n_kv = c.n_kv_heads;
    p.num_pages = c.num_pages;
    p.pt_stride = m->pages_per_seq_max;
    long long plane = (long long)c.num_pages * c.n_kv_heads * c.page_size;
    p.k_row0 = (long long)layer * 2 * plane;
    p.page_table = w.page_table;
    p.seq_len = w.seq_len;
    p.part = w.part;
    p.tickets = w.att_tickets;
    p.tickets2 = w.att_tickets2;
    p.Ob = w.Ob;
    p.lo_off = m->act_parts == 2 ? (size_t)m->Rmax * c.n_q_heads * c.head_dim : (size_t)0;
    p.status = w.status;
    p.evict_first = m->evict_first ? 1 : 0;
    if (qf) {
        p.qkv_P = qf->P;
        p.qkv_nsplit = qf->nsplit;
        p.qkv_stride = qf->stride;
        p.ss = qf->ss;
        p.ss_tiles = qf->ss_tiles;
        p.ss_ld = qf->ss_ld;
        p.d_norm = c.d_model;
        p.eps = c.rms_eps;
        p.coup_a = qf->coup_a;
        p.rope = w.rope;
        p.kpool = reinterpret_cast<__nv_bfloat16 *>(m->kv_pool) + (size_t)layer * 2 * plane * c.head_dim;
        p.vpool = p.kpool + (size_t)plane * c.head_dim;
    }
    // prompt chunks: 16 / G consecutive positions of a sequence share a query tile (the 16-row kernel)
    const bool packed = pack_prompt && !grouped && !qf && rm.cn > 1;
    if (packed && 16 % G == 0 && !m->prompt_attn_off) {
        // the prompt kernel: eight query tiles per CTA share every page the CTA brings in
        PromptAttnParams q{};
        q.Q = w.Q;
        q.B = rm.B;
        q.cn = rm.cn;
        q.G = G;
        q.n_kv = c.n_kv_heads;
        q.num_pages = c.num_pages;
        q.pt_stride = m->pages_per_seq_max;
        q.k_row0 = p.k_row0;
        q.page_table = w.page_table;
        q.seq_len = w.seq_len;
        q.Ob = w.Ob;
        q.lo_off = p.lo_off;
        q.status = w.status;
        q.nqb = (rm.cn + kPaWarps * (16 / G) - 1) / (kPaWarps * (16 / G));
        dim3 gp(rm.B * c.n_kv_heads * q.nqb);
        LAUNCH(m, "attention", kv_bytes, attn_prompt_kernel<DH>, gp, (kPaWarps + 1) * 32, PromptAttCfg<DH>::kSmemBytes, m->map_kv, q);
        return DBT_OK;
    }
    if (packed) {
        p.pack = 16 / G;
        p.cn = rm.cn;
        p.nbk = (rm.cn + p.pack - 1) / p.pack;
    }
    if (planned && !packed) {  // from the second layer on the plan may be read before the dependency wait
        p.plan = m->ws.att_plan;
        p.plan_prewait = layer > 0 ? 1 : 0;
    }
    if (!packed && items > kAttMaxItems) return fail(m, DBT_ERR_CAPACITY, "attention rows %d exceed %d", items, kAttMaxItems);
    dim3 grid(2 * m->num_sms);  // two resident CTAs per SM; each takes an equal share of all K/V tiles
    if (!packed && attn_deep(m, items)) {
        dim3 g1(m->num_sms);
        LAUNCH(m, "attention", kv_bytes, (attn_mma_kernel<DH, true, true>), g1, 160, (AttCfg<DH, true>::kSmemBytes), m->map_kv, p);
        return DBT_OK;
    }
    // up to 8 query rows per KV head over both paths: the transposed-product variant (fixed per
    // model, so that grouped and primary-only steps run the same arithmetic on the primary rows)
    if (paths_of(c) * G <= 8 && !packed)
        LAUNCH(m, "attention", kv_bytes, (attn_mma_kernel<DH, true>), grid, 160, AttCfg<DH>::kSmemBytes, m->map_kv, p);
    else
        LAUNCH(m, "attention", kv_bytes, (attn_mma_kernel<DH, false>), grid, 160, AttCfg<DH>::kSmemBytes, m->map_kv, p);
    return DBT_OK;
}

// MoE sub-layer on the tensor cores (Eq. moe_layer, Eq. moe_budget, Section 4.3).  Rows of both
// paths are sorted by expert; one grouped GEMM launch covers all experts (blockIdx.z), CTAs of
// experts nobody selected exit before touching their weights, so each selected expert's
// matrices are read once for the union of the primary top-k_1 and branch top-k_2 rows.
// wide: the rows in Xb are g * S, not yet divided by rms(S) (shares of sum(S^2) in ws.ss): every
// consumer of a GEMM on them applies the row's factor itself, and the combine leaves the next layer's
// input in the same form when it is given that layer's gain g_next.
dbt_status run_moe_tc(dbt_model *m, int l, const RowMap &rm, int grouped, bool record_experts, bool wide,
                      const float *g_next) {
    typedef __nv_bfloat16 WT;
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    const dbt_layer_weights &lw = m->layers[l];
    const LayerMaps &mp = m->maps[l];
    int Bc = rm.B * rm.cn, R = npaths(grouped) * Bc, d = c.d_model;
    int E = c.n_experts, Fe = c.d_expert, km = kmax_of(c), Fs = c.n_shared_experts * Fe, Rk = m->Rmax * km;
    // Row tile (and with it the resident-CTA count that sizes the split-K factors of the router and the shared
    // expert) from the batch, never from the mode: a primary-only step uses the tile of the grouped step, so both
    // add the same partials in the same order and write the same K/V bits.
    int n_tile = pad_rows(paths_of(c) * Bc <= 256 ? paths_of(c) * Bc : 256);
    m->cur_rows = Bc;
    size_t lo_x = m->act_parts == 2 ? (size_t)m->Rmax * d : 0;
    size_t lo_xs = m->act_parts == 2 ? (size_t)Rk * d : 0, lo_hs = m->act_parts == 2 ? (size_t)Rk * Fe : 0;
    const float *ssp = wide ? w.ss : nullptr;
    const int ss_tiles = (d + 255) / 256, ss_ld = m->Rmax;
    dbt_status st;
    // shared expert(s) on every row of both paths; b couples its hidden state
    const float *Psh = nullptr;
    int nsp = 1;
    size_t sstride = 0;
    // compute-matched allocation (Eq. matched_shared_expert): the shared expert runs on the primary rows only
    const bool matched = grouped && c.compute_matched;
    const int Rs = matched ? Bc : R;
    auto shared_expert = [&](float *Pbuf, size_t Pbuf_floats) -> dbt_status {
        int nt = n_tile;
        TcCall sg{};
        sg.W[0] = &mp.wg; sg.n_out[0] = Fs; sg.rows[0] = Rs;
        sg.W[1] = &mp.wu; sg.n_out[1] = Fs; sg.rows[1] = Rs;
        sg.nseg = 2; sg.X = &m->map_Xb; sg.K = d; sg.R = Rs; sg.P = Pbuf; sg.P_floats = Pbuf_floats; sg.tag = "shared_gateup";
        sg.parts = m->act_parts; sg.lo_row0 = m->Rmax;
        if ((st = run_gemm_tc(m, sg, nt, &nsp, &sstride)) != DBT_OK) return st;
        LAUNCH(m, "swiglu_couple", 0, swiglu_couple_kernel, dim3(Bc, (Fs + 255) / 256, branch_blocks(matched ? 0 : grouped)), 256, 0, Pbuf, nsp, sstride, Fs, Bc,
               matched ? 0 : grouped, c.moe_b_coupling ? lw.coup_b : (const float *)nullptr, w.Hb,
               m->act_parts == 2 ? (size_t)m->Rmax * Fs : (size_t)0, ssp, ss_tiles, ss_ld, d, c.rms_eps);
        TcCall sd{};
        sd.W[0] = &mp.wd; sd.n_out[0] = d; sd.rows[0] = Rs; sd.nseg = 1; sd.X = &m->map_Hb; sd.K = Fs; sd.R = Rs;
        sd.P = Pbuf; sd.P_floats = Pbuf_floats; sd.tag = "shared_down"; sd.parts = m->act_parts; sd.lo_row0 = m->Rmax;
        if ((st = run_gemm_tc(m, sd, nt, &nsp, &sstride)) != DBT_OK) return st;
        Psh = Pbuf;
        return DBT_OK;
    };
    // The shared expert depends on the normalised rows only: its three kernels run on a second stream
    // beside the router, the routing kernels and the routed experts, and join before the combine.
    const bool overlap = Fs > 0 && m->moe_overlap && m->side_stream;
    cudaStream_t main_stream = m->stream;
    if (overlap) {
        CUDA_TRY(m, cudaEventRecord(m->ev_fork, main_stream));
        CUDA_TRY(m, cudaStreamWaitEvent(m->side_stream, m->ev_fork, 0));
        m->stream = m->side_stream;
        st = shared_expert(w.P2, w.P2_floats);
        m->stream = main_stream;
        if (st != DBT_OK) return st;
        CUDA_TRY(m, cudaEventRecord(m->ev_join, m->side_stream));
    }
    // router logits on the tensor cores (split-K partials summed by the routing kernel), then
    // top-k per path and renormalised weights
    int rnsp = 1;
    size_t rstride = 0;
    TcCall rt{};
    rt.W[0] = &mp.rt; rt.n_out[0] = E; rt.rows[0] = R; rt.nseg = 1; rt.X = &m->map_Xb; rt.K = d; rt.R = R;
    rt.P = w.P; rt.P_floats = w.P_floats; rt.tag = "router"; rt.parts = m->act_parts; rt.lo_row0 = m->Rmax;
    if ((st = run_gemm_tc(m, rt, n_tile, &rnsp, &rstride)) != DBT_OK) return st;
    int32_t *last = record_experts ? w.last_experts + (size_t)l * paths_of(c) * c.max_batch * km : nullptr;
    if (last && !grouped)
        CUDA_TRY(m, cudaMemsetAsync(last + (size_t)c.max_batch * km, 0xff, sizeof(int32_t) * (paths_of(c) - 1) * c.max_batch * km,
                                    m->stream));
    LAUNCH(m, "route", 0, route_kernel, R, 32, 2 * E * sizeof(float), w.P, rnsp, rstride, E, Bc, c.k_primary, c.k_branch, km,
           c.router_mode == DBT_ROUTER_REPLAY, w.ridx, w.rwts, last, c.max_batch * km, ssp, ss_tiles, ss_ld, d, c.rms_eps);
    LAUNCH(m, "moe_sort", 0, moe_sort_kernel, 1, R * km > 512 ? 1024 : (E + 31) / 32 * 32 < 64 ? 64 : (E + 31) / 32 * 32, 0, w.ridx, R, km, E, w.ecnt, w.eoff, w.epos,
           record_experts ? w.union_cnt + l : (int32_t *)nullptr);
    LAUNCH(m, "moe_gather", 0, moe_gather_kernel, R * km, 256, 0, w.Xb, lo_x, w.ridx, w.epos, km, d, w.Xs, lo_xs, ssp, ss_tiles, ss_ld,
           c.rms_eps, w.rs_sorted);
    // routed experts: gate|up, SwiGLU, down
    TcCall gu{};
    gu.W[0] = &mp.eg; gu.n_out[0] = Fe; gu.rows[0] = Rk;
    gu.W[1] = &mp.eu; gu.n_out[1] = Fe; gu.rows[1] = Rk;
    gu.nseg = 2; gu.X = &m->map_Xs; gu.K = d; gu.R = Rk; gu.P = w.Pe; gu.P_floats = (size_t)Rk * 2 * Fe;
    gu.tag = "expert_gateup"; gu.parts = m->act_parts; gu.lo_row0 = Rk;
    gu.grp_cnt = w.ecnt; gu.grp_off = w.eoff; gu.grp_w_rows = Fe; gu.n_groups = E;
    // An expert's list is short on average (rows x k / experts) but may hold every row: row tiles of
    // 16 rows (32 from 64 sequences on; chosen from the batch, not the mode, so that grouped and
    // primary-only steps use the same instruction shape), as many per expert as the rows of this step
    // could need, keep two CTAs per SM and their deeper rings at large batches (measured: 4.86 -> 4.53 ms
    // at batch 32, 6.43 -> 4.81 at batch 64).  DBT_MOE_ROWTILE=0: one tile of all rows; 16/32/64: that tile.
    int gt = n_tile, grt = 0;
    // (prompt chunks of more than 256 rows: tiles of 64 rows, an expert's share of such a chunk)
    const int want_tile = m->moe_row_tile >= 0 ? m->moe_row_tile : (paths_of(c) * Bc <= 64 ? 16 : Bc <= 256 ? 32 : 64);
    if (want_tile > 0 && n_tile > want_tile) {
        gt = want_tile;
        grt = (R + gt - 1) / gt;
    }
    gu.grp_row_tiles = grt;
    gu.grp_mt2 = (gt == 64 && Bc > 256) ? 1 : 0;
    gu.grp_prewait = m->use_pdl ? 1 : 0;  // the gather kernel before it lets its dependents in only after its own wait
    const SwigluEpi se{w.Hs, lo_hs, wide ? (const float *)w.rs_sorted : (const float *)nullptr, Fe};
    bool swiglu_done = false;
    gu.swiglu = &se;
    gu.fused = &swiglu_done;
    if ((st = run_gemm_tc(m, gu, gt, nullptr, nullptr)) != DBT_OK) return st;
    if (!swiglu_done)
        LAUNCH(m, "moe_swiglu", 0, moe_swiglu_kernel, dim3(R * km, (Fe + 255) / 256), 256, 0, w.Pe, w.eoff + E, Fe, w.Hs, lo_hs,
               wide ? (const float *)w.rs_sorted : (const float *)nullptr);
    TcCall dn{};
    dn.W[0] = &mp.ed; dn.n_out[0] = d; dn.rows[0] = Rk; dn.nseg = 1; dn.X = &m->map_Hs; dn.K = Fe; dn.R = Rk;
    dn.P = w.Yexp; dn.P_floats = (size_t)Rk * d; dn.tag = "expert_down"; dn.parts = m->act_parts; dn.lo_row0 = Rk;
    dn.grp_cnt = w.ecnt; dn.grp_off = w.eoff; dn.grp_w_rows = d; dn.n_groups = E;
    dn.grp_row_tiles = grt;
    dn.grp_mt2 = gu.grp_mt2;
    // The lists come from the sort kernel, several launches back.  A CTA of this launch can only be resident once
    // every CTA of the launch before it has started (the SwiGLU kernel, or the gate|up GEMM where that applies the
    // SwiGLU itself), hence once every CTA of the gate|up GEMM is resident, hence once every CTA of the gather kernel
    // has let its dependents in -- which it does only after its own wait on the sort kernel.
    dn.grp_prewait = m->use_pdl ? 1 : 0;
    if ((st = run_gemm_tc(m, dn, gt, nullptr, nullptr)) != DBT_OK) return st;
    if (Fs > 0 && !overlap && (st = shared_expert(w.P, w.P_floats)) != DBT_OK) return st;
    if (overlap) CUDA_TRY(m, cudaStreamWaitEvent(main_stream, m->ev_join, 0));
    const bool next_in = wide && g_next != nullptr;
    if (!grouped && wide && rm.cn > 1 && Bc > 256 && d % 4 == 0 && ((size_t)m->Rmax * d) % 4 == 0) {  // prompt chunks: the vector form
        LAUNCH(m, "moe_combine", 0, moe_combine_rows_kernel, dim3((Bc + 3) / 4, (d + 255) / 256), 256, 0, w.Yexp, Psh, nsp, sstride, w.ridx,
               w.epos, w.rwts, km, Bc, d, w.S, next_in ? g_next : (const float *)nullptr, next_in ? w.Xb : (__nv_bfloat16 *)nullptr, lo_x,
               next_in ? w.ss : (float *)nullptr, ss_ld);
        return DBT_OK;
    }
    LAUNCH_BR(m, grouped, "moe_combine", 0, moe_combine_sorted_kernel, dim3(Bc, (d + 255) / 256, branch_blocks(grouped)), 256, 0, w.Yexp, Psh, nsp, sstride, w.ridx, w.epos, w.rwts, km,
           Bc, grouped, lw.coup_c, matched ? lw.gate_g : (const float *)nullptr, d, w.S, next_in ? g_next : (const float *)nullptr,
           next_in ? w.Xb : (__nv_bfloat16 *)nullptr, lo_x, next_in ? w.ss : (float *)nullptr, ss_ld);
    return DBT_OK;
}

// bf16 layer stack: TMA + tcgen05 GEMMs with the elementwise work between them fused into
// three small kernels.  On return the last layer's MLP output is still pending in P (dense
// models): `pending` tells the caller how to fold it into S (mode of resid_norm_kernel).
dbt_status run_layers_tc(dbt_model *m, const RowMap &rm, int grouped, int n_tile, bool record_experts, int *pending_mode,
                         int *pending_split, size_t *pending_stride) {
    typedef __nv_bfloat16 WT;
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int Bc = rm.B * rm.cn, R = npaths(grouped) * Bc;
    int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
    size_t pool_layer_elems = (size_t)2 * c.num_pages * c.n_kv_heads * c.page_size * c.head_dim;
    size_t pool_kv_elems = pool_layer_elems / 2;
    int att_split = (2 * 148 + Bc * c.n_kv_heads - 1) / (Bc * c.n_kv_heads);
    att_split = att_split < 1 ? 1 : att_split > 16 ? 16 : att_split;
    double kv_bytes = 0;
    for (int b = 0; b < rm.B; b++)
        for (int j = 0; j < rm.cn; j++) kv_bytes += (double)(m->len_host[b] + j + 1) * 2 * kvd * sizeof(WT);
    bool moe = c.n_experts > 0;
    // compute-matched allocation (Eq. matched_attention): attention is evaluated on the primary rows alone
    const bool matched = grouped && c.compute_matched;
    const int ga = matched ? 0 : grouped, Ra = npaths(ga) * Bc;
    // MoE on the tensor cores: norm factor behind the GEMMs, no row-wide reduction kernel (DBT_MOE_WIDE=0: before them)
    const bool mwide = moe && m->moe_tc && m->moe_wide;
    const int mss_tiles = (d + 255) / 256;
    size_t lo_x = m->act_parts == 2 ? (size_t)m->Rmax * d : 0;
    // prompt chunks of more than one row tile (MoE models): the prompt attention kernel and the vector forms of the
    // kernels around it, as in the dense prompt pass
    const bool rows_form = mwide && m->att_fast && !grouped && rm.cn > 1 && Bc > 256 && d % 4 == 0 && c.head_dim % 8 == 0 &&
                           ((size_t)m->Rmax * d) % 4 == 0;
    dbt_status st;
    int mode = 0, nsp = 1;
    size_t sstride = 0;
    for (int l = 0; l < c.n_layers; l++) {
        const dbt_layer_weights &lw = m->layers[l];
        const LayerMaps &mp = m->maps[l];
        WT *kpool = reinterpret_cast<WT *>(m->kv_pool) + (size_t)l * pool_layer_elems;
        WT *vpool = kpool + pool_kv_elems;
        // fold the previous layer's MLP output into S (Eq. mlp), N_i = RMSNorm(S_i).  MoE, wide form: the
        // GEMM input is g * S with the 1/rms factor applied behind the GEMM; the previous layer's combine
        // has left it already, the first layer gets it from the residual kernel with nothing to add.
        if (mwide) {
            if (l == 0)
                LAUNCH_BR(m, grouped, "resid_wide", 0, resid_wide_kernel, dim3(Bc, mss_tiles, branch_blocks(grouped)), 256, 0, w.S, w.P, 0, (size_t)0, 1,
                       (const float *)nullptr, Bc, grouped, lw.attn_norm_g, d, w.Xb, lo_x, w.ss, m->Rmax);
        } else {
            LAUNCH(m, "resid_norm", 0, resid_norm_kernel, dim3(Bc, 1, branch_blocks(grouped)), norm_threads(d), 0, w.S, w.P, nsp, sstride, mode,
                   l > 0 ? m->layers[l - 1].coup_c : nullptr, Bc, grouped, lw.attn_norm_g, c.rms_eps, d, 1, 1, 0, w.Xb,
                   lo_x, (float *)nullptr);
        }
        TcCall qkv{};
        qkv.W[0] = &mp.wq; qkv.n_out[0] = qd; qkv.rows[0] = Ra;
        qkv.W[1] = &mp.wk; qkv.n_out[1] = kvd; qkv.rows[1] = Bc;
        qkv.W[2] = &mp.wv; qkv.n_out[2] = kvd; qkv.rows[2] = Bc;
        qkv.nseg = 3; qkv.X = &m->map_Xb; qkv.K = d; qkv.R = Ra; qkv.P = w.P; qkv.P_floats = w.P_floats; qkv.parts = m->act_parts; qkv.lo_row0 = m->Rmax; qkv.tag = "gemm_qkv";
        if ((st = run_gemm_tc(m, qkv, n_tile, &nsp, &sstride)) != DBT_OK) return st;
        const bool fuse = m->fuse_qkv && m->att_fast && rm.cn == 1;
        QkvFuse qf{w.P, nsp, sstride, mwide ? w.ss : nullptr, mwide ? mss_tiles : 0, mwide ? m->Rmax : 0, lw.coup_a};
        if (rows_form)
            LAUNCH(m, "qkv_epilogue", 0, qkv_rows_kernel, dim3(Bc, ((c.n_q_heads + c.n_kv_heads) * (c.head_dim / 8) + 255) / 256), 256, 0,
                   w.P, nsp, sstride, w.Q, rm, c.n_q_heads, c.n_kv_heads, c.head_dim, w.rope, w.seq_len, w.page_table,
                   m->pages_per_seq_max, c.num_pages, c.page_size, kpool, vpool, w.status, (const float *)w.ss, mss_tiles, m->Rmax, d,
                   c.rms_eps);
        else if (!fuse)
            LAUNCH(m, "qkv_epilogue", 0, qkv_epilogue_kernel<WT>, dim3(Bc, c.n_q_heads + c.n_kv_heads, branch_blocks(ga)), 64, 0, w.P, nsp, sstride, w.Q, rm, ga, c.n_q_heads,
                   c.n_kv_heads, c.head_dim, lw.coup_a, w.rope, w.seq_len, w.page_table, m->pages_per_seq_max, c.num_pages,
                   c.page_size, kpool, vpool, w.status, mwide ? (const float *)w.ss : (const float *)nullptr, mwide ? mss_tiles : 0,
                   mwide ? m->Rmax : 0, d, c.rms_eps);
        if (m->att_fast)
            st = c.head_dim == 128 ? run_attention_mma<128>(m, rm, ga, l, kv_bytes, fuse ? &qf : nullptr, rows_form, m->att_planned)
                                   : run_attention_mma<64>(m, rm, ga, l, kv_bytes, fuse ? &qf : nullptr, rows_form, m->att_planned);
        else if (c.head_dim == 128)
            st = run_attention<WT, 128>(m, rm, ga, kpool, vpool, att_split, kv_bytes, true);
        else
            st = run_attention<WT, 64>(m, rm, ga, kpool, vpool, att_split, kv_bytes, true);
        if (st != DBT_OK) return st;
        TcCall op{};
        op.W[0] = &mp.wo; op.n_out[0] = d; op.rows[0] = Ra; op.nseg = 1; op.X = &m->map_Ob; op.K = qd; op.R = Ra;
        op.P = w.P; op.P_floats = w.P_floats; op.parts = m->act_parts; op.lo_row0 = m->Rmax; op.tag = "gemm_o";
        if ((st = run_gemm_tc(m, op, n_tile, &nsp, &sstride)) != DBT_OK) return st;
        // S-bar_i = S_i + Attn_i W_O (matched: S-bar_2 = S_2 + g_A * Attn_1 W_O) ; RMSNorm for the MLP
        if (rows_form)
            LAUNCH(m, "resid_wide", 0, resid_rows_kernel, dim3((Bc + 3) / 4, mss_tiles), 256, 0, w.S, w.P, nsp, sstride, lw.mlp_norm_g, Bc, d,
                   w.Xb, lo_x, w.ss, m->Rmax);
        else if (mwide)
            LAUNCH_BR(m, grouped, "resid_wide", 0, resid_wide_kernel, dim3(Bc, mss_tiles, branch_blocks(grouped)), 256, 0, w.S, w.P, nsp, sstride, matched ? 3 : 1,
                   matched ? lw.gate_a : (const float *)nullptr, Bc, grouped, lw.mlp_norm_g, d, w.Xb, lo_x, w.ss, m->Rmax);
        else
        LAUNCH(m, "resid_norm", 0, resid_norm_kernel, dim3(Bc, 1, branch_blocks(grouped)), norm_threads(d), 0, w.S, w.P, nsp, sstride, matched ? 3 : 1,
               matched ? lw.gate_a : (const float *)nullptr, Bc,
               grouped, lw.mlp_norm_g, c.rms_eps, d, 1, 1, 0, w.Xb, lo_x, moe && !m->moe_tc ? w.X : (float *)nullptr);
        if (!moe) {
            int F = c.d_ff;
            TcCall gu{};
            gu.W[0] = &mp.wg; gu.n_out[0] = F; gu.rows[0] = R;
            gu.W[1] = &mp.wu; gu.n_out[1] = F; gu.rows[1] = R;
            gu.nseg = 2; gu.X = &m->map_Xb; gu.K = d; gu.R = R; gu.P = w.P; gu.P_floats = w.P_floats; gu.parts = m->act_parts; gu.lo_row0 = m->Rmax; gu.tag = "gemm_gateup";
            if ((st = run_gemm_tc(m, gu, n_tile, &nsp, &sstride)) != DBT_OK) return st;
            dim3 sg(Bc, (F + 255) / 256, branch_blocks(grouped));
            LAUNCH(m, "swiglu_couple", 0, swiglu_couple_kernel, sg, 256, 0, w.P, nsp, sstride, F, Bc, grouped, lw.coup_b,
                   w.Hb, m->act_parts == 2 ? (size_t)m->Rmax * F : (size_t)0, (const float *)nullptr, 0, 0, d, c.rms_eps);
            TcCall dn{};
            dn.W[0] = &mp.wd; dn.n_out[0] = d; dn.rows[0] = R; dn.nseg = 1; dn.X = &m->map_Hb; dn.K = F; dn.R = R;
            dn.P = w.P; dn.P_floats = w.P_floats; dn.parts = m->act_parts; dn.lo_row0 = m->Rmax; dn.tag = "gemm_down";
            if ((st = run_gemm_tc(m, dn, n_tile, &nsp, &sstride)) != DBT_OK) return st;
            mode = 2;
        } else {
            st = m->moe_tc ? run_moe_tc(m, l, rm, grouped, record_experts, mwide,
                                        l + 1 < c.n_layers ? m->layers[l + 1].attn_norm_g : nullptr)
                           : run_moe<WT>(m, l, rm, grouped, record_experts);
            if (st != DBT_OK) return st;
            mode = 0;
        }
    }
    *pending_mode = mode;
    *pending_split = nsp;
    *pending_stride = sstride;
    return DBT_OK;
}

// Fold the pending MLP output, final norm, shared output matrix on tensor cores -> Z.
dbt_status run_head_tc(dbt_model *m, int Bc_src, int grouped, int n_rows_out, int src_mul, int src_add, int n_tile,
                       int mode, int nsp, size_t sstride) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    LAUNCH(m, "resid_norm", 0, resid_norm_kernel, dim3(n_rows_out, 1, branch_blocks(grouped)), norm_threads(c.d_model), 0, w.S, w.P, nsp, sstride, mode,
           m->layers[c.n_layers - 1].coup_c, Bc_src, grouped, m->w.final_norm_g, c.rms_eps, c.d_model, c.final_norm,
           src_mul, src_add, w.Xb, m->act_parts == 2 ? (size_t)m->Rmax * c.d_model : (size_t)0, (float *)nullptr);
    int R = npaths(grouped) * n_rows_out;
    TcCall lm{};
    lm.W[0] = &m->map_lm; lm.n_out[0] = c.vocab; lm.rows[0] = R; lm.nseg = 1; lm.X = &m->map_Xb; lm.K = c.d_model;
    lm.R = R; lm.P = w.Z; lm.P_floats = (size_t)R * c.vocab;  // exactly one split: Z is the output itself
    lm.parts = m->act_parts; lm.lo_row0 = m->Rmax; lm.tag = "gemm_lm_head";
    int one = 0;
    return run_gemm_tc(m, lm, n_tile, &one, nullptr);
}

dbt_status step_tc(dbt_model *m, const int32_t *tokens_dev, int B, int grouped, int32_t *next_dev, float *z1_dev,
                   float *z2_dev, float *alpha_dev) {
    typedef __nv_bfloat16 WT;
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    RowMap rm{B, 1};
    int R = npaths(grouped) * B;
    int n_tile = pad_rows(paths_of(c) * B);  // the same instruction shape in both modes
    dbt_status st;
    if (m->att_fast && (st = run_attention_plan(m, rm)) != DBT_OK) return st;
    LAUNCH(m, "embed", 0, embed_norm_kernel<WT>, R, 256, 0, tokens_dev, m->tok_stride, m->tok_p0, rm, (const WT *)m->w.embed_primary,
           (const WT *)m->w.embed_branch, m->w.embed_norm_g, c.rms_eps, c.d_model, c.vocab, w.S, w.status);
    int mode, nsp;
    size_t sstride;
    st = run_layers_tc(m, rm, grouped, n_tile, true, &mode, &nsp, &sstride);
    m->att_planned = false;
    if (st != DBT_OK) return st;
    if ((st = run_head_tc(m, B, grouped, B, 1, 0, n_tile, mode, nsp, sstride)) != DBT_OK) return st;
    // the readout also bumps the sequence lengths: nothing after it in the step reads them
    if ((st = run_readout(m, B, grouped, next_dev, alpha_dev)) != DBT_OK) return st;
    size_t zb = sizeof(float) * (size_t)B * c.vocab;
    if (z1_dev) CUDA_TRY(m, cudaMemcpyAsync(z1_dev, w.Z, zb, cudaMemcpyDeviceToDevice, m->stream));
    if (z2_dev && grouped)  // the branches' logits, branch-major [K-1][B][V]
        CUDA_TRY(m, cudaMemcpyAsync(z2_dev, w.Z + (size_t)B * c.vocab, zb * (npaths(grouped) - 1), cudaMemcpyDeviceToDevice, m->stream));
    for (int b = 0; b < B; b++) m->len_host[b] += 1;
    m->pending_union = c.n_experts > 0;
    return DBT_OK;
}

dbt_status prefill_tc(dbt_model *m, const int32_t *tokens_dev, int B, int n, float *last_logits) {
    typedef __nv_bfloat16 WT;
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    // chunks of up to Rmax rows where every kernel of the chain takes more than one row tile (the tensor-core MoE
    // chain with the norm factor behind the GEMMs); 256 rows otherwise
    const bool big = c.n_experts > 0 && m->moe_tc && m->moe_wide && m->att_fast;
    int cn_max = (big ? m->Rmax : (m->Rmax < 256 ? m->Rmax : 256)) / B;
    if (cn_max < 1) cn_max = 1;
    dbt_status st;
    for (int p0 = 0; p0 < n; p0 += cn_max) {
        int cn = n - p0 < cn_max ? n - p0 : cn_max;
        RowMap rm{B, cn};
        int R = B * cn, n_tile = pad_rows(R);
        LAUNCH(m, "embed", 0, embed_norm_kernel<WT>, R, 256, 0, tokens_dev, m->tok_stride > 1 ? m->tok_stride : n, p0, rm, (const WT *)m->w.embed_primary,
               (const WT *)m->w.embed_branch, m->w.embed_norm_g, c.rms_eps, c.d_model, c.vocab, w.S, w.status);
        int mode, nsp;
        size_t sstride;
        if ((st = run_layers_tc(m, rm, 0, n_tile, false, &mode, &nsp, &sstride)) != DBT_OK) return st;
        bool last = p0 + cn >= n;
        if (last && last_logits) {
            if ((st = run_head_tc(m, R, 0, B, cn, cn - 1, pad_rows(B), mode, nsp, sstride)) != DBT_OK) return st;
            CUDA_TRY(m, cudaMemcpyAsync(last_logits, w.Z, sizeof(float) * (size_t)B * c.vocab, cudaMemcpyDeviceToDevice,
                                        m->stream));
        }
        LAUNCH(m, "advance_len", 0, advance_len_kernel, (B + 127) / 128, 128, 0, w.seq_len, B, cn);
    }
    for (int b = 0; b < B; b++) m->len_host[b] += n;
    return DBT_OK;
}

// ---- dense bf16 path with the RMSNorm factor applied after the GEMM ---------------------------
// No kernel of this chain reduces over a whole row: the residual kernel is column-parallel and
// leaves per-block shares of sum(S^2); the kernels after the Q|K|V and gate|up GEMMs (and the
// output-matrix GEMM's own epilogue) multiply by 1/rms.  9 kernels per layer.

int wide_ss_tiles(const dbt_model *m) { return (m->cfg.d_model + 255) / 256; }

dbt_status run_layers_wide(dbt_model *m, const RowMap &rm, int grouped, int n_tile) {
    typedef __nv_bfloat16 WT;
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int Bc = rm.B * rm.cn, R = npaths(grouped) * Bc;
    int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim, F = c.d_ff;
    size_t pool_layer_elems = (size_t)2 * c.num_pages * c.n_kv_heads * c.page_size * c.head_dim;
    size_t lo_x = m->act_parts == 2 ? (size_t)m->Rmax * d : 0, lo_h = m->act_parts == 2 ? (size_t)m->Rmax * F : 0;
    int ss_tiles = wide_ss_tiles(m), ss_ld = m->Rmax;
    // prompt chunks of more than one row tile: the kernels between the GEMMs stream tens of MB and take
    // their vector form (four elements per thread)
    const bool rows_form = !grouped && rm.cn > 1 && Bc > 256 && d % 4 == 0 && F % 4 == 0 && c.head_dim % 8 == 0 && ((size_t)m->Rmax * d) % 4 == 0;
    double kv_bytes = 0;
    for (int b = 0; b < rm.B; b++)
        for (int j = 0; j < rm.cn; j++) kv_bytes += (double)(m->len_host[b] + j + 1) * 2 * kvd * sizeof(WT);
    dbt_status st;
    int nsp = 1;
    size_t sstride = 0;
    auto call = [&](const char *tag, const CUtensorMap *X, int K) {
        TcCall t{};
        t.X = X; t.K = K; t.R = R; t.P = w.P; t.P_floats = w.P_floats; t.tag = tag;
        t.parts = m->act_parts; t.lo_row0 = m->Rmax;
        return t;
    };
    for (int l = 0; l < c.n_layers; l++) {
        const dbt_layer_weights &lw = m->layers[l];
        const LayerMaps &mp = m->maps[l];
        WT *kpool = reinterpret_cast<WT *>(m->kv_pool) + (size_t)l * pool_layer_elems;
        WT *vpool = kpool + pool_layer_elems / 2;
        TcCall qkv = call("gemm_qkv", &m->map_Xb, d);
        qkv.W[0] = &mp.wq; qkv.n_out[0] = qd; qkv.rows[0] = R;
        qkv.W[1] = &mp.wk; qkv.n_out[1] = kvd; qkv.rows[1] = Bc;
        qkv.W[2] = &mp.wv; qkv.n_out[2] = kvd; qkv.rows[2] = Bc;
        qkv.nseg = 3;
        if ((st = run_gemm_tc(m, qkv, n_tile, &nsp, &sstride)) != DBT_OK) return st;
        const bool fuse = m->fuse_qkv && rm.cn == 1;
        QkvFuse qf{w.P, nsp, sstride, w.ss, ss_tiles, ss_ld, lw.coup_a};
        if (rows_form)
            LAUNCH(m, "qkv_epilogue", 0, qkv_rows_kernel, dim3(Bc, ((c.n_q_heads + c.n_kv_heads) * (c.head_dim / 8) + 255) / 256), 256, 0,
                   w.P, nsp, sstride, w.Q, rm, c.n_q_heads, c.n_kv_heads, c.head_dim, w.rope, w.seq_len, w.page_table,
                   m->pages_per_seq_max, c.num_pages, c.page_size, kpool, vpool, w.status, (const float *)w.ss, ss_tiles, ss_ld, d,
                   c.rms_eps);
        else if (!fuse)
            LAUNCH(m, "qkv_epilogue", 0, qkv_epilogue_kernel<WT>, dim3(Bc, c.n_q_heads + c.n_kv_heads, branch_blocks(grouped)), 64, 0, w.P, nsp, sstride,
                   w.Q, rm, grouped, c.n_q_heads, c.n_kv_heads, c.head_dim, lw.coup_a, w.rope, w.seq_len, w.page_table,
                   m->pages_per_seq_max, c.num_pages, c.page_size, kpool, vpool, w.status, (const float *)w.ss, ss_tiles, ss_ld, d,
                   c.rms_eps);
        st = c.head_dim == 128 ? run_attention_mma<128>(m, rm, grouped, l, kv_bytes, fuse ? &qf : nullptr, true, m->att_planned)
                               : run_attention_mma<64>(m, rm, grouped, l, kv_bytes, fuse ? &qf : nullptr, true, m->att_planned);
        if (st != DBT_OK) return st;
        TcCall op = call("gemm_o", &m->map_Ob, qd);
        op.W[0] = &mp.wo; op.n_out[0] = d; op.rows[0] = R; op.nseg = 1;
        {
            if ((st = run_gemm_tc(m, op, n_tile, &nsp, &sstride)) != DBT_OK) return st;
            if (rows_form)
                LAUNCH(m, "resid_wide", 0, resid_rows_kernel, dim3((Bc + 3) / 4, ss_tiles), 256, 0, w.S, w.P, nsp, sstride, lw.mlp_norm_g, Bc, d,
                       w.Xb, lo_x, w.ss, ss_ld);
            else
            LAUNCH_BR(m, grouped, "resid_wide", 0, resid_wide_kernel, dim3(Bc, ss_tiles, branch_blocks(grouped)), 256, 0, w.S, w.P, nsp, sstride, 1,
                   (const float *)nullptr, Bc, grouped, lw.mlp_norm_g, d, w.Xb, lo_x, w.ss, ss_ld);
        }
        TcCall gu = call("gemm_gateup", &m->map_Xb, d);
        gu.W[0] = &mp.wg; gu.n_out[0] = F; gu.rows[0] = R;
        gu.W[1] = &mp.wu; gu.n_out[1] = F; gu.rows[1] = R;
        gu.nseg = 2;
        {
            bool gu_done = false;
            GuEpi ge{};
            if (rows_form) {
                ge.Hb = w.Hb; ge.lo_off = lo_h; ge.ss = w.ss; ge.ss_tiles = ss_tiles; ge.ss_ld = ss_ld; ge.d_norm = d; ge.F = F;
                ge.eps = c.rms_eps;
                gu.gu = &ge;
                gu.gu_fused = &gu_done;
            }
            if ((st = run_gemm_tc(m, gu, n_tile, &nsp, &sstride)) != DBT_OK) return st;
            if (gu_done) {
            } else if (rows_form)
                LAUNCH(m, "swiglu_couple", 0, swiglu_rows_kernel, dim3(Bc, (F + 1023) / 1024), 256, 0, w.P, nsp, sstride, F, w.Hb, lo_h,
                       (const float *)w.ss, ss_tiles, ss_ld, d, c.rms_eps);
            else
            LAUNCH(m, "swiglu_couple", 0, swiglu_couple_kernel, dim3(Bc, (F + 255) / 256, branch_blocks(grouped)), 256, 0, w.P, nsp, sstride, F, Bc,
                   grouped, lw.coup_b, w.Hb, lo_h, (const float *)w.ss, ss_tiles, ss_ld, d, c.rms_eps);
        }
        TcCall dn = call("gemm_down", &m->map_Hb, F);
        dn.W[0] = &mp.wd; dn.n_out[0] = d; dn.rows[0] = R; dn.nseg = 1;
        const float *g_next = l + 1 < c.n_layers ? m->layers[l + 1].attn_norm_g
                                                 : (c.final_norm ? m->w.final_norm_g : (const float *)nullptr);
        {
            if ((st = run_gemm_tc(m, dn, n_tile, &nsp, &sstride)) != DBT_OK) return st;
            if (rows_form)
                LAUNCH(m, "resid_wide", 0, resid_rows_kernel, dim3((Bc + 3) / 4, ss_tiles), 256, 0, w.S, w.P, nsp, sstride, g_next, Bc, d, w.Xb,
                       lo_x, w.ss, ss_ld);
            else
            LAUNCH_BR(m, grouped, "resid_wide", 0, resid_wide_kernel, dim3(Bc, ss_tiles, branch_blocks(grouped)), 256, 0, w.S, w.P, nsp, sstride, 2, lw.coup_c, Bc,
                   grouped, g_next, d, w.Xb, lo_x, w.ss, ss_ld);
        }
    }
    return DBT_OK;
}

dbt_status run_head_wide(dbt_model *m, const RowMap &rm, int grouped, int n_tile) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int R = npaths(grouped) * rm.B * rm.cn;
    TcCall lm{};
    lm.W[0] = &m->map_lm; lm.n_out[0] = c.vocab; lm.rows[0] = R; lm.nseg = 1; lm.X = &m->map_Xb; lm.K = c.d_model;
    lm.R = R; lm.P = w.Z; lm.P_floats = (size_t)R * c.vocab; lm.tag = "gemm_lm_head";
    lm.parts = m->act_parts; lm.lo_row0 = m->Rmax;
    LmEpi e{};
    e.Z = w.Z;
    e.ss_in = w.ss;
    e.ss_tiles = wide_ss_tiles(m);
    e.ss_ld = m->Rmax;
    e.d_norm = c.d_model;
    e.use_scale = c.final_norm;
    e.eps = c.rms_eps;
    return run_gemm_tc(m, lm, n_tile, nullptr, nullptr, 0, e);
}

template <typename WT>
dbt_status run_embed_wide(dbt_model *m, const int32_t *tokens_dev, int n, int p0, const RowMap &rm, int R, int n_tile) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    LAUNCH(m, "embed", 0, embed_fused_kernel<WT>, R, 256, 0, tokens_dev, n, p0, rm, (const WT *)m->w.embed_primary,
           (const WT *)m->w.embed_branch, m->w.embed_norm_g, c.rms_eps, c.d_model, c.vocab, w.S,
           m->layers[0].attn_norm_g, w.Xb, m->act_parts == 2 ? (size_t)m->Rmax * c.d_model : (size_t)0, w.ss, m->Rmax,
           wide_ss_tiles(m), w.status);
    return DBT_OK;
}

dbt_status step_wide(dbt_model *m, const int32_t *tokens_dev, int B, int grouped, int32_t *next_dev, float *z1_dev,
                     float *z2_dev, float *alpha_dev) {
    typedef __nv_bfloat16 WT;
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    RowMap rm{B, 1};
    int R = npaths(grouped) * B, n_tile = pad_rows(paths_of(c) * B);
    dbt_status st;
    if ((st = run_attention_plan(m, rm)) != DBT_OK) return st;
    if ((st = run_embed_wide<WT>(m, tokens_dev, m->tok_stride, m->tok_p0, rm, R, n_tile)) != DBT_OK) return st;
    st = run_layers_wide(m, rm, grouped, n_tile);
    m->att_planned = false;
    if (st != DBT_OK) return st;
    if ((st = run_head_wide(m, rm, grouped, n_tile)) != DBT_OK) return st;
    // the readout also bumps the sequence lengths: nothing after it in the step reads them
    if ((st = run_readout(m, B, grouped, next_dev, alpha_dev)) != DBT_OK) return st;
    size_t zb = sizeof(float) * (size_t)B * c.vocab;
    if (z1_dev) CUDA_TRY(m, cudaMemcpyAsync(z1_dev, w.Z, zb, cudaMemcpyDeviceToDevice, m->stream));
    if (z2_dev && grouped)  // the branches' logits, branch-major [K-1][B][V]
        CUDA_TRY(m, cudaMemcpyAsync(z2_dev, w.Z + (size_t)B * c.vocab, zb * (npaths(grouped) - 1), cudaMemcpyDeviceToDevice, m->stream));
    for (int b = 0; b < B; b++) m->len_host[b] += 1;
    return DBT_OK;
}

dbt_status prefill_wide(dbt_model *m, const int32_t *tokens_dev, int B, int n, float *last_logits) {
    typedef __nv_bfloat16 WT;
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int cn_max = m->Rmax / B;  // a chunk of up to Rmax rows: GEMMs over several row tiles, packed causal attention
    if (cn_max < 1) cn_max = 1;
    // when logits are wanted the last position runs as its own chunk, so that the rows of the
    // output-matrix GEMM are exactly the B last positions
    int n_bulk = last_logits ? n - 1 : n;
    dbt_status st;
    for (int p0 = 0; p0 < n;) {
        int cn = p0 < n_bulk ? (n_bulk - p0 < cn_max ? n_bulk - p0 : cn_max) : 1;
        RowMap rm{B, cn};
        int R = B * cn, n_tile = pad_rows(R < 256 ? R : 256);
        if ((st = run_embed_wide<WT>(m, tokens_dev, m->tok_stride > 1 ? m->tok_stride : n, p0, rm, R, n_tile)) != DBT_OK) return st;
        if ((st = run_layers_wide(m, rm, 0, n_tile)) != DBT_OK) return st;
        if (last_logits && p0 + cn >= n) {
            if ((st = run_head_wide(m, rm, 0, n_tile)) != DBT_OK) return st;
            CUDA_TRY(m, cudaMemcpyAsync(last_logits, w.Z, sizeof(float) * (size_t)B * c.vocab, cudaMemcpyDeviceToDevice,
                                        m->stream));
        }
        LAUNCH(m, "advance_len", 0, advance_len_kernel, (B + 127) / 128, 128, 0, w.seq_len, B, cn);
        for (int b = 0; b < B; b++) m->len_host[b] += cn;
        p0 += cn;
    }
    return DBT_OK;
}


template <int N_TILE>
bool allow_smem() {
    return cudaFuncSetAttribute(gemm_tc_kernel<N_TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                TcCfg<N_TILE>::kSmemBytes) == cudaSuccess;
}
// The attribute is per device: set it on every call for the device that is current (it is cheap).
bool allow_smem_all() {
    return allow_smem<16>() && allow_smem<32>() && allow_smem<64>() && allow_smem<128>() && allow_smem<256>() &&
           cudaFuncSetAttribute(gemm_tc_kernel<256, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<256, 2>::kSmemBytes) ==
               cudaSuccess &&
           cudaFuncSetAttribute(gemm_tc_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<64, 2>::kSmemBytes) ==
               cudaSuccess;
}

// Build the TMA descriptors of a bf16 model.  Returns false when the path cannot be used.
bool setup_tc(dbt_model *m) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    const char *force = getenv("DBT_FORCE_PATH");
    if (force && strcmp(force, "simt") == 0) return false;
    if (c.weight_dtype != DBT_DTYPE_BF16) return false;
    if (!allow_smem_all()) return false;
    int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
    bool moe = c.n_experts > 0;
    int F = moe ? 0 : c.d_ff;
    bool ok = true;
    m->maps.resize(c.n_layers);
    for (int l = 0; l < c.n_layers && ok; l++) {
        const dbt_layer_weights &lw = m->layers[l];
        LayerMaps &mp = m->maps[l];
        ok = ok && make_bf16_map(&mp.wq, lw.wq, qd, d, kTcM) && make_bf16_map(&mp.wk, lw.wk, kvd, d, kTcM) &&
             make_bf16_map(&mp.wv, lw.wv, kvd, d, kTcM) && make_bf16_map(&mp.wo, lw.wo, d, qd, kTcM);
        if (!moe)
            ok = ok && make_bf16_map(&mp.wg, lw.w_gate, F, d, kTcM) && make_bf16_map(&mp.wu, lw.w_up, F, d, kTcM) &&
                 make_bf16_map(&mp.wd, lw.w_down, d, F, kTcM);
    }
    m->moe_tc = false;
    if (moe && ok) {
        int E = c.n_experts, Fe = c.d_expert, Fs = c.n_shared_experts * Fe, Rk = m->Rmax * kmax_of(c);
        const char *mo = getenv("DBT_MOE");
        bool want = !(mo && strcmp(mo, "simt") == 0);
        bool mok = want;
        for (int l = 0; l < c.n_layers && mok; l++) {
            const dbt_layer_weights &lw = m->layers[l];
            LayerMaps &mp = m->maps[l];
            mok = make_bf16_map(&mp.eg, lw.exp_gate, (uint64_t)E * Fe, d, kTcM) &&
                  make_bf16_map(&mp.eu, lw.exp_up, (uint64_t)E * Fe, d, kTcM) &&
                  make_bf16_map(&mp.ed, lw.exp_down, (uint64_t)E * d, Fe, kTcM) &&
                  make_bf16_map(&mp.rt, lw.router, E, d, kTcM);
            if (mok && Fs > 0)
                mok = make_bf16_map(&mp.wg, lw.sh_gate, Fs, d, kTcM) && make_bf16_map(&mp.wu, lw.sh_up, Fs, d, kTcM) &&
                      make_bf16_map(&mp.wd, lw.sh_down, d, Fs, kTcM);
        }
        mok = mok && make_bf16_map(&m->map_Xs, w.Xs, 2 * (uint64_t)Rk, d, 16) &&
              make_bf16_map(&m->map_Hs, w.Hs, 2 * (uint64_t)Rk, Fe, 16);
        if (mok && Fs > 0) mok = make_bf16_map(&m->map_Hb, w.Hb, 2 * m->Rmax, Fs, 16);
        // (a weight tile that runs past its expert's last row only computes features that the
        // epilogue never stores)
        m->moe_tc = mok;
    }
    ok = ok && make_bf16_map(&m->map_lm, m->w.lm_head, c.vocab, d, kTcM);
    ok = ok && make_bf16_map(&m->map_Xb, w.Xb, 2 * m->Rmax, d, 16) && make_bf16_map(&m->map_Ob, w.Ob, 2 * m->Rmax, qd, 16);
    if (!moe) ok = ok && make_bf16_map(&m->map_Hb, w.Hb, 2 * m->Rmax, F, 16);
    m->act_base[&m->map_Xb] = {w.Xb};
    m->act_base[&m->map_Ob] = {w.Ob};
    m->act_base[&m->map_Hb] = {w.Hb};
    if (m->moe_tc) {
        m->act_base[&m->map_Xs] = {w.Xs};
        m->act_base[&m->map_Hs] = {w.Hs};
    }
    const char *fa = getenv("DBT_ATTN");
    m->att_fast = ok && !(fa && strcmp(fa, "simt") == 0) &&
                  make_kv_page_map(&m->map_kv, m->kv_pool, (uint64_t)c.n_layers * 2 * c.num_pages * c.n_kv_heads * c.page_size,
                                   (uint64_t)c.num_pages * c.n_kv_heads * c.page_size, c.head_dim) &&
                  cudaFuncSetAttribute(attn_prompt_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       PromptAttCfg<128>::kSmemBytes) == cudaSuccess &&
                  cudaFuncSetAttribute(attn_prompt_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       PromptAttCfg<64>::kSmemBytes) == cudaSuccess &&
                  cudaFuncSetAttribute(attn_mma_kernel<128, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       AttCfg<128, true>::kSmemBytes) == cudaSuccess &&
                  cudaFuncSetAttribute(attn_mma_kernel<64, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       AttCfg<64, true>::kSmemBytes) == cudaSuccess &&
                  cudaFuncSetAttribute(attn_mma_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       AttCfg<128>::kSmemBytes) == cudaSuccess &&
                  cudaFuncSetAttribute(attn_mma_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       AttCfg<128>::kSmemBytes) == cudaSuccess &&
                  cudaFuncSetAttribute(attn_mma_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       AttCfg<64>::kSmemBytes) == cudaSuccess &&
                  cudaFuncSetAttribute(attn_mma_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       AttCfg<64>::kSmemBytes) == cudaSuccess;
    // Default chain of a dense bf16 model: the RMSNorm factor is applied after the GEMM, so no kernel
    // reduces over a whole row.
    m->wide = ok && m->att_fast && !moe;
    m->act_parts = 2;
    return ok;
}

template <typename WT>
dbt_status step_impl(dbt_model *m, const int32_t *tokens_dev, int B, int grouped, int32_t *next_dev, float *z1_dev,
                     float *z2_dev, float *alpha_dev) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    RowMap rm{B, 1};
    int R = npaths(grouped) * B;
    dbt_status st;
    LAUNCH(m, "embed", 0, embed_norm_kernel<WT>, R, 256, 0, tokens_dev, m->tok_stride, m->tok_p0, rm, (const WT *)m->w.embed_primary,
           (const WT *)m->w.embed_branch, m->w.embed_norm_g, c.rms_eps, c.d_model, c.vocab, w.S, w.status);
    if ((st = run_layers<WT>(m, rm, grouped, true)) != DBT_OK) return st;
    if ((st = run_head<WT>(m, R, 1, 0)) != DBT_OK) return st;
    // the readout also bumps the sequence lengths: nothing after it in the step reads them
    if ((st = run_readout(m, B, grouped, next_dev, alpha_dev)) != DBT_OK) return st;
    size_t zb = sizeof(float) * (size_t)B * c.vocab;
    if (z1_dev) CUDA_TRY(m, cudaMemcpyAsync(z1_dev, w.Z, zb, cudaMemcpyDeviceToDevice, m->stream));
    if (z2_dev && grouped)  // the branches' logits, branch-major [K-1][B][V]
        CUDA_TRY(m, cudaMemcpyAsync(z2_dev, w.Z + (size_t)B * c.vocab, zb * (npaths(grouped) - 1), cudaMemcpyDeviceToDevice, m->stream));
    for (int b = 0; b < B; b++) m->len_host[b] += 1;
    m->pending_union = c.n_experts > 0;
    return DBT_OK;
}

template <typename WT>
dbt_status prefill_impl(dbt_model *m, const int32_t *tokens_dev, int B, int n, float *last_logits) {
    const dbt_config &c = m->cfg;
    const Workspace &w = m->ws;
    int cn_max = m->Rmax / B;
    if (cn_max < 1) cn_max = 1;
    dbt_status st;
    for (int p0 = 0; p0 < n; p0 += cn_max) {
        int cn = n - p0 < cn_max ? n - p0 : cn_max;
        RowMap rm{B, cn};
        int R = B * cn;
        LAUNCH(m, "embed", 0, embed_norm_kernel<WT>, R, 256, 0, tokens_dev, m->tok_stride > 1 ? m->tok_stride : n, p0, rm, (const WT *)m->w.embed_primary,
               (const WT *)m->w.embed_branch, m->w.embed_norm_g, c.rms_eps, c.d_model, c.vocab, w.S, w.status);
        if ((st = run_layers<WT>(m, rm, 0, false)) != DBT_OK) return st;
        bool last = p0 + cn >= n;
        if (last && last_logits) {
            if ((st = run_head<WT>(m, B, cn, cn - 1)) != DBT_OK) return st;
            CUDA_TRY(m, cudaMemcpyAsync(last_logits, w.Z, sizeof(float) * (size_t)B * c.vocab,
                                        cudaMemcpyDeviceToDevice, m->stream));
        }
        LAUNCH(m, "advance_len", 0, advance_len_kernel, (B + 127) / 128, 128, 0, w.seq_len, B, cn);
    }
    for (int b = 0; b < B; b++) m->len_host[b] += n;
    return DBT_OK;
}

dbt_status check_step_args(dbt_model *m, const int32_t *tokens, int B, int n) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (!tokens) return fail(m, DBT_ERR_INVALID_ARG, "tokens pointer is NULL");
    if (B <= 0 || n <= 0) return fail(m, DBT_ERR_INVALID_ARG, "B and n must be positive");
    if (B > m->cfg.max_batch) return fail(m, DBT_ERR_CAPACITY, "B=%d exceeds max_batch=%d", B, m->cfg.max_batch);
    int cap = m->pages_per_seq * m->cfg.page_size;
    if (cap > m->cfg.max_seq) cap = m->cfg.max_seq;
    for (int b = 0; b < B; b++)
        if (m->len_host[b] + n > cap)
            return fail(m, DBT_ERR_CAPACITY, "sequence %d: %d + %d positions exceed capacity %d", b, m->len_host[b], n,
                        cap);
    return DBT_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------

extern "C" {

const char *dbt_version(void) { return "dbt-b200 0.1 (sm_100a)"; }

const char *dbt_last_error(const dbt_model *m) { return m ? m->err.c_str() : g_create_error.c_str(); }

dbt_status dbt_query_sizes(const dbt_config *cfg, size_t *kv_bytes, size_t *workspace_bytes) {
    dbt_status st;
    const char *why = check_config(cfg, &st);
    if (why) return fail(nullptr, st, "%s", why);
    if (kv_bytes)
        *kv_bytes = (size_t)cfg->n_layers * 2 * cfg->num_pages * cfg->n_kv_heads * cfg->page_size * cfg->head_dim *
                    elem_bytes(*cfg);
    if (workspace_bytes) *workspace_bytes = carve(*cfg, nullptr, nullptr, nullptr, nullptr);
    return DBT_OK;
}

dbt_status dbt_create(const dbt_config *cfg, const dbt_weights *w, void *kv_pool_dev, void *workspace_dev,
                      void *cuda_stream, dbt_model **out) {
    if (out) *out = nullptr;
    dbt_status st;
    const char *why = check_config(cfg, &st);
    if (why) return fail(nullptr, st, "%s", why);
    if (!w || !kv_pool_dev || !workspace_dev || !out || !w->layers)
        return fail(nullptr, DBT_ERR_INVALID_ARG, "NULL pointer argument");
    if (((uintptr_t)kv_pool_dev | (uintptr_t)workspace_dev) & 255)
        return fail(nullptr, DBT_ERR_INVALID_ARG, "kv pool and workspace must be 256-byte aligned");
    bool moe = cfg->n_experts > 0;
    if (!w->embed_primary || !w->embed_branch || !w->embed_norm_g || !w->lm_head || (cfg->final_norm && !w->final_norm_g))
        return fail(nullptr, DBT_ERR_INVALID_ARG, "NULL top-level weight pointer");
    for (int l = 0; l < cfg->n_layers; l++) {
        const dbt_layer_weights &lw = w->layers[l];
        bool ok = lw.attn_norm_g && lw.wq && lw.wk && lw.wv && lw.wo && lw.coup_a && lw.mlp_norm_g && lw.coup_c;
        if (cfg->compute_matched) ok = ok && lw.gate_a && lw.gate_g;
        if (moe) {
            ok = ok && lw.router && lw.exp_gate && lw.exp_up && lw.exp_down;
            if (cfg->n_shared_experts > 0)
                ok = ok && lw.sh_gate && lw.sh_up && lw.sh_down && (!cfg->moe_b_coupling || lw.coup_b);
        } else {
            ok = ok && lw.w_gate && lw.w_up && lw.w_down && lw.coup_b;
        }
        if (!ok) return fail(nullptr, DBT_ERR_INVALID_ARG, "NULL weight pointer in layer %d", l);
    }
    dbt_model *m = new (std::nothrow) dbt_model();
    if (!m) return fail(nullptr, DBT_ERR_INVALID_ARG, "out of host memory");
    m->cfg = *cfg;
    m->w = *w;
    m->layers.assign(w->layers, w->layers + cfg->n_layers);
    m->w.layers = m->layers.data();
    m->stream = (cudaStream_t)cuda_stream;
    m->kv_pool = (char *)kv_pool_dev;
    m->ws_base = (char *)workspace_dev;
    m->ws_bytes = carve(*cfg, m->ws_base, &m->ws, &m->Rmax, &m->part_items);
    m->pages_per_seq_max = (cfg->max_seq + cfg->page_size - 1) / cfg->page_size;
    m->pages_per_seq = m->pages_per_seq_max;
    m->len_host.assign(cfg->max_batch, 0);
    m->launches = 0;
    m->pending_union = false;
    m->prof_on = false;
    {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        m->num_sms = sms > 0 && sms <= 148 ? sms : 148;  // the partial buffer is sized for 2 x 148 CTAs
    }
    m->tc = setup_tc(m);
    {
        const char *ef = getenv("DBT_EVICT_FIRST");
        m->evict_first = !(ef && strcmp(ef, "0") == 0);
        const char *fq = getenv("DBT_FUSE_QKV");
        m->fuse_qkv = m->att_fast && !(fq && strcmp(fq, "0") == 0);
        const char *mp = getenv("DBT_MOE_PERSIST");
        m->moe_persist = !mp ? -1 : strcmp(mp, "1") == 0 ? 1 : 0;
        const char *fs = getenv("DBT_MOE_FUSE_SWIGLU");
        m->moe_fuse_swiglu = !(fs && strcmp(fs, "0") == 0);
        const char *pf = getenv("DBT_PROMPT_FUSE_SWIGLU");
        m->prompt_fuse_swiglu = !(pf && strcmp(pf, "0") == 0);
        const char *pa = getenv("DBT_PROMPT_ATTN");
        m->prompt_attn_off = pa && strcmp(pa, "tile") == 0;
    }
    const char *ro = getenv("DBT_READOUT");
    m->readout_row = ro && strcmp(ro, "row") == 0;
    const char *pd = getenv("DBT_PDL");
    m->use_pdl = !(pd && strcmp(pd, "0") == 0);
    const char *po = getenv("DBT_PDL_OFF");
    m->pdl_off = po ? po : "";
    const char *gr = getenv("DBT_GRAPH");
    m->use_graph = !(gr && strcmp(gr, "0") == 0);
    m->cap_stream = nullptr;
    m->side_stream = nullptr;
    m->ev_fork = m->ev_join = nullptr;
    {
        const char *ov = getenv("DBT_MOE_OVERLAP");
        m->moe_overlap = m->moe_tc && cfg->n_shared_experts > 0 && !(ov && strcmp(ov, "0") == 0);
        const char *rt = getenv("DBT_MOE_ROWTILE");
        m->moe_row_tile = rt ? atoi(rt) : -1;
        if (m->moe_row_tile != 0 && m->moe_row_tile != 16 && m->moe_row_tile != 32 && m->moe_row_tile != 64) m->moe_row_tile = -1;
        m->moe_wide = m->moe_tc && m->act_parts == 2;
        if (m->moe_overlap &&
            (cudaStreamCreateWithFlags(&m->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
             cudaEventCreateWithFlags(&m->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
             cudaEventCreateWithFlags(&m->ev_join, cudaEventDisableTiming) != cudaSuccess)) {
            m->moe_overlap = false;  // one stream serves as well, only later
            cudaGetLastError();
        }
    }
    if (m->use_graph && cudaStreamCreateWithFlags(&m->cap_stream, cudaStreamNonBlocking) != cudaSuccess) {
        m->use_graph = false;
        cudaGetLastError();
    }

    // RoPE table in double: angle = t * base^(-2i/d_h), stored as (cos, sin) fp32 pairs.
    int half = cfg->head_dim / 2;
    std::vector<float2> tab((size_t)cfg->max_seq * half);
    std::vector<double> inv_freq(half);
    for (int i = 0; i < half; i++) inv_freq[i] = std::exp(-std::log((double)cfg->rope_base) * (2.0 * i) / cfg->head_dim);
    for (int t = 0; t < cfg->max_seq; t++)
        for (int i = 0; i < half; i++) {
            double ang = (double)t * inv_freq[i];
            tab[(size_t)t * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
        }
    // Default page table: sequence b owns a contiguous run of pages (clamped into the pool;
    // capacity checks use the pool size).
    std::vector<int32_t> pt((size_t)cfg->max_batch * m->pages_per_seq_max);
    for (int b = 0; b < cfg->max_batch; b++)
        for (int p = 0; p < m->pages_per_seq_max; p++) {
            long long id = (long long)b * m->pages_per_seq_max + p;
            pt[(size_t)b * m->pages_per_seq_max + p] = id < cfg->num_pages ? (int32_t)id : -1;
        }
    cudaError_t e = cudaMemcpyAsync(m->ws.rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, m->stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(m->ws.page_table, pt.data(), pt.size() * sizeof(int32_t), cudaMemcpyHostToDevice, m->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m->ws.seq_len, 0, sizeof(int32_t) * cfg->max_batch, m->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m->ws.status, 0, sizeof(int32_t) * 4, m->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m->ws.att_tickets, 0, sizeof(int32_t) * (size_t)att_rows_of(*cfg) * cfg->n_kv_heads, m->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m->ws.att_tickets2, 0, sizeof(int32_t) * (size_t)att_rows_of(*cfg) * cfg->n_kv_heads * kAttMaxGroups, m->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m->ws.ro_tickets, 0, sizeof(int32_t) * (size_t)cfg->max_batch, m->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(m->ws.gemm_tickets, 0, sizeof(int32_t) * 4096, m->stream);
    if (e == cudaSuccess && moe) {
        e = cudaMemsetAsync(m->ws.last_experts, 0xff, sizeof(int32_t) * (size_t)cfg->n_layers * paths_of(*cfg) * cfg->max_batch * kmax_of(*cfg), m->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(m->ws.union_cnt, 0, sizeof(int32_t) * cfg->n_layers, m->stream);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(m->stream);  // the host vectors go out of scope
    if (e != cudaSuccess) {
        fail(nullptr, DBT_ERR_CUDA, "dbt_create: %s", cudaGetErrorString(e));
        delete m;
        return DBT_ERR_CUDA;
    }
    if ((long long)cfg->max_batch * m->pages_per_seq_max > cfg->num_pages) {
        // the default table cannot give every sequence max_seq positions: shrink per-sequence capacity
        m->pages_per_seq = cfg->num_pages / cfg->max_batch;
        if (m->pages_per_seq < 1) {
            fail(nullptr, DBT_ERR_CAPACITY, "num_pages=%d cannot hold one page per sequence", cfg->num_pages);
            delete m;
            return DBT_ERR_CAPACITY;
        }
        std::vector<int32_t> pt2((size_t)cfg->max_batch * m->pages_per_seq_max, -1);
        for (int b = 0; b < cfg->max_batch; b++)
            for (int p = 0; p < m->pages_per_seq; p++) pt2[(size_t)b * m->pages_per_seq_max + p] = b * m->pages_per_seq + p;
        e = cudaMemcpy(m->ws.page_table, pt2.data(), pt2.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            fail(nullptr, DBT_ERR_CUDA, "dbt_create: %s", cudaGetErrorString(e));
            delete m;
            return DBT_ERR_CUDA;
        }
    }
    *out = m;
    return DBT_OK;
}

void dbt_destroy(dbt_model *m) {
    if (!m) return;
    for (auto &r : m->prof) {
        cudaEventDestroy(r.e0);
        cudaEventDestroy(r.e1);
    }
    for (auto e : m->prof_pool) cudaEventDestroy(e);
    for (auto &g : m->graphs) {
        cudaGraphExecDestroy(g.exec);
        cudaGraphDestroy(g.graph);
    }
    if (m->cap_stream) cudaStreamDestroy(m->cap_stream);
    if (m->side_stream) cudaStreamDestroy(m->side_stream);
    if (m->ev_fork) cudaEventDestroy(m->ev_fork);
    if (m->ev_join) cudaEventDestroy(m->ev_join);
    delete m;
}

dbt_status dbt_profile_begin(dbt_model *m) {
    if (!m) return DBT_ERR_INVALID_ARG;
    for (auto &r : m->prof) {
        m->prof_pool.push_back(r.e0);
        m->prof_pool.push_back(r.e1);
    }
    m->prof.clear();
    m->prof_on = true;
    return DBT_OK;
}

dbt_status dbt_profile_end(dbt_model *m, dbt_profile_entry *entries_host, int32_t max_entries, int32_t *n_entries) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (!entries_host || !n_entries || max_entries <= 0) return fail(m, DBT_ERR_INVALID_ARG, "bad profile buffer");
    m->prof_on = false;
    CUDA_TRY(m, cudaStreamSynchronize(m->stream));
    int n = 0;
    for (auto &r : m->prof) {
        float ms = 0.f;
        CUDA_TRY(m, cudaEventElapsedTime(&ms, r.e0, r.e1));
        int i = 0;
        while (i < n && strncmp(entries_host[i].name, r.tag, sizeof entries_host[i].name) != 0) i++;
        if (i == n) {
            if (n == max_entries) continue;
            memset(&entries_host[n], 0, sizeof entries_host[n]);
            strncpy(entries_host[n].name, r.tag, sizeof entries_host[n].name - 1);
            n++;
        }
        entries_host[i].launches += 1;
        entries_host[i].total_ms += ms;
        entries_host[i].bytes += r.bytes;
    }
    for (auto &r : m->prof) {
        m->prof_pool.push_back(r.e0);
        m->prof_pool.push_back(r.e1);
    }
    m->prof.clear();
    *n_entries = n;
    return DBT_OK;
}

dbt_status dbt_set_page_table(dbt_model *m, const int32_t *table_host, int32_t B, int32_t pages_per_seq) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (!table_host || B <= 0 || pages_per_seq <= 0) return fail(m, DBT_ERR_INVALID_ARG, "bad page-table argument");
    if (B > m->cfg.max_batch || pages_per_seq > m->pages_per_seq_max)
        return fail(m, DBT_ERR_CAPACITY, "page table [%d][%d] exceeds [%d][%d]", B, pages_per_seq, m->cfg.max_batch,
                    m->pages_per_seq_max);
    std::vector<char> seen(m->cfg.num_pages, 0);
    std::vector<int32_t> pt((size_t)m->cfg.max_batch * m->pages_per_seq_max, -1);
    for (int b = 0; b < B; b++)
        for (int p = 0; p < pages_per_seq; p++) {
            int32_t id = table_host[(size_t)b * pages_per_seq + p];
            if (id < 0 || id >= m->cfg.num_pages) return fail(m, DBT_ERR_INVALID_ARG, "page id %d out of range", id);
            if (seen[id]) return fail(m, DBT_ERR_INVALID_ARG, "page id %d appears twice", id);
            seen[id] = 1;
            pt[(size_t)b * m->pages_per_seq_max + p] = id;
        }
    CUDA_TRY(m, cudaStreamSynchronize(m->stream));
    CUDA_TRY(m, cudaMemcpy(m->ws.page_table, pt.data(), pt.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    m->pages_per_seq = pages_per_seq;
    return DBT_OK;
}

dbt_status dbt_reset(dbt_model *m) {
    if (!m) return DBT_ERR_INVALID_ARG;
    CUDA_TRY(m, cudaMemsetAsync(m->ws.seq_len, 0, sizeof(int32_t) * m->cfg.max_batch, m->stream));
    CUDA_TRY(m, cudaMemsetAsync(m->ws.status, 0, sizeof(int32_t) * 4, m->stream));
    CUDA_TRY(m, cudaMemsetAsync(m->ws.att_tickets, 0, sizeof(int32_t) * (size_t)att_rows_of(m->cfg) * m->cfg.n_kv_heads, m->stream));
    CUDA_TRY(m, cudaMemsetAsync(m->ws.att_tickets2, 0, sizeof(int32_t) * (size_t)att_rows_of(m->cfg) * m->cfg.n_kv_heads * kAttMaxGroups, m->stream));
    CUDA_TRY(m, cudaMemsetAsync(m->ws.gemm_tickets, 0, sizeof(int32_t) * 4096, m->stream));
    CUDA_TRY(m, cudaMemsetAsync(m->ws.ro_tickets, 0, sizeof(int32_t) * (size_t)m->cfg.max_batch, m->stream));
    std::fill(m->len_host.begin(), m->len_host.end(), 0);
    return DBT_OK;
}

dbt_status dbt_set_seq_lens(dbt_model *m, const int32_t *lens_host, int32_t B) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (!lens_host || B <= 0 || B > m->cfg.max_batch) return fail(m, DBT_ERR_INVALID_ARG, "bad argument");
    int cap = m->pages_per_seq * m->cfg.page_size;
    if (cap > m->cfg.max_seq) cap = m->cfg.max_seq;
    for (int b = 0; b < B; b++)
        if (lens_host[b] < 0 || lens_host[b] > cap) return fail(m, DBT_ERR_CAPACITY, "length %d out of range", lens_host[b]);
    CUDA_TRY(m, cudaStreamSynchronize(m->stream));
    CUDA_TRY(m, cudaMemcpy(m->ws.seq_len, lens_host, sizeof(int32_t) * B, cudaMemcpyHostToDevice));
    for (int b = 0; b < B; b++) m->len_host[b] = lens_host[b];
    return DBT_OK;
}

int32_t dbt_seq_len(const dbt_model *m, int32_t b) {
    if (!m || b < 0 || b >= m->cfg.max_batch) return -1;
    return m->len_host[b];
}

dbt_status dbt_prefill(dbt_model *m, const int32_t *tokens_dev, int32_t B, int32_t n, float *last_primary_logits_dev) {
    dbt_status st = check_step_args(m, tokens_dev, B, n);
    if (st != DBT_OK) return st;
    if (m->cfg.weight_dtype == DBT_DTYPE_F32) return prefill_impl<float>(m, tokens_dev, B, n, last_primary_logits_dev);
    if (m->wide) return prefill_wide(m, tokens_dev, B, n, last_primary_logits_dev);
    if (m->tc) return prefill_tc(m, tokens_dev, B, n, last_primary_logits_dev);
    return prefill_impl<__nv_bfloat16>(m, tokens_dev, B, n, last_primary_logits_dev);
}

static dbt_status step_direct(dbt_model *m, const int32_t *tokens_dev, int B, int grouped, int32_t *next_dev,
                              float *z1, float *z2, float *alpha) {
    if (m->cfg.weight_dtype == DBT_DTYPE_F32) return step_impl<float>(m, tokens_dev, B, grouped, next_dev, z1, z2, alpha);
    if (m->wide) return step_wide(m, tokens_dev, B, grouped, next_dev, z1, z2, alpha);
    if (m->tc) return step_tc(m, tokens_dev, B, grouped, next_dev, z1, z2, alpha);
    return step_impl<__nv_bfloat16>(m, tokens_dev, B, grouped, next_dev, z1, z2, alpha);
}

// Replay the step as a CUDA graph: every kernel reads the sequence lengths from device
// memory, so one capture per (batch, mode, buffer set) serves every later step.
static dbt_status step_graphed(dbt_model *m, const int32_t *tokens_dev, int B, int grouped, int32_t *next_dev,
                               float *z1, float *z2, float *alpha) {
    if (!m->use_graph || m->prof_on) return step_direct(m, tokens_dev, B, grouped, next_dev, z1, z2, alpha);
    const void *key[5] = {tokens_dev, next_dev, z1, z2, alpha};
    dbt_model::GraphEntry *hit = nullptr;
    for (auto &g : m->graphs)
        if (g.B == B && g.grouped == grouped && memcmp(g.ptr, key, sizeof key) == 0) hit = &g;
    if (!hit) {
        if (m->graphs.size() >= 64) {  // a caller that never reuses buffers: stop caching
            return step_direct(m, tokens_dev, B, grouped, next_dev, z1, z2, alpha);
        }
        std::vector<int32_t> len_save = m->len_host;
        int64_t l0 = m->launches;
        cudaStream_t user = m->stream;
        CUDA_TRY(m, cudaStreamBeginCapture(m->cap_stream, cudaStreamCaptureModeThreadLocal));
        m->stream = m->cap_stream;
        dbt_status st = step_direct(m, tokens_dev, B, grouped, next_dev, z1, z2, alpha);
        m->stream = user;
        cudaGraph_t graph = nullptr;
        cudaError_t e = cudaStreamEndCapture(m->cap_stream, &graph);
        int64_t captured = m->launches - l0;
        m->launches = l0;
        m->len_host = len_save;
        if (st != DBT_OK) {
            if (graph) cudaGraphDestroy(graph);
            return st;
        }
        if (e != cudaSuccess) return fail(m, DBT_ERR_CUDA, "graph capture: %s", cudaGetErrorString(e));
        cudaGraphExec_t exec = nullptr;
        e = cudaGraphInstantiate(&exec, graph, 0);
        if (e != cudaSuccess) {
            cudaGraphDestroy(graph);
            return fail(m, DBT_ERR_CUDA, "graph instantiate: %s", cudaGetErrorString(e));
        }
        dbt_model::GraphEntry g{};
        g.B = B;
        g.grouped = grouped;
        memcpy(g.ptr, key, sizeof key);
        g.graph = graph;
        g.exec = exec;
        g.launches = captured;
        m->graphs.push_back(g);
        hit = &m->graphs.back();
    }
    CUDA_TRY(m, cudaGraphLaunch(hit->exec, m->stream));
    m->launches += hit->launches;
    for (int b = 0; b < B; b++) m->len_host[b] += 1;
    m->pending_union = m->cfg.n_experts > 0;
    return DBT_OK;
}

dbt_status dbt_decode_step(dbt_model *m, const int32_t *tokens_dev, int32_t B, int32_t *next_tokens_dev,
                           float *logits_primary_dev, float *logits_branch_dev, float *alpha_dev) {
    dbt_status st = check_step_args(m, tokens_dev, B, 1);
    if (st != DBT_OK) return st;
    return step_graphed(m, tokens_dev, B, paths_of(m->cfg), next_tokens_dev, logits_primary_dev, logits_branch_dev, alpha_dev);
}

dbt_status dbt_prefill_boundary(dbt_model *m, const int32_t *tokens_dev, int32_t B, int32_t S, int32_t *next_tokens_dev,
                                float *logits_primary_dev, float *logits_branch_dev, float *alpha_dev) {
    dbt_status st = check_step_args(m, tokens_dev, B, S);
    if (st != DBT_OK) return st;
    if (S > 1) {
        // positions 1..S-1 of every row of tokens_dev [B][S]: the prompt-wide prefill walks rows of stride S
        m->tok_stride = S;
        st = m->cfg.weight_dtype == DBT_DTYPE_F32 ? prefill_impl<float>(m, tokens_dev, B, S - 1, nullptr)
             : m->wide                             ? prefill_wide(m, tokens_dev, B, S - 1, nullptr)
             : m->tc                               ? prefill_tc(m, tokens_dev, B, S - 1, nullptr)
                                                   : prefill_impl<__nv_bfloat16>(m, tokens_dev, B, S - 1, nullptr);
        m->tok_stride = 1;
        if (st != DBT_OK) return st;
    }
    // position S: the primary's step and the branch's boundary evaluation in one grouped pass (launched
    // directly: the token addressing differs from a decode step's, so the captured graphs do not apply)
    m->tok_stride = S;
    m->tok_p0 = S - 1;
    st = step_direct(m, tokens_dev, B, paths_of(m->cfg), next_tokens_dev, logits_primary_dev, logits_branch_dev, alpha_dev);
    m->tok_stride = 1;
    m->tok_p0 = 0;
    return st;
}

dbt_status dbt_decode_step_primary_only(dbt_model *m, const int32_t *tokens_dev, int32_t B, int32_t *next_tokens_dev,
                                        float *logits_primary_dev) {
    dbt_status st = check_step_args(m, tokens_dev, B, 1);
    if (st != DBT_OK) return st;
    return step_graphed(m, tokens_dev, B, 0, next_tokens_dev, logits_primary_dev, nullptr, nullptr);
}

static dbt_status step_host(dbt_model *m, const int32_t *tokens_host, int32_t B, int32_t *next_host, float *alpha_host,
                            int grouped) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (!tokens_host || !next_host) return fail(m, DBT_ERR_INVALID_ARG, "NULL host buffer");
    if (B <= 0 || B > m->cfg.max_batch) return fail(m, DBT_ERR_CAPACITY, "B=%d out of range", B);
    const Workspace &w = m->ws;
    CUDA_TRY(m, cudaMemcpyAsync(w.tokens_stage, tokens_host, sizeof(int32_t) * B, cudaMemcpyHostToDevice, m->stream));
    dbt_status st = grouped ? dbt_decode_step(m, w.tokens_stage, B, w.next_stage, nullptr, nullptr, w.alpha_stage)
                            : dbt_decode_step_primary_only(m, w.tokens_stage, B, w.next_stage, nullptr);
    if (st != DBT_OK) return st;
    CUDA_TRY(m, cudaMemcpyAsync(next_host, w.next_stage, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, m->stream));
    if (alpha_host && grouped)
        CUDA_TRY(m, cudaMemcpyAsync(alpha_host, w.alpha_stage, sizeof(float) * B, cudaMemcpyDeviceToHost, m->stream));
    CUDA_TRY(m, cudaStreamSynchronize(m->stream));
    return DBT_OK;
}

dbt_status dbt_decode_step_host(dbt_model *m, const int32_t *tokens_host, int32_t B, int32_t *next_tokens_host,
                                float *alpha_host) {
    return step_host(m, tokens_host, B, next_tokens_host, alpha_host, 1);
}

dbt_status dbt_decode_step_primary_only_host(dbt_model *m, const int32_t *tokens_host, int32_t B,
                                             int32_t *next_tokens_host) {
    return step_host(m, tokens_host, B, next_tokens_host, nullptr, 0);
}

// Moves nb sequences x nt positions of one layer's K (or V) plane between the paged pool and the staging
// buffer, through the page table.  One thread per 16 bytes.
static dbt_status kv_stage_copy(dbt_model *m, int layer, int which, const int32_t *seq_ids_dev, int s0, int nb, int t0, int nt,
                                int to_pool) {
    const dbt_config &c = m->cfg;
    const int row_bytes = c.head_dim * elem_bytes(c);
    char *plane = m->kv_pool + ((size_t)layer * 2 + which) * c.num_pages * c.n_kv_heads * c.page_size * row_bytes;
    size_t vecs = (size_t)nb * nt * c.n_kv_heads * (row_bytes / 16);
    LAUNCH(m, "kv_copy", 0, kv_copy_kernel, (unsigned)((vecs + 255) / 256), 256, 0, plane, m->ws.page_table, m->pages_per_seq_max,
           c.num_pages, c.n_kv_heads, row_bytes, seq_ids_dev, s0, nb, t0, nt, m->ws.kv_stage, to_pool, m->ws.status);
    return DBT_OK;
}

static dbt_status kv_transfer(dbt_model *m, const int32_t *seq_ids_host, int32_t B, int32_t T, char *k_host, char *v_host,
                              int to_pool) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (!k_host || !v_host) return fail(m, DBT_ERR_INVALID_ARG, "NULL host buffer");
    if (B <= 0 || T <= 0 || B > m->cfg.max_batch) return fail(m, DBT_ERR_INVALID_ARG, "bad B or T");
    const dbt_config &c = m->cfg;
    int cap = m->pages_per_seq * c.page_size;
    if (cap > c.max_seq) cap = c.max_seq;
    if (T > cap) return fail(m, DBT_ERR_CAPACITY, "T=%d exceeds the per-sequence capacity %d", T, cap);
    std::vector<int32_t> ids(B);
    for (int b = 0; b < B; b++) {
        ids[b] = seq_ids_host ? seq_ids_host[b] : b;
        if (ids[b] < 0 || ids[b] >= c.max_batch) return fail(m, DBT_ERR_INVALID_ARG, "sequence id %d out of range", ids[b]);
        if (!to_pool && m->len_host[ids[b]] < T)
            return fail(m, DBT_ERR_STATE, "sequence %d holds %d positions, %d requested", ids[b], m->len_host[ids[b]], T);
    }
    // the ids travel in the token staging buffer (max_batch ints)
    CUDA_TRY(m, cudaMemcpyAsync(m->ws.tokens_stage, ids.data(), sizeof(int32_t) * B, cudaMemcpyHostToDevice, m->stream));
    const size_t row = (size_t)c.n_kv_heads * c.head_dim * elem_bytes(c);  // one position of one sequence
    const size_t rows_cap = kKvStageBytes / row;
    if (rows_cap == 0) return fail(m, DBT_ERR_UNSUPPORTED, "kv row larger than the staging buffer");
    const bool use_pdl = m->use_pdl;
    m->use_pdl = false;  // copies and kernels alternate on the stream: plain stream order
    dbt_status st = DBT_OK;
    for (int l = 0; l < c.n_layers && st == DBT_OK; l++)
        for (int which = 0; which < 2 && st == DBT_OK; which++) {
            char *host = (which ? v_host : k_host) + (size_t)l * B * T * row;
            // whole sequences per chunk when a sequence fits, else one sequence in position ranges
            const int seq_per = (size_t)T <= rows_cap ? (int)(rows_cap / T) : 0;
            for (int s0 = 0; s0 < B && st == DBT_OK; s0 += seq_per > 0 ? seq_per : 1) {
                const int nb = seq_per > 0 ? (B - s0 < seq_per ? B - s0 : seq_per) : 1;
                const int t_step = seq_per > 0 ? T : (int)rows_cap;
                for (int t0 = 0; t0 < T && st == DBT_OK; t0 += t_step) {
                    const int nt = T - t0 < t_step ? T - t0 : t_step;
                    char *hp = host + ((size_t)s0 * T + t0) * row;
                    const size_t bytes = (size_t)nb * nt * row;
                    cudaError_t e = cudaSuccess;
                    if (to_pool) e = cudaMemcpyAsync(m->ws.kv_stage, hp, bytes, cudaMemcpyHostToDevice, m->stream);
                    if (e == cudaSuccess) st = kv_stage_copy(m, l, which, m->ws.tokens_stage, s0, nb, t0, nt, to_pool);
                    if (e == cudaSuccess && st == DBT_OK && !to_pool)
                        e = cudaMemcpyAsync(hp, m->ws.kv_stage, bytes, cudaMemcpyDeviceToHost, m->stream);
                    if (e != cudaSuccess) st = fail(m, DBT_ERR_CUDA, "kv transfer: %s", cudaGetErrorString(e));
                }
            }
        }
    m->use_pdl = use_pdl;
    if (st != DBT_OK) return st;
    CUDA_TRY(m, cudaStreamSynchronize(m->stream));
    if (to_pool) {  // the imported sequences now hold T positions
        for (int b = 0; b < B; b++) {
            m->len_host[ids[b]] = T;
            CUDA_TRY(m, cudaMemcpy(m->ws.seq_len + ids[b], &T, sizeof(int32_t), cudaMemcpyHostToDevice));
        }
    }
    return DBT_OK;
}

dbt_status dbt_kv_export(dbt_model *m, const int32_t *seq_ids_host, int32_t B, int32_t T, void *k_host, void *v_host) {
    return kv_transfer(m, seq_ids_host, B, T, (char *)k_host, (char *)v_host, 0);
}

dbt_status dbt_kv_import(dbt_model *m, const int32_t *seq_ids_host, int32_t B, int32_t T, const void *k_host,
                         const void *v_host) {
    return kv_transfer(m, seq_ids_host, B, T, (char *)const_cast<void *>(k_host), (char *)const_cast<void *>(v_host), 1);
}

dbt_status dbt_last_experts(dbt_model *m, const int32_t **experts_dev, int32_t *kmax) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (m->cfg.n_experts == 0) return fail(m, DBT_ERR_STATE, "not an MoE model");
    if (experts_dev) *experts_dev = m->ws.last_experts;
    if (kmax) *kmax = kmax_of(m->cfg);
    return DBT_OK;
}

dbt_status dbt_last_expert_union(dbt_model *m, int32_t *count_per_layer_host) {
    if (!m) return DBT_ERR_INVALID_ARG;
    if (m->cfg.n_experts == 0) return fail(m, DBT_ERR_STATE, "not an MoE model");
    if (!count_per_layer_host) return fail(m, DBT_ERR_INVALID_ARG, "NULL output");
    CUDA_TRY(m, cudaStreamSynchronize(m->stream));
    CUDA_TRY(m, cudaMemcpy(count_per_layer_host, m->ws.union_cnt, sizeof(int32_t) * m->cfg.n_layers, cudaMemcpyDeviceToHost));
    return DBT_OK;
}

dbt_status dbt_sync_status(dbt_model *m, int32_t *device_status, int32_t *detail) {
    if (!m) return DBT_ERR_INVALID_ARG;
    int32_t h[2] = {0, 0};
    CUDA_TRY(m, cudaStreamSynchronize(m->stream));
    CUDA_TRY(m, cudaMemcpy(h, m->ws.status, sizeof h, cudaMemcpyDeviceToHost));
    if (device_status) *device_status = h[0];
    if (detail) *detail = h[1];
    if (h[0] == kStatusWaitExpired)
        return fail(m, DBT_ERR_TIMEOUT, "a bounded device wait ran out (wait site %d)", h[1]);
    if (h[0] != 0) return fail(m, DBT_ERR_DEVICE, "device status %d (detail %d)", h[0], h[1]);
    return DBT_OK;
}

int64_t dbt_launch_count(const dbt_model *m) { return m ? m->launches : 0; }

static dbt_status op_gemm_tc_impl(dbt_model *m, const void *W_dev, const void *X_dev, int32_t n_out, int32_t K,
                                  int32_t R, int32_t force_split, float *Y_dev, float *scratch_dev,
                                  size_t scratch_floats, int32_t *status_dev, int32_t *split_used) {
    if (!W_dev || !X_dev || !Y_dev || !scratch_dev || !status_dev) return fail(m, DBT_ERR_INVALID_ARG, "NULL pointer");
    if (n_out <= 0 || K <= 0 || K % 8 || R <= 0 || R > 256) return fail(m, DBT_ERR_UNSUPPORTED, "need K %% 8 == 0, 1 <= R <= 256");
    if (((uintptr_t)W_dev | (uintptr_t)X_dev) & 15) return fail(m, DBT_ERR_INVALID_ARG, "operands must be 16-byte aligned");
    CUtensorMap mw, mx;
    if (!allow_smem_all()) return fail(m, DBT_ERR_CUDA, "cannot raise the shared-memory limit");
    if (!make_bf16_map(&mw, W_dev, n_out, K, kTcM) || !make_bf16_map(&mx, X_dev, R, K, 16))
        return fail(m, DBT_ERR_CUDA, "cuTensorMapEncodeTiled failed");
    m->ws.status = status_dev;
    TcCall c{};
    c.W[0] = &mw; c.n_out[0] = n_out; c.rows[0] = R; c.nseg = 1; c.X = &mx; c.K = K; c.R = R;
    c.P = scratch_dev; c.P_floats = scratch_floats; c.tag = "gemm"; c.parts = 1; c.lo_row0 = 0;
    if (force_split > (K + kTcK - 1) / kTcK) force_split = (K + kTcK - 1) / kTcK;  // at most one k-tile per split
    if (force_split > 0) {  // honour the request by shrinking the scratch the heuristic may use
        size_t per = (size_t)pad_rows(R) * n_out;
        if ((size_t)force_split * per > scratch_floats) return fail(m, DBT_ERR_CAPACITY, "scratch too small");
    }
    int nsp = 1;
    size_t stride = 0;
    // Test hook (host-set, off by default): DBT_TEST_EXPIRE_WAIT=1 makes CTA (0,0,0) skip one weight-tile request
    // and shortens every wait to about a millisecond, so that a test can watch a bounded wait run out: the kernel
    // records status 3 in status_dev and returns normally.  No other entry point reads the variable.
    const char *tw = getenv("DBT_TEST_EXPIRE_WAIT");
    dbt_status st = run_gemm_tc(m, c, pad_rows(R), &nsp, &stride, force_split, LmEpi{}, tw && strcmp(tw, "1") == 0);
    if (st != DBT_OK) return st;
    size_t n = (size_t)R * n_out;
    LAUNCH(m, "reduce", 0, reduce_splits_kernel, (unsigned)((n + 255) / 256), 256, 0, scratch_dev, nsp, stride, n, Y_dev);
    if (split_used) *split_used = nsp;
    return DBT_OK;
}

// ---- no-allocation variant -----------------------------------------------------------------
// Split-K scratch for dbt_op_gemm_tc_static lives in this file-scope device array: 2^21 floats
// (8 MiB), held by every GPU that loads the library until the process exits.  Host code may
// not pass the symbol to a kernel (on the host it is only a stand-in for the device array):
// its device address is looked up once per device with cudaGetSymbolAddress.
constexpr size_t kStaticScratchFloats = (size_t)1 << 21;
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

static float *static_scratch_for_current_device(cudaError_t *err) {
    static std::mutex mu;
    static float *ptr_of_device[64] = {nullptr};
    int dev = -1;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= 64) {
        *err = cudaErrorInvalidDevice;
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!ptr_of_device[dev]) {
        void *p = nullptr;
        *err = cudaGetSymbolAddress(&p, g_static_scratch);  // resolved for the current device
        if (*err != cudaSuccess) return nullptr;
        ptr_of_device[dev] = static_cast<float *>(p);
    }
    return ptr_of_device[dev];
}

dbt_status dbt_op_gemm_tc_static(const void *W_dev, const void *X_dev, int32_t n_out, int32_t K, int32_t R,
                                 int32_t force_split, float *Y_dev, int32_t *status_dev, void *cuda_stream,
                                 int32_t *split_used) {
    static thread_local dbt_model scratch_handle;  // carries the stream and the error text only
    dbt_model *m = &scratch_handle;
    m->stream = (cudaStream_t)cuda_stream;
    m->prof_on = false;
    m->use_pdl = false;
    dbt_status st;
    cudaError_t ce = cudaSuccess;
    float *scratch = static_scratch_for_current_device(&ce);
    if (!scratch) {
        st = fail(m, DBT_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(ce));
    } else if (n_out > 0 && R > 0 && R <= 256 && (size_t)pad_rows(R) * (size_t)n_out > kStaticScratchFloats) {
        st = fail(m, DBT_ERR_CAPACITY,
                  "roundup(R)=%d rows x n_out=%d = %zu floats exceed the static scratch of %zu floats (8 MiB); "
                  "use dbt_op_gemm_tc with caller-provided scratch",
                  pad_rows(R), n_out, (size_t)pad_rows(R) * (size_t)n_out, kStaticScratchFloats);
    } else if (force_split > 0 && K > 0 &&
               (size_t)(force_split < (K + kTcK - 1) / kTcK ? force_split : (K + kTcK - 1) / kTcK) *
                       pad_rows(R > 0 && R <= 256 ? R : 1) * (size_t)(n_out > 0 ? n_out : 0) >
                   kStaticScratchFloats) {
        st = fail(m, DBT_ERR_CAPACITY, "force_split=%d needs more than the static scratch of %zu floats (8 MiB)",
                  force_split, kStaticScratchFloats);
    } else {
        st = op_gemm_tc_impl(m, W_dev, X_dev, n_out, K, R, force_split, Y_dev, scratch, kStaticScratchFloats, status_dev,
                             split_used);
    }
    if (st != DBT_OK) g_create_error = m->err;
    return st;
}

dbt_status dbt_op_gemm_tc(const void *W_dev, const void *X_dev, int32_t n_out, int32_t K, int32_t R, int32_t force_split,
                          float *Y_dev, float *scratch_dev, size_t scratch_floats, int32_t *status_dev,
                          void *cuda_stream, int32_t *split_used) {
    static thread_local dbt_model scratch_handle;  // carries the stream and the error text only
    dbt_model *m = &scratch_handle;
    m->stream = (cudaStream_t)cuda_stream;
    m->prof_on = false;
    m->use_pdl = false;
    dbt_status st = op_gemm_tc_impl(m, W_dev, X_dev, n_out, K, R, force_split, Y_dev, scratch_dev, scratch_floats,
                                    status_dev, split_used);
    if (st != DBT_OK) g_create_error = m->err;
    return st;
}

}  // extern "C"

#ifdef DBT_TIMELINE
// Instrumentation builds only: copies the kernels' timeline records out and clears the list.
extern "C" int dbt_debug_timeline(unsigned long long *out_host, int max_records) {
    unsigned int n = 0;
    cudaDeviceSynchronize();
    if (cudaMemcpyFromSymbol(&n, dbt::g_tl_n, sizeof n) != cudaSuccess) return -1;
    if ((int)n > max_records) n = max_records;
    if (n > (unsigned)dbt::kTlMax) n = dbt::kTlMax;
    if (n && cudaMemcpyFromSymbol(out_host, dbt::g_tl, sizeof(unsigned long long) * 8 * n) != cudaSuccess) return -1;
    unsigned int zero = 0;
    cudaMemcpyToSymbol(dbt::g_tl_n, &zero, sizeof zero);
    return (int)n;
}
#endif
