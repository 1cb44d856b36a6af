// Grouped decode attention for a bf16 paged KV cache (sm_100a).
//
// One CTA per (primary row, KV head, split of the context).  The G primary query heads of
// that KV head and, in grouped mode, the G coupled branch heads (Q~_2 = Q_2 + a*Q_1) form one
// 16-row query tile, so every K/V page is fetched from HBM once and serves both paths
// (Section 4.1: "grouped or fused query execution lets the two paths share reads of the
// primary keys and values").  Keys 0..pos inclusive: the K_1,V_1 appended this step is
// already in its page.
//
// Data movement: a producer warp walks the page table and brings 16-token pages in with
// tiled TMA copies (128B swizzle) into a shared-memory ring, 64 tokens per stage.  Math:
// four consumer warps, one page each per stage; S = Q K^T and O += P V with mma.sync
// m16n8k16 (bf16 in, fp32 accumulate), operands read with ldmatrix through the swizzle; each
// warp keeps its own running (max, sum, O) and the four are folded in warp order at the end.
// The CTA writes an un-normalised partial (m, l, O) per split; attn_merge_kernel folds the
// splits in split order.  All waits are bounded.
#pragma once

#include "dbt_gemm_tc.cuh"

namespace dbt {

struct AttnParams {
    const float *Q;  // [rows][q_dim] fp32, post-RoPE, branch rows already coupled
    RowMap rm;
    int grouped, G, n_kv, nsplit, num_pages, pt_stride;
    long long k_row0, v_row0;  // first row of this layer's K / V planes in the pool's 2-D view
    const int32_t *page_table, *seq_len;
    float *part;  // [items][n_kv][nsplit][16][DH + 2]
    int *tickets;  // [items][n_kv] arrival counters (zero between launches)
    __nv_bfloat16 *Ob;  // [rows][q_dim] attention output, hi plane (+ lo plane at lo_off)
    size_t lo_off;
    int *status;
};

constexpr int kAttTile = 64;      // tokens per pipeline stage (4 pages)
constexpr int kAttWarps = 4;      // consumer warps, one page each
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int DH>
struct AttCfg {
    static constexpr int kHalves = DH / 64;                 // 128-byte column groups per row
    static constexpr int kPageBytes = 16 * DH * 2;          // one page of K (or V) for one head
    static constexpr int kStageBytes = 2 * 4 * kPageBytes;  // K + V, 4 pages
    static constexpr int kStages = DH == 128 ? 2 : 4;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 128;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

template <int DH>
__global__ void __launch_bounds__(160, 3) attn_mma_kernel(const __grid_constant__ CUtensorMap tmKV, AttnParams p) {
    using Cfg = AttCfg<DH>;
    constexpr int STAGES = Cfg::kStages, HALVES = Cfg::kHalves, KS = DH / 16, NB = DH / 8;
    extern __shared__ uint8_t smem_raw[];
    uint32_t raw = smem_u32(smem_raw);
    uint32_t tiles = (raw + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (tiles - raw);
    uint32_t bars = tiles + STAGES * Cfg::kStageBytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };

    int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int item = blockIdx.x, g = blockIdx.y, sp = blockIdx.z;
    int Bc = p.rm.Bc(), seq = p.rm.seq(item);
    int nq_act = p.grouped ? 2 * p.G : p.G, q_dim = p.n_kv * p.G * DH;

    if (tid == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), kAttWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();  // sequence lengths, Q and the freshly appended K/V come from earlier kernels of the step
    int nkeys = ld_mut(p.seq_len + seq) + p.rm.off(item) + 1;
    int total_pages = (nkeys + 15) >> 4;
    int pps = (total_pages + p.nsplit - 1) / p.nsplit;
    int pb = sp * pps, pe = min(total_pages, pb + pps);
    int jbeg = pb * 16, jend = min(nkeys, pe * 16);
    int ntiles = jend > jbeg ? (jend - jbeg + kAttTile - 1) / kAttTile : 0;

    float *out = p.part + (((size_t)item * p.n_kv + g) * p.nsplit + sp) * 16 * (DH + 2);

    if (warp == kAttWarps) {
        // ---- producer: page table walk + TMA
        if (lane == 0) {
            tma_prefetch_desc(&tmKV);
            bool ok = true;
            for (int i = 0; i < ntiles && ok; i++) {
                int s = i % STAGES;
                if (i >= STAGES) ok = mbar_wait(empty_bar(s), ((i / STAGES) - 1) & 1);
                if (!ok) break;
                int p0 = pb + i * 4, np = min(4, pe - p0);
                mbar_expect_tx(full_bar(s), (uint32_t)np * 2 * Cfg::kPageBytes);
                uint32_t kdst = tiles + s * Cfg::kStageBytes, vdst = kdst + 4 * Cfg::kPageBytes;
                for (int j = 0; j < np; j++) {
                    int page = p.page_table[(size_t)seq * p.pt_stride + p0 + j];
                    if (page < 0 || page >= p.num_pages) {
                        report(p.status, kStatusBadPage, page);
                        page = 0;
                    }
                    int row = (int)(((long long)page * p.n_kv + g) * 16);
                    for (int h = 0; h < HALVES; h++) {
                        tma_load_2d(kdst + (j * HALVES + h) * 2048, &tmKV, full_bar(s), h * 64, (int)(p.k_row0 + row));
                        tma_load_2d(vdst + (j * HALVES + h) * 2048, &tmKV, full_bar(s), h * 64, (int)(p.v_row0 + row));
                    }
                }
            }
            if (!ok) report(p.status, kStatusWaitExpired, 300);
        }
        return;
    }

    // ---- consumers.  Query tile as mma A fragments (bf16), pre-scaled by log2(e)/sqrt(d_h).
    uint32_t qa[KS][4];
    {
        float scale = kLog2e / sqrtf((float)DH);
        int r0 = lane >> 2, r1 = r0 + 8, c = (lane & 3) * 2;
        auto qrow = [&](int q) -> const float * {
            if (q >= nq_act) return nullptr;
            int row = q < p.G ? item : Bc + item;
            int h = g * p.G + (q < p.G ? q : q - p.G);
            return p.Q + (size_t)row * q_dim + (size_t)h * DH;
        };
        const float *q0 = qrow(r0), *q1 = qrow(r1);
#pragma unroll
        for (int ks = 0; ks < KS; ks++) {
            int k = ks * 16 + c;
            qa[ks][0] = q0 ? pack_bf16(__ldcg(q0 + k) * scale, __ldcg(q0 + k + 1) * scale) : 0u;
            qa[ks][1] = q1 ? pack_bf16(__ldcg(q1 + k) * scale, __ldcg(q1 + k + 1) * scale) : 0u;
            qa[ks][2] = q0 ? pack_bf16(__ldcg(q0 + k + 8) * scale, __ldcg(q0 + k + 9) * scale) : 0u;
            qa[ks][3] = q1 ? pack_bf16(__ldcg(q1 + k + 8) * scale, __ldcg(q1 + k + 9) * scale) : 0u;
        }
    }
    float o[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; nb++) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    bool ok = true;
    for (int i = 0; i < ntiles; i++) {
        int s = i % STAGES;
        ok = mbar_wait(full_bar(s), (i / STAGES) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        int tile_j0 = jbeg + i * kAttTile;
        int valid = min(16, jend - (tile_j0 + warp * 16));  // valid tokens in this warp's page
        if (valid > 0) {
            uint32_t kpage = tiles + s * Cfg::kStageBytes + warp * HALVES * 2048;
            uint32_t vpage = kpage + 4 * Cfg::kPageBytes;
            if (valid < 16) {
                // stale slots past the end of the sequence: their scores are masked below, and
                // their V rows are zeroed here so that 0 * garbage cannot produce a NaN
                for (int idx = lane; idx < (16 - valid) * HALVES * 8; idx += 32) {
                    int r = valid + idx / (HALVES * 8), rest = idx % (HALVES * 8);
                    uint32_t a = vpage + (rest / 8) * 2048 + r * 128 + (rest % 8) * 16;
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                }
                __syncwarp();
            }
            // S = Q K^T for this warp's 16 tokens: two 8-token column blocks
            float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            {
                int r = (lane & 7) + ((lane >> 4) << 3);  // token row this lane addresses
                int cb = (lane >> 3) & 1;                 // which 8-dim chunk of the k-step
#pragma unroll
                for (int ks = 0; ks < KS; ks++) {
                    int chunk = ks * 2 + cb;  // 16-byte chunk index within the row
                    uint32_t a = kpage + (chunk >> 3) * 2048 + r * 128 + (((chunk & 7) ^ (r & 7)) << 4);
                    uint32_t kb[4];
                    ldsm_x4(a, kb);
                    mma_bf16(sacc[0], qa[ks], kb[0], kb[1]);
                    mma_bf16(sacc[1], qa[ks], kb[2], kb[3]);
                }
            }
            // mask, online softmax (base 2), pack P as the A operand of P V
            int col = (lane & 3) * 2;
            float rmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nb = 0; nb < 2; nb++)
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    int t = nb * 8 + col + (e & 1);
                    if (t >= valid) sacc[nb][e] = -INFINITY;
                    rmax[e >> 1] = fmaxf(rmax[e >> 1], sacc[nb][e]);
                }
            float corr[2], msub[2];
#pragma unroll
            for (int h = 0; h < 2; h++) {
                rmax[h] = fmaxf(rmax[h], __shfl_xor_sync(0xffffffffu, rmax[h], 1));
                rmax[h] = fmaxf(rmax[h], __shfl_xor_sync(0xffffffffu, rmax[h], 2));
                float mnew = fmaxf(m_run[h], rmax[h]);
                msub[h] = mnew == -INFINITY ? 0.f : mnew;
                corr[h] = m_run[h] == -INFINITY ? 0.f : exp2f(m_run[h] - msub[h]);
                m_run[h] = mnew;
            }
            float rsum[2] = {0.f, 0.f};
            uint32_t pa[4];
#pragma unroll
            for (int nb = 0; nb < 2; nb++) {
                float p0 = exp2f(sacc[nb][0] - msub[0]), p1 = exp2f(sacc[nb][1] - msub[0]);
                float p2 = exp2f(sacc[nb][2] - msub[1]), p3 = exp2f(sacc[nb][3] - msub[1]);
                rsum[0] += p0 + p1;
                rsum[1] += p2 + p3;
                pa[nb * 2 + 0] = pack_bf16(p0, p1);
                pa[nb * 2 + 1] = pack_bf16(p2, p3);
            }
#pragma unroll
            for (int h = 0; h < 2; h++) {
                rsum[h] += __shfl_xor_sync(0xffffffffu, rsum[h], 1);
                rsum[h] += __shfl_xor_sync(0xffffffffu, rsum[h], 2);
                l_run[h] = l_run[h] * corr[h] + rsum[h];
            }
#pragma unroll
            for (int nb = 0; nb < NB; nb++) {
                o[nb][0] *= corr[0];
                o[nb][1] *= corr[0];
                o[nb][2] *= corr[1];
                o[nb][3] *= corr[1];
            }
            // O += P V: V read transposed, two 8-dim column blocks per ldmatrix
            {
                int r = (lane & 7) + (((lane >> 3) & 1) << 3);  // token row
                int cb = lane >> 4;                              // which of the two dim blocks
#pragma unroll
                for (int np = 0; np < NB / 2; np++) {
                    int chunk = np * 2 + cb;
                    uint32_t a = vpage + (chunk >> 3) * 2048 + r * 128 + (((chunk & 7) ^ (r & 7)) << 4);
                    uint32_t vb[4];
                    ldsm_x4_trans(a, vb);
                    mma_bf16(o[np * 2], pa, vb[0], vb[1]);
                    mma_bf16(o[np * 2 + 1], pa, vb[2], vb[3]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(s)) : "memory");
    }
    if (!ok && lane == 0) report(p.status, kStatusWaitExpired, 310 + warp);

    // ---- fold the four warps' states in warp order and write this split's partial
    asm volatile("bar.sync 1, 128;" ::: "memory");  // every consumer is done with the ring
    float *sc_o = reinterpret_cast<float *>(gen);            // [4][16][DH]
    float *sc_m = sc_o + kAttWarps * 16 * DH;                // [4][16]
    float *sc_l = sc_m + kAttWarps * 16;                     // [4][16]
    {
        int r0 = lane >> 2, c = (lane & 3) * 2;
#pragma unroll
        for (int nb = 0; nb < NB; nb++) {
            *reinterpret_cast<float2 *>(sc_o + ((size_t)warp * 16 + r0) * DH + nb * 8 + c) = make_float2(o[nb][0], o[nb][1]);
            *reinterpret_cast<float2 *>(sc_o + ((size_t)warp * 16 + r0 + 8) * DH + nb * 8 + c) = make_float2(o[nb][2], o[nb][3]);
        }
        if ((lane & 3) == 0) {
            sc_m[warp * 16 + r0] = m_run[0];
            sc_m[warp * 16 + r0 + 8] = m_run[1];
            sc_l[warp * 16 + r0] = l_run[0];
            sc_l[warp * 16 + r0 + 8] = l_run[1];
        }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    for (int idx = tid; idx < nq_act * DH; idx += 128) {
        int q = idx / DH, e = idx % DH;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kAttWarps; w++) M = fmaxf(M, sc_m[w * 16 + q]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kAttWarps; w++) {
            float mw = sc_m[w * 16 + q];
            float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
            L += sc_l[w * 16 + q] * f;
            acc += sc_o[((size_t)w * 16 + q) * DH + e] * f;
        }
        out[(size_t)q * (DH + 2) + e] = ok ? acc : 0.f;
        if (e == 0) {
            out[(size_t)q * (DH + 2) + DH] = ok ? M * kLn2 : -INFINITY;  // natural-log units
            out[(size_t)q * (DH + 2) + DH + 1] = ok ? L : 0.f;
        }
    }
    // ---- the last split to arrive for this (row, KV head) folds all splits in split order
    __threadfence();
    asm volatile("bar.sync 1, 128;" ::: "memory");
    int *flag = reinterpret_cast<int *>(sc_l + kAttWarps * 16);
    if (tid == 0) {
        int *tk = p.tickets + (size_t)item * p.n_kv + g;
        int t = atomicAdd(tk, 1);
        int last = t == p.nsplit - 1;
        if (last) atomicExch(tk, 0);
        *flag = last;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (!*flag) return;
    __threadfence();
    const float *base = p.part + ((size_t)item * p.n_kv + g) * p.nsplit * 16 * (DH + 2);
    for (int idx = tid; idx < nq_act * DH; idx += 128) {
        int q = idx / DH, e = idx % DH;
        float M = -INFINITY;
        for (int s2 = 0; s2 < p.nsplit; s2++) M = fmaxf(M, __ldcg(base + ((size_t)s2 * 16 + q) * (DH + 2) + DH));
        float L = 0.f, acc = 0.f;
        for (int s2 = 0; s2 < p.nsplit; s2++) {
            const float *pp = base + ((size_t)s2 * 16 + q) * (DH + 2);
            float ms = __ldcg(pp + DH);
            float f = ms == -INFINITY ? 0.f : expf(ms - M);
            L += __ldcg(pp + DH + 1) * f;
            acc += __ldcg(pp + e) * f;
        }
        float x = acc / L;
        int row = q < p.G ? item : Bc + item;
        int h = g * p.G + (q < p.G ? q : q - p.G);
        size_t o_idx = (size_t)row * q_dim + (size_t)h * DH + e;
        __nv_bfloat16 hi = __float2bfloat16_rn(x);
        p.Ob[o_idx] = hi;
        if (p.lo_off) p.Ob[o_idx + p.lo_off] = __float2bfloat16_rn(x - __bfloat162float(hi));
    }
}

// The whole pool as one 2-D bf16 tensor [rows][head_dim], rows = (layer, K|V, page, head, slot).
inline bool make_kv_map(CUtensorMap *map, const void *pool, uint64_t total_rows, int head_dim) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || total_rows >= (1ull << 31)) return false;
    cuuint64_t dims[2] = {(cuuint64_t)head_dim, total_rows};
    cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
    cuuint32_t box[2] = {64, 16};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace dbt
