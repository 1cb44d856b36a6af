// Grouped decode attention for a bf16 paged KV cache (sm_100a).
//
// The G primary query heads of a KV head and, in grouped mode, the G coupled branch heads
// (Q~_2 = Q_2 + a*Q_1) form one 16-row query tile, so every K/V page is fetched from HBM once
// and serves both paths (Section 4.1: "grouped or fused query execution lets the two paths
// share reads of the primary keys and values").  Keys 0..pos inclusive: the K_1,V_1 appended
// this step is already in its page.
//
// Work decomposition.  A (row, KV head) pair of u 64-token stages is cut into n ~ u / q equal
// segments (q: a target length chosen so that the segments fill one to three rounds of the
// grid); the segments of all pairs, in (row, KV head, segment) order, are dealt to a fixed grid
// of CTAs (two per SM) round robin.
// A CTA never straddles two pairs (the per-segment costs -- building the queries, folding the
// warps, the merge -- are then paid once per CTA for equal-length batches), and the split depends
// on the lengths only.  A segment's un-normalised partial (m, l, O) goes to the slot of its
// index, consecutive for one pair; the last segment of a pair to arrive merges them in segment
// order (in two levels above 8 segments), so the result does not depend on arrival order.
//
// Data movement: a producer warp walks the page table and brings 16-token pages in with one 4-D
// TMA box per page (K and V, 128B swizzle) into a shared-memory ring, 64 tokens per stage, ~190 KB
// in flight per SM, with the evict-first L2 hint.  Math: four consumer warps, one page each per
// stage, mma.sync m16n8k16 (bf16 in, fp32 accumulate), operands read with ldmatrix through the
// swizzle; with at most 8 query rows per KV head the products are taken transposed (keys on the
// M side).  Each warp keeps its own running (max, sum, O) and the four are folded in a fixed
// order at the end of a segment.  In decode steps the kernel also builds its queries and the
// new K,V row from the Q|K|V GEMM's split-K partials.  All waits are bounded.
#pragma once

#include "dbt_fused.cuh"
#include "dbt_gemm_tc.cuh"

namespace dbt {

struct AttnParams {
    const float *Q;  // [rows][q_dim] fp32, post-RoPE, branch rows already coupled
    RowMap rm;
    int grouped;  // paths present: 0 or 1 = the primary alone, P >= 2 = the primary and P-1 decode branches
    int G, n_kv, num_pages, pt_stride;
    long long k_row0;  // first row of this layer's K plane in the pool's row numbering (the V plane is one plane further)
    const int32_t *page_table, *seq_len;
    float *part;        // [CTAs + pairs][16][DH + 2] segment partials
    int *tickets;       // [rows][n_kv] arrival counters (zero between launches)
    int *tickets2;      // [rows][n_kv][kAttMaxGroups] arrival counters of the segment groups
    __nv_bfloat16 *Ob;  // [rows][q_dim] attention output, hi plane (+ lo plane at lo_off)
    size_t lo_off;
    int *status;
    int evict_first;  // K/V pages carry the evict-first L2 hint (read once per step)
    // Decode steps take the Q|K|V GEMM's split-K partials directly (no kernel in between): each CTA
    // builds its pair's queries itself (1/rms, RoPE, Q~_2 = Q_2 + a*Q_1, Eq. asymattn), and the CTA that
    // owns the pair's last stage computes the new K_1, V_1 row, writes it to the pool for later steps
    // and patches it into the staged page.  qkv_P == nullptr: Q comes from `Q`, the cache is complete.
    const float *qkv_P;  // [nsplit][rows][q_dim | kv_dim | kv_dim]
    int qkv_nsplit;
    size_t qkv_stride;
    const float *ss;  // shares of sum(S^2) per row (nullptr: the GEMM input was already normalised)
    int ss_tiles, ss_ld, d_norm;
    float eps;
    const float *coup_a;
    const float2 *rope;
    __nv_bfloat16 *kpool, *vpool;  // this layer's K and V planes
    // Prompt chunks (Section 4.4 item 1, the primary path alone): pack > 0 packs `pack` consecutive positions of
    // a sequence (times the G heads of the KV head) into one 16-row query tile, each row with its own causal
    // limit; a chunk holds cn positions per sequence, nbk = ceil(cn / pack) tiles per sequence, one CTA pass per
    // (tile, KV head) over all its keys, no split.  Q rows and output rows are seq * cn + position.
    int pack, cn, nbk;
    const int *plan;   // the step's precomputed work split (attn_plan_kernel), or nullptr
    int plan_prewait;  // the plan may be read before the dependency wait
};

constexpr int kAttTile = 64;       // tokens per pipeline stage (4 pages)
constexpr int kAttWarps = 4;       // consumer warps, one page each
constexpr int kAttMaxItems = 256;  // rows per launch (prefill chunks and batches stay below)
constexpr int kAttMinUnits = 4;    // a CTA takes at least 4 tiles (256 tokens)
constexpr int kAttPauseAt = 1;     // the producer pauses after stage 1 (the second) until the queries are built
constexpr int kAttMaxSeg = 256;    // most segments a (sequence, KV head) pair is split into
constexpr int kAttGroup = 8;       // segments merged at once (one round of loads)
constexpr int kAttSingle = 16;     // up to this many segments, one CTA merges them all (two rounds of loads)
constexpr int kAttMaxGroups = kAttMaxSeg / kAttGroup;
constexpr float kLog2e = 1.4426950408889634f;

// DEEP: one CTA per SM with a ring twice as deep instead of two CTAs per SM: the same bytes in flight per SM,
// half as many segments (fewer query builds, partials and merges).  (A second group of four consumer warps
// taking alternate stages of the deep ring was measured 1 % slower: the stream, not the consumers, sets the pace.)
template <int DH, bool DEEP = false>
struct AttCfg {
    static constexpr int kHalves = DH / 64;                 // 128-byte column groups per row
    static constexpr int kPageBytes = 16 * DH * 2;          // one page of K (or V) for one head
    static constexpr int kStageBytes = 2 * 4 * kPageBytes;  // K + V, 4 pages
    static constexpr int kStages = (DH == 128 ? 3 : 6) * (DEEP ? 2 : 1);  // 96 KB ring: two CTAs keep ~190 KB in flight per SM
    // scratch: one [16][DH + 8] fp32 slot (Q tile / warp fold; the padding keeps the fold's
    // fragment-shaped accesses off a single bank), m, l, flag, row tables
    static constexpr int kFoldStride = DH + 8;
    static constexpr int kScratchBytes = (16 * kFoldStride + 2 * 16 + 16 + 3 * kAttMaxItems + 12) * 4 + 2 * DH * 2 + 32;
    // room for the ring's barriers (two per stage, up to 12 stages) ahead of the scratch
    static constexpr int kBarBytes = 256;
    static_assert(2 * kStages * 8 <= kBarBytes, "the barriers must not reach into the scratch");
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + kBarBytes + kScratchBytes;
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
// Transpose of an 8x8 matrix of 16-bit elements held one row pair per lane (the layout of an
// accumulator's 8x8 block packed to bf16).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3,
                                                 uint64_t hint) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, "
        "%6}], [%2], %7;" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(hint)
        : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// The work split of one attention launch, computed by one warp from the sequence lengths: cum[i] = stages of the
// rows before row i, nk[i] = keys visible to row i, segcum[i] = segments (per KV head) of the rows before row i.
// The same for every layer of a decode step, so a step computes it once (attn_plan_kernel) and the attention
// launches copy it; launches without a plan (prompt chunks) compute it themselves.
__device__ __forceinline__ void att_plan_warp(int lane, int items, RowMap rm, const int32_t *seq_len, int n_kv, int C0_arg,
                                              int *cum, int *nk_s, int *segcum) {
    int running = 0, longest = 0;
    if (lane == 0) cum[0] = 0;
    for (int base = 0; base < items; base += 32) {
        int i = base + lane, nk = 0, u = 0;
        if (i < items) {
            nk = ld_mut(seq_len + rm.seq(i)) + rm.off(i) + 1;
            u = (nk + kAttTile - 1) / kAttTile;
            nk_s[i] = nk;
        }
        int incl = u, mx = u;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
            mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        longest = max(longest, mx);
        if (i < items) cum[i + 1] = running + incl;
        running += __shfl_sync(0xffffffffu, incl, 31);
    }
    __syncwarp();
    // Work split: a (row, KV head) pair of u stages is cut into n equal segments and CTA c takes
    // segments c, c + C0_arg, ...: a CTA never straddles two pairs, and the split depends on
    // the lengths only.  n = round or floor of u / q for a target segment length q = all stages /
    // (k * CTAs), k = 1..3 rounds; of these six candidates the one with the smallest estimated
    // time (rounds x (longest segment + a fixed per-segment cost of ~6 stages)) is taken, fewer
    // segments on ties.
    const int C0 = C0_arg, U0 = cum[items] * n_kv;
    auto seg_count = [&](int u, int q, int mode) {  // mode 0: round, 1: floor
        int n = mode == 0 ? (2 * u + q) / (2 * q) : u / q;
        return min(max(n, 1), min(max(u, 1), kAttMaxSeg));
    };
    int best_q = max((U0 + C0 - 1) / C0, kAttMinUnits), best_mode = 0;
    int best_cost = -1, best_sg = 0;
    for (int cand = 0; cand < 6; cand++) {
        const int k = cand / 2 + 1, mode = cand & 1;
        const int q = max((U0 + k * C0 - 1) / (k * C0), kAttMinUnits);
        int sg = 0, longest_seg = 0;
        for (int base = 0; base < items; base += 32) {
            int i = base + lane;
            if (i < items) {
                int u = cum[i + 1] - cum[i], n = seg_count(u, q, mode);
                sg += n;
                longest_seg = max(longest_seg, (u + n - 1) / n);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            sg += __shfl_xor_sync(0xffffffffu, sg, o);
            longest_seg = max(longest_seg, __shfl_xor_sync(0xffffffffu, longest_seg, o));
        }
        sg *= n_kv;
        int rounds = (sg + C0 - 1) / C0, cost = rounds * (longest_seg + 6);
        if (best_cost < 0 || cost < best_cost || (cost == best_cost && sg < best_sg)) {
            best_cost = cost;
            best_q = q;
            best_mode = mode;
            best_sg = sg;
        }
        // the plain split fits one round, or every pair is already whole: take it (the common cases)
        if (cand == 0 && (rounds == 1 || sg == items * n_kv)) break;
    }
    int run2 = 0;
    if (lane == 0) segcum[0] = 0;
    for (int base = 0; base < items; base += 32) {
        int i = base + lane, n = 0;
        if (i < items) n = seg_count(cum[i + 1] - cum[i], best_q, best_mode);
        int incl = n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (i < items) segcum[i + 1] = run2 + incl;
        run2 += __shfl_sync(0xffffffffu, incl, 31);
    }
}

constexpr int kAttPlanInts = 3 * kAttMaxItems + 2;  // cum [items + 1] | nk [items] | segcum [items + 1], at fixed offsets

__global__ void __launch_bounds__(32) attn_plan_kernel(RowMap rm, const int32_t *seq_len, int n_kv, int C0, int *plan) {
    pdl_enter();
    att_plan_warp(threadIdx.x, rm.Bc(), rm, seq_len, n_kv, C0, plan, plan + kAttMaxItems + 1, plan + 2 * kAttMaxItems + 1);
}

template <int DH, bool NARROW, bool DEEP = false>
__global__ void __launch_bounds__(160, DEEP ? 1 : 2) attn_mma_kernel(const __grid_constant__ CUtensorMap tmKV, AttnParams p) {
    using Cfg = AttCfg<DH, DEEP>;
    constexpr int STAGES = Cfg::kStages, HALVES = Cfg::kHalves, KS = DH / 16, NB = DH / 8;
    extern __shared__ uint8_t smem_raw[];
    uint32_t raw = smem_u32(smem_raw);
    uint32_t tiles = (raw + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (tiles - raw);
    uint32_t bars = tiles + STAGES * Cfg::kStageBytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    constexpr int FS = Cfg::kFoldStride;
    float *sc_o = reinterpret_cast<float *>(gen + STAGES * Cfg::kStageBytes + Cfg::kBarBytes);  // [16][FS]
    float *sc_m = sc_o + 16 * FS;                                                   // [16]
    float *sc_l = sc_m + 16;                                                        // [16]
    int *flag = reinterpret_cast<int *>(sc_l + 16);                                 // [0] last?, [1] longest pair, [8..15] 1/rms per path
    int *cum = flag + 16;                // [items + 1] prefix of tiles per row
    int *nk_s = cum + kAttMaxItems + 1;  // [items] visible keys per row
    int *segcum = nk_s + kAttMaxItems;   // [items + 1] prefix of segments per row (per KV head)
    __nv_bfloat16 *kv_new =  // [2][DH] this step's K, V row (16-byte aligned)
        reinterpret_cast<__nv_bfloat16 *>((reinterpret_cast<uintptr_t>(segcum + kAttMaxItems + 1) + 15) & ~(uintptr_t)15);

    DBT_TL_DECL;
    int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int items = p.rm.Bc(), Bc = items;
    const int P = p.grouped > 1 ? p.grouped : 1;  // query rows of a KV head: G heads of every path, path-major
    int nq_act = P * p.G, q_dim = p.n_kv * p.G * DH;
    const bool packed = p.pack > 0;
    if (packed) items = p.rm.B * p.nbk;
    // geometry of an item: its sequence, the keys visible to its last row, the positions it holds
    auto item_seq = [&](int i) { return packed ? i / p.nbk : p.rm.seq(i); };
    auto item_npos = [&](int i) { return packed ? min(p.pack, p.cn - (i % p.nbk) * p.pack) : 1; };
    auto item_row0 = [&](int i) { return packed ? (i / p.nbk) * p.cn + (i % p.nbk) * p.pack : i; };  // first Q / output row

    if (tid == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), kAttWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_launch_dependents();
    // A decode step's work split comes precomputed (the same for all its layers).  From the second layer on
    // it is read before the dependency wait: the kernel that wrote it finished long before any kernel that
    // could still be running now; in the first layer that kernel may still be running, so the wait comes first.
    const bool use_plan = p.plan != nullptr && !packed;
    if (!(use_plan && p.plan_prewait)) pdl_wait();  // sequence lengths, Q and the freshly appended K/V come from earlier kernels of the step
    if (use_plan) {
        if (!p.plan_prewait) pdl_wait();
        for (int i = tid; i <= items; i += blockDim.x) {
            cum[i] = ld_mut(p.plan + i);
            segcum[i] = ld_mut(p.plan + 2 * kAttMaxItems + 1 + i);
            if (i < items) nk_s[i] = ld_mut(p.plan + kAttMaxItems + 1 + i);
        }
    } else if (warp == 0 && !packed) {
        att_plan_warp(lane, items, p.rm, p.seq_len, p.n_kv, (int)gridDim.x, cum, nk_s, segcum);
    }
    __syncthreads();
    if (use_plan && p.plan_prewait) pdl_wait();
    DBT_TL_WAITED;
    const int C = gridDim.x, Sg = packed ? items * p.n_kv : segcum[items] * p.n_kv;  // all segments, ordered (row, KV head, segment)
    DBT_TL_MARK(3);
    if ((int)blockIdx.x >= Sg) return;
    // segment sidx -> its row, KV head, stage range and the pair's segment count
    auto item_nkeys = [&](int i) {
        if (!packed) return nk_s[i];
        return ld_mut(p.seq_len + i / p.nbk) + (i % p.nbk) * p.pack + item_npos(i);
    };
    auto locate = [&](int sidx, int &item, int &g, int &seg, int &n, int &ui, int &t0, int &t1) {
        if (packed) {  // one pass per (tile, KV head) over all its keys
            item = sidx / p.n_kv;
            g = sidx % p.n_kv;
            seg = 0;
            n = 1;
            ui = (item_nkeys(item) + kAttTile - 1) / kAttTile;
            t0 = 0;
            t1 = ui;
            return;
        }
        int lo = 0, hi = items - 1;
        while (lo < hi) {  // largest row whose first segment is <= sidx
            int mid = (lo + hi + 1) >> 1;
            if (segcum[mid] * p.n_kv <= sidx) lo = mid; else hi = mid - 1;
        }
        item = lo;
        n = segcum[item + 1] - segcum[item];
        int rel = sidx - segcum[item] * p.n_kv;
        g = rel / n;
        seg = rel % n;
        ui = cum[item + 1] - cum[item];
        t0 = (int)(((long long)seg * ui) / n);
        t1 = (int)(((long long)(seg + 1) * ui) / n);
    };

    if (warp == kAttWarps) {
        // ---- producer: walks the same segments as the consumers.  Lane 0 waits for the stage and
        // arms its barrier; up to four lanes then issue one box each (a page's K and V, both
        // 64-column pieces: 8 KB at d_h = 128), each after its own page-table lookup.
        if (lane == 0) tma_prefetch_desc(&tmKV);
        const uint64_t pol = l2_evict_first_policy();
        bool ok = true;
        int it = 0;
        for (int sidx = blockIdx.x; sidx < Sg && ok; sidx += C) {
            int item, g, seg, n, ui, t0, t1;
            locate(sidx, item, g, seg, n, ui, t0, t1);
            int seq = item_seq(item), total_pages = (item_nkeys(item) + 15) >> 4;
            // page ids 32 at a time (eight stages' worth, one coalesced load): a lookup per stage would put an
            // L2 round trip on every stage of this loop and cap a CTA at one stage per ~0.7 us
            int pt_base = -(1 << 30), my_page = 0;
            for (int t = t0; t < t1; t++, it++) {
                int s = it % STAGES;
                int p0 = t * 4, np = min(4, total_pages - p0);
                if (p0 + 4 > pt_base + 32) {
                    pt_base = p0;
                    my_page = p0 + lane < total_pages ? __ldg(p.page_table + (size_t)seq * p.pt_stride + p0 + lane) : 0;
                }
                if (lane == 0) {
                    if (it >= STAGES) ok = mbar_wait(empty_bar(s), ((it / STAGES) - 1) & 1);
                    if (ok) mbar_expect_tx(full_bar(s), (uint32_t)np * 2 * Cfg::kPageBytes);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                int page = __shfl_sync(0xffffffffu, my_page, (p0 - pt_base + lane) & 31);
                if (lane < np) {
                    if (page < 0 || page >= p.num_pages) {
                        report(p.status, kStatusBadPage, page);
                        page = 0;
                    }
                    int row = (int)(((long long)page * p.n_kv + g) * 16);
                    if (p.evict_first)
                        tma_load_4d_hint(tiles + s * Cfg::kStageBytes + lane * 2 * Cfg::kPageBytes, &tmKV, full_bar(s), 0, 0,
                                         (int)(p.k_row0 + row), 0, pol);
                    else
                        tma_load_4d(tiles + s * Cfg::kStageBytes + lane * 2 * Cfg::kPageBytes, &tmKV, full_bar(s), 0, 0,
                                    (int)(p.k_row0 + row), 0);
                }
                // After the first two stages the stream pauses until the consumers have their queries: their
                // few small loads would otherwise queue behind hundreds of CTAs' page traffic for several
                // microseconds, and nothing can be consumed before they return anyway.  (Letting the ring fill
                // at once instead, with the small loads issued first, was measured slower: the queries are ready
                // 0.8 us sooner but the stream then runs 10 % slower; pausing after one, two, four or six stages
                // gave 1.0446, 1.0384, 1.0420 and 1.0462 ms per step of the 1B model at batch 16.)
                if (it == kAttPauseAt || (it < kAttPauseAt && sidx + C >= Sg && t == t1 - 1)) asm volatile("bar.sync 2, 160;" ::: "memory");
            }
        }
        if (!ok && lane == 0) report(p.status, kStatusWaitExpired, 300);
        return;
    }

    // ---- consumers
    bool ok = true;
    int it = 0;
    const float qscale = kLog2e / sqrtf((float)DH);
    // The staged copy of the page that holds this step's position was read while the row was being
    // written: overwrite the row in shared memory with the values computed here (16-byte pieces,
    // lanes 0..15 the K row, lanes 16..31 the V row; DH = 64 uses half of each).
    auto patch_new_row = [&](uint32_t kpage, uint32_t vpage, int row) {
        int piece = lane & 15;
        if (piece < DH / 8) {
            int sg = row * HALVES + (piece >> 3);
            uint32_t dst = (lane < 16 ? kpage : vpage) + sg * 128 + (((piece & 7) ^ (sg & 7)) << 4);
            const uint4 v = *reinterpret_cast<const uint4 *>(kv_new + (lane < 16 ? 0 : DH) + piece * 8);
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
        __syncwarp();
    };
    for (int sidx = blockIdx.x; sidx < Sg; sidx += C) {
        int item, g, seg, nseg, ui, t0, t1;
        locate(sidx, item, g, seg, nseg, ui, t0, t1);
        int nkeys = item_nkeys(item);
        if (packed) nq_act = item_npos(item) * p.G;  // rows: position-major, the G heads of each position

        // Query tile (16 rows x DH, fp32) into shared memory, then mma A fragments (bf16),
        // pre-scaled by log2(e)/sqrt(d_h).  Rows: G primary heads, then G coupled branch heads.
        consumer_sync();  // the previous segment is done with the scratch
        const bool owns_last = p.qkv_P != nullptr && seg == nseg - 1;  // this segment ends the pair
        if (p.qkv_P == nullptr) {
            for (int idx = tid; idx < 16 * DH / 4; idx += 128) {
                int q = idx / (DH / 4), c4 = idx % (DH / 4);
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (q < nq_act) {
                    int row = packed ? item_row0(item) + q / p.G : (q / p.G) * Bc + item;
                    int h = g * p.G + q % p.G;
                    v = __ldcg(reinterpret_cast<const float4 *>(p.Q + (size_t)row * q_dim + (size_t)h * DH) + c4);
                }
                reinterpret_cast<float4 *>(sc_o)[idx] = v;
            }
        } else {
            constexpr int half = DH / 2;
            const int kv_dim = p.n_kv * DH, ldp = q_dim + 2 * kv_dim, pos = nkeys - 1;
            const bool grp = P > 1;
            const int twin = grp ? Bc + item : item;  // the first branch's row travels with the primary's loads
            const size_t p1 = (size_t)item * ldp, p2 = (size_t)twin * ldp;
            // One round of loads: the first warp requests the norm shares of the pair's rows (lanes
            // 0..15 the primary row, 16..31 the first branch's) and hands 1/rms to the others through
            // shared memory; every thread requests the partials, the rotation and the coupling of its
            // outputs before anyone waits.  Further decode branches (Appendix C.1) follow in rounds of
            // their own.
            float myss = 0.f;
            if (p.ss && warp == 0)
                for (int t = lane & 15; t < p.ss_tiles; t += 16) myss += __ldcg(p.ss + (size_t)t * p.ss_ld + (lane < 16 ? item : twin));
            for (int idx = tid; idx < (16 - nq_act) * DH / 4; idx += 128)  // unused query rows
                reinterpret_cast<float4 *>(sc_o + (size_t)nq_act * DH)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
            const int nitems = p.G * half;
            const bool do_kv = owns_last && tid < half;
            float *rs_s = reinterpret_cast<float *>(flag + 8);  // [path]
            // the page of this step's position: requested with the first round of loads, used after it
            const int page_new = do_kv ? __ldg(p.page_table + (size_t)p.rm.seq(item) * p.pt_stride + (pos >> 4)) : 0;
            float rs1 = 1.f, rs2 = 1.f, kvs[4] = {0.f, 0.f, 0.f, 0.f};
            float2 t_kv = make_float2(1.f, 0.f);
            for (int it0 = 0; it0 * 128 < nitems; it0++) {
                int idx = it0 * 128 + tid;
                bool act = idx < nitems;
                int j = act ? idx / half : 0, i = act ? idx % half : tid % half;
                int o0 = (g * p.G + j) * DH + i, o1 = o0 + half;
                float2 t = p.rope[(size_t)pos * half + i];
                float ca0 = grp ? p.coup_a[o0] : 0.f, ca1 = grp ? p.coup_a[o1] : 0.f;
                const size_t offs[4] = {p1 + o0, p1 + o1, p2 + o0, p2 + o1};
                float sm[4] = {0.f, 0.f, 0.f, 0.f};
                if (act) sum_splits_k<4, 12>(p.qkv_P, p.qkv_stride, p.qkv_nsplit, offs, sm);
                if (it0 == 0) {
                    if (do_kv) {  // K_1 and V_1 of this step's token for this KV head (tid = rotation pair)
                        size_t ko = p1 + q_dim + (size_t)g * DH + tid, vo = ko + kv_dim;
                        const size_t koffs[4] = {ko, ko + half, vo, vo + half};
                        sum_splits_k<4, 12>(p.qkv_P, p.qkv_stride, p.qkv_nsplit, koffs, kvs);
                        t_kv = t;  // idx = tid < half in the first round: the same rotation pair
                    }
                    if (warp == 0) {
                        sc_m[lane] = myss;  // sc_m[0..15], sc_l[0..15] are contiguous
                        __syncwarp();
                        if ((lane & 15) == 0) {
                            float a = 0.f;
                            for (int k = 0; k < 16; k++) a += sc_m[lane + k];
                            rs_s[lane >> 4] = p.ss ? 1.f / sqrtf(a / (float)p.d_norm + p.eps) : 1.f;
                        }
                        for (int jp = 2; jp < P; jp++) {  // further branches: the whole warp per row
                            float a = 0.f;
                            if (p.ss)
                                for (int t2 = lane; t2 < p.ss_tiles; t2 += 32) a += __ldcg(p.ss + (size_t)t2 * p.ss_ld + jp * Bc + item);
                            sc_m[lane] = a;
                            __syncwarp();
                            if (lane == 0) {
                                float tot = 0.f;
                                for (int k = 0; k < 32; k++) tot += sc_m[k];
                                rs_s[jp] = p.ss ? 1.f / sqrtf(tot / (float)p.d_norm + p.eps) : 1.f;
                            }
                            __syncwarp();
                        }
                    }
                    consumer_sync();
                    rs1 = rs_s[0];
                    rs2 = rs_s[1];
                }
                if (act) {
                    float x0 = rs1 * sm[0], x1 = rs1 * sm[1];
                    float r0 = x0 * t.x - x1 * t.y, r1 = x1 * t.x + x0 * t.y;
                    sc_o[(size_t)j * DH + i] = r0;
                    sc_o[(size_t)j * DH + i + half] = r1;
                    if (grp) {
                        float y0 = rs2 * sm[2], y1 = rs2 * sm[3];
                        sc_o[(size_t)(p.G + j) * DH + i] = (y0 * t.x - y1 * t.y) + ca0 * r0;
                        sc_o[(size_t)(p.G + j) * DH + i + half] = (y1 * t.x + y0 * t.y) + ca1 * r1;
                    }
                    for (int jp = 2; jp < P; jp++) {  // Q~_j = Q_j + a * Q_1 for the further branches
                        const size_t pj = (size_t)(jp * Bc + item) * ldp;
                        const size_t offj[2] = {pj + o0, pj + o1};
                        float sj[2];
                        sum_splits_k<2, 12>(p.qkv_P, p.qkv_stride, p.qkv_nsplit, offj, sj);
                        const float rsj = rs_s[jp];
                        float y0 = rsj * sj[0], y1 = rsj * sj[1];
                        sc_o[(size_t)(jp * p.G + j) * DH + i] = (y0 * t.x - y1 * t.y) + ca0 * r0;
                        sc_o[(size_t)(jp * p.G + j) * DH + i + half] = (y1 * t.x + y0 * t.y) + ca1 * r1;
                    }
                }
            }
            if (do_kv) {
                // K_1 = RoPE(N_1 W_K), V_1 = N_1 W_V: to the staging row for the patch and to the pool
                int i = tid;
                float x0 = rs1 * kvs[0], x1 = rs1 * kvs[1];
                __nv_bfloat16 k0 = __float2bfloat16_rn(x0 * t_kv.x - x1 * t_kv.y), k1 = __float2bfloat16_rn(x1 * t_kv.x + x0 * t_kv.y);
                __nv_bfloat16 v0 = __float2bfloat16_rn(rs1 * kvs[2]), v1 = __float2bfloat16_rn(rs1 * kvs[3]);
                kv_new[i] = k0;
                kv_new[i + half] = k1;
                kv_new[DH + i] = v0;
                kv_new[DH + i + half] = v1;
                const int page = page_new;
                if (page < 0 || page >= p.num_pages) {
                    if (i == 0) report(p.status, kStatusBadPage, page);
                } else {
                    size_t base = (((size_t)page * p.n_kv + g) * 16 + (pos & 15)) * DH;
                    p.kpool[base + i] = k0;
                    p.kpool[base + i + half] = k1;
                    p.vpool[base + i] = v0;
                    p.vpool[base + i + half] = v1;
                }
            }
        }
        consumer_sync();
        if (sidx == (int)blockIdx.x) {
            asm volatile("bar.arrive 2, 160;" ::: "memory");  // the producer may stream on
            DBT_TL_MARK(0);
        }
        int pair = item * p.n_kv + g;
        int first_slot = sidx - seg;  // the pair's segments occupy consecutive partial slots
        float *out = p.part + (size_t)sidx * 16 * (DH + 2);
        if constexpr (!NARROW) {
            uint32_t qa[KS][4];
            {
                int r0 = lane >> 2, c = (lane & 3) * 2;
                const float *q0 = sc_o + r0 * DH, *q1 = sc_o + (r0 + 8) * DH;
    #pragma unroll
                for (int ks = 0; ks < KS; ks++) {
                    int k = ks * 16 + c;
                    qa[ks][0] = pack_bf16(q0[k] * qscale, q0[k + 1] * qscale);
                    qa[ks][1] = pack_bf16(q1[k] * qscale, q1[k + 1] * qscale);
                    qa[ks][2] = pack_bf16(q0[k + 8] * qscale, q0[k + 9] * qscale);
                    qa[ks][3] = pack_bf16(q1[k + 8] * qscale, q1[k + 9] * qscale);
                }
            }
            consumer_sync();  // everyone has its fragments: the scratch is free again
            float o[NB][4];
    #pragma unroll
            for (int nb = 0; nb < NB; nb++) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
            float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

            for (int t = t0; t < t1 && ok; t++, it++) {
                int s = it % STAGES;
                ok = mbar_wait(full_bar(s), (it / STAGES) & 1);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                int valid = min(16, nkeys - (t * kAttTile + warp * 16));  // valid tokens in this warp's page
                if (valid > 0) {
                    // a page's box: K then V, each [16 rows][DH], the 128-byte pieces of a row swizzled
                    uint32_t kpage = tiles + s * Cfg::kStageBytes + warp * 2 * Cfg::kPageBytes;
                    uint32_t vpage = kpage + Cfg::kPageBytes;
                    if (valid < 16) {
                        // stale slots past the end of the sequence: their scores are masked below, and
                        // their V rows are zeroed here so that 0 * garbage cannot produce a NaN
                        for (int idx = lane; idx < (16 - valid) * HALVES * 8; idx += 32) {
                            uint32_t a = vpage + valid * HALVES * 128 + idx * 16;
                            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                        }
                        __syncwarp();
                    }
                    if (owns_last && t == ui - 1 && ((nkeys - 1) >> 4 & 3) == warp) patch_new_row(kpage, vpage, (nkeys - 1) & 15);
                // S = Q K^T for this warp's 16 tokens: two 8-token column blocks
                    float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                    {
                        int r = (lane & 7) + ((lane >> 4) << 3);  // token row this lane addresses
                        int cb = (lane >> 3) & 1;                 // which 8-dim chunk of the k-step
    #pragma unroll
                        for (int ks = 0; ks < KS; ks++) {
                            int chunk = ks * 2 + cb;  // 16-byte chunk index within the row
                            int sg = r * HALVES + (chunk >> 3);
                            uint32_t a = kpage + sg * 128 + (((chunk & 7) ^ (sg & 7)) << 4);
                            uint32_t kb[4];
                            ldsm_x4(a, kb);
                            mma_bf16(sacc[0], qa[ks], kb[0], kb[1]);
                            mma_bf16(sacc[1], qa[ks], kb[2], kb[3]);
                        }
                    }
                    // mask, online softmax (base 2), pack P as the A operand of P V
                    int col = (lane & 3) * 2;
                    float rmax[2] = {-INFINITY, -INFINITY};
                    // packed prompt tiles: the row of position pp sees the keys up to its own position only
                    int vrow[2] = {valid, valid};
                    if (packed) {
                        const int npos = nq_act / p.G, rem = nkeys - (t * kAttTile + warp * 16);
    #pragma unroll
                        for (int h = 0; h < 2; h++) vrow[h] = min(16, rem - max(npos - 1 - ((lane >> 2) + 8 * h) / p.G, 0));
                    }
    #pragma unroll
                    for (int nb = 0; nb < 2; nb++)
    #pragma unroll
                        for (int e = 0; e < 4; e++) {
                            int tk = nb * 8 + col + (e & 1);
                            if (tk >= vrow[e >> 1]) sacc[nb][e] = -INFINITY;
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
                            int sg = r * HALVES + (chunk >> 3);
                            uint32_t a = vpage + sg * 128 + (((chunk & 7) ^ (sg & 7)) << 4);
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
            if (!ok) {
                // a ring that stopped filling stops for all four warps: every consumer leaves here
                if (lane == 0) report(p.status, kStatusWaitExpired, 310 + warp);
                return;
            }

            // ---- fold the four warps' states, (0+2) + (1+3), in registers through the one-slot
            // scratch; warp 0 then writes this segment's partial
            {
                int r0 = lane >> 2, c = (lane & 3) * 2;
                auto put = [&]() {
    #pragma unroll
                    for (int nb = 0; nb < NB; nb++) {
                        *reinterpret_cast<float2 *>(sc_o + (size_t)r0 * FS + nb * 8 + c) = make_float2(o[nb][0], o[nb][1]);
                        *reinterpret_cast<float2 *>(sc_o + (size_t)(r0 + 8) * FS + nb * 8 + c) = make_float2(o[nb][2], o[nb][3]);
                    }
                    if ((lane & 3) == 0) {
                        sc_m[r0] = m_run[0];
                        sc_m[r0 + 8] = m_run[1];
                        sc_l[r0] = l_run[0];
                        sc_l[r0 + 8] = l_run[1];
                    }
                };
                auto take = [&]() {  // this warp's state := this warp's state (+) the slot's state
    #pragma unroll
                    for (int h = 0; h < 2; h++) {
                        int r = r0 + 8 * h;
                        float mb = sc_m[r], lb = sc_l[r];
                        float M = fmaxf(m_run[h], mb);
                        float fa = m_run[h] == -INFINITY ? 0.f : exp2f(m_run[h] - M);
                        float fb = mb == -INFINITY ? 0.f : exp2f(mb - M);
                        l_run[h] = l_run[h] * fa + lb * fb;
                        m_run[h] = M;
    #pragma unroll
                        for (int nb = 0; nb < NB; nb++) {
                            float2 ob = *reinterpret_cast<const float2 *>(sc_o + (size_t)r * FS + nb * 8 + c);
                            o[nb][2 * h] = o[nb][2 * h] * fa + ob.x * fb;
                            o[nb][2 * h + 1] = o[nb][2 * h + 1] * fa + ob.y * fb;
                        }
                    }
                };
                for (int step = 0; step < 3; step++) {  // 2 -> 0, 3 -> 1, 1 -> 0
                    int src = step == 0 ? 2 : step == 1 ? 3 : 1, dst = step == 1 ? 1 : 0;
                    if (warp == src) put();
                    consumer_sync();
                    if (warp == dst) take();
                    consumer_sync();
                }
                if (warp == 0) {
    #pragma unroll
                    for (int h = 0; h < 2; h++) {
                        int q = r0 + 8 * h;
                        if (q < nq_act) {
                            if (nseg == 1) {
                                // the pair's only segment: normalise and write the head's output
                                int row = packed ? item_row0(item) + q / p.G : (q / p.G) * Bc + item;
                                int hq = g * p.G + q % p.G;
                                size_t ob = (size_t)row * q_dim + (size_t)hq * DH;
                                float inv = 1.f / l_run[h];
    #pragma unroll
                                for (int nb = 0; nb < NB; nb++)
    #pragma unroll
                                    for (int e = 0; e < 2; e++) {
                                        float x = o[nb][2 * h + e] * inv;
                                        __nv_bfloat16 hi = __float2bfloat16_rn(x);
                                        p.Ob[ob + nb * 8 + c + e] = hi;
                                        if (p.lo_off) p.Ob[ob + nb * 8 + c + e + p.lo_off] = __float2bfloat16_rn(x - __bfloat162float(hi));
                                    }
                            } else {
    #pragma unroll
                                for (int nb = 0; nb < NB; nb++)
                                    *reinterpret_cast<float2 *>(out + (size_t)q * (DH + 2) + nb * 8 + c) =
                                        make_float2(o[nb][2 * h], o[nb][2 * h + 1]);
                                if ((lane & 3) == 0) {
                                    out[(size_t)q * (DH + 2) + DH] = m_run[h];  // base-2 units
                                    out[(size_t)q * (DH + 2) + DH + 1] = l_run[h];
                                }
                            }
                        }
                    }
                    if (nseg > 1) __threadfence();
                }
            }
        } else {
            // ---- narrow variant: at most 8 query rows per KV head.  The products are taken transposed,
            // S^T = K Q^T and O^T = V^T P^T, so that the 16 keys of a page fill the M side of
            // m16n8k16 and the (few) queries sit on the 8-wide N side: half the MMAs and half the
            // accumulators of the 16-query form.
            uint32_t qb[KS][2];
            {
                int n = lane >> 2, c = (lane & 3) * 2;
                const float *q0 = sc_o + n * DH;
#pragma unroll
                for (int ks = 0; ks < KS; ks++) {
                    int k = ks * 16 + c;
                    qb[ks][0] = pack_bf16(q0[k] * qscale, q0[k + 1] * qscale);
                    qb[ks][1] = pack_bf16(q0[k + 8] * qscale, q0[k + 9] * qscale);
                }
            }
            consumer_sync();  // everyone has its fragments: the scratch is free again
            constexpr int MB = DH / 16;  // 16-row blocks of O^T
            float o[MB][4];
#pragma unroll
            for (int mb = 0; mb < MB; mb++) o[mb][0] = o[mb][1] = o[mb][2] = o[mb][3] = 0.f;
            // per query column (2t, 2t+1): running max (same in the 8 lanes of a column) and this
            // lane's share of the running sum (reduced over the lanes once, after the loop)
            float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
            const int g8 = lane >> 2;

            for (int t = t0; t < t1 && ok; t++, it++) {
                int s = it % STAGES;
                ok = mbar_wait(full_bar(s), (it / STAGES) & 1);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                int valid = min(16, nkeys - (t * kAttTile + warp * 16));  // valid tokens in this warp's page
                if (valid > 0) {
                    uint32_t kpage = tiles + s * Cfg::kStageBytes + warp * 2 * Cfg::kPageBytes;
                    uint32_t vpage = kpage + Cfg::kPageBytes;
                    if (valid < 16) {
                        for (int idx = lane; idx < (16 - valid) * HALVES * 8; idx += 32) {
                            uint32_t a = vpage + valid * HALVES * 128 + idx * 16;
                            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                        }
                        __syncwarp();
                    }
                    if (owns_last && t == ui - 1 && ((nkeys - 1) >> 4 & 3) == warp) patch_new_row(kpage, vpage, (nkeys - 1) & 15);
                    // S^T = K Q^T: K rows as the A operand
                    float sacc[4] = {0.f, 0.f, 0.f, 0.f};
                    {
                        int r = (lane & 7) + (((lane >> 3) & 1) << 3);  // key row this lane addresses
                        int cb = lane >> 4;                              // which 8-dim chunk of the k-step
#pragma unroll
                        for (int ks = 0; ks < KS; ks++) {
                            int chunk = ks * 2 + cb;
                            int sg = r * HALVES + (chunk >> 3);
                            uint32_t a = kpage + sg * 128 + (((chunk & 7) ^ (sg & 7)) << 4);
                            uint32_t ka[4];
                            ldsm_x4(a, ka);
                            mma_bf16(sacc, ka, qb[ks][0], qb[ks][1]);
                        }
                    }
                    // sacc: keys g8, g8+8 (rows) x queries 2t, 2t+1 (columns)
                    if (valid < 16) {
                        if (g8 >= valid) sacc[0] = sacc[1] = -INFINITY;
                        if (g8 + 8 >= valid) sacc[2] = sacc[3] = -INFINITY;
                    }
                    float rmax[2] = {fmaxf(sacc[0], sacc[2]), fmaxf(sacc[1], sacc[3])};
                    float corr[2], msub[2];
#pragma unroll
                    for (int j = 0; j < 2; j++) {
                        rmax[j] = fmaxf(rmax[j], __shfl_xor_sync(0xffffffffu, rmax[j], 4));
                        rmax[j] = fmaxf(rmax[j], __shfl_xor_sync(0xffffffffu, rmax[j], 8));
                        rmax[j] = fmaxf(rmax[j], __shfl_xor_sync(0xffffffffu, rmax[j], 16));
                        float mnew = fmaxf(m_run[j], rmax[j]);
                        msub[j] = mnew == -INFINITY ? 0.f : mnew;
                        corr[j] = m_run[j] == -INFINITY ? 0.f : exp2f(m_run[j] - msub[j]);
                        m_run[j] = mnew;
                    }
                    float p0 = exp2f(sacc[0] - msub[0]), p1 = exp2f(sacc[1] - msub[1]);
                    float p2 = exp2f(sacc[2] - msub[0]), p3 = exp2f(sacc[3] - msub[1]);
                    l_run[0] = l_run[0] * corr[0] + (p0 + p2);
                    l_run[1] = l_run[1] * corr[1] + (p1 + p3);
                    // P^T as the B operand of O^T += V^T P^T: transpose the two 8x8 blocks across the warp
                    uint32_t pb0 = movmatrix_trans(pack_bf16(p0, p1)), pb1 = movmatrix_trans(pack_bf16(p2, p3));
                    if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
                        for (int mb = 0; mb < MB; mb++) {
                            o[mb][0] *= corr[0];
                            o[mb][1] *= corr[1];
                            o[mb][2] *= corr[0];
                            o[mb][3] *= corr[1];
                        }
                    }
                    {
                        int r = (lane & 7) + ((lane >> 4) << 3);  // key row
                        int cb = (lane >> 3) & 1;                 // which 8-dim half of the 16-dim block
#pragma unroll
                        for (int mb = 0; mb < MB; mb++) {
                            int chunk = mb * 2 + cb;
                            int sg = r * HALVES + (chunk >> 3);
                            uint32_t a = vpage + sg * 128 + (((chunk & 7) ^ (sg & 7)) << 4);
                            uint32_t va[4];
                            ldsm_x4_trans(a, va);
                            mma_bf16(o[mb], va, pb0, pb1);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(s)) : "memory");
            }
            if (!ok) {
                if (lane == 0) report(p.status, kStatusWaitExpired, 310 + warp);
                return;
            }
#pragma unroll
            for (int j = 0; j < 2; j++) {  // the lanes' shares of the running sums
                l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 4);
                l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 8);
                l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 16);
            }
            // ---- fold the four warps' states, (0+2) + (1+3), through the scratch ([8 queries][DH + 4])
            {
                constexpr int FN = DH + 4;
                int c = (lane & 3) * 2;
                auto put = [&]() {
#pragma unroll
                    for (int mb = 0; mb < MB; mb++) {
                        sc_o[(size_t)c * FN + mb * 16 + g8] = o[mb][0];
                        sc_o[(size_t)(c + 1) * FN + mb * 16 + g8] = o[mb][1];
                        sc_o[(size_t)c * FN + mb * 16 + g8 + 8] = o[mb][2];
                        sc_o[(size_t)(c + 1) * FN + mb * 16 + g8 + 8] = o[mb][3];
                    }
                    if (g8 == 0) {
                        sc_m[c] = m_run[0];
                        sc_m[c + 1] = m_run[1];
                        sc_l[c] = l_run[0];
                        sc_l[c + 1] = l_run[1];
                    }
                };
                auto take = [&]() {
                    float fa[2], fb[2];
#pragma unroll
                    for (int j = 0; j < 2; j++) {
                        float mb2 = sc_m[c + j], lb = sc_l[c + j];
                        float M = fmaxf(m_run[j], mb2);
                        fa[j] = m_run[j] == -INFINITY ? 0.f : exp2f(m_run[j] - M);
                        fb[j] = mb2 == -INFINITY ? 0.f : exp2f(mb2 - M);
                        l_run[j] = l_run[j] * fa[j] + lb * fb[j];
                        m_run[j] = M;
                    }
#pragma unroll
                    for (int mb = 0; mb < MB; mb++) {
                        o[mb][0] = o[mb][0] * fa[0] + sc_o[(size_t)c * FN + mb * 16 + g8] * fb[0];
                        o[mb][1] = o[mb][1] * fa[1] + sc_o[(size_t)(c + 1) * FN + mb * 16 + g8] * fb[1];
                        o[mb][2] = o[mb][2] * fa[0] + sc_o[(size_t)c * FN + mb * 16 + g8 + 8] * fb[0];
                        o[mb][3] = o[mb][3] * fa[1] + sc_o[(size_t)(c + 1) * FN + mb * 16 + g8 + 8] * fb[1];
                    }
                };
                for (int step = 0; step < 3; step++) {  // 2 -> 0, 3 -> 1, 1 -> 0
                    int src = step == 0 ? 2 : step == 1 ? 3 : 1, dst = step == 1 ? 1 : 0;
                    if (warp == src) put();
                    consumer_sync();
                    if (warp == dst) take();
                    consumer_sync();
                }
                if (warp == 0) {
#pragma unroll
                    for (int j = 0; j < 2; j++) {
                        int q = c + j;
                        if (q < nq_act) {
                            if (nseg == 1) {
                                int row = packed ? item_row0(item) + q / p.G : (q / p.G) * Bc + item;
                                int hq = g * p.G + q % p.G;
                                size_t ob = (size_t)row * q_dim + (size_t)hq * DH;
                                float inv = 1.f / l_run[j];
#pragma unroll
                                for (int mb = 0; mb < MB; mb++)
#pragma unroll
                                    for (int e = 0; e < 2; e++) {
                                        float x = o[mb][2 * e + j] * inv;
                                        size_t oi = ob + mb * 16 + g8 + 8 * e;
                                        __nv_bfloat16 hi = __float2bfloat16_rn(x);
                                        p.Ob[oi] = hi;
                                        if (p.lo_off) p.Ob[oi + p.lo_off] = __float2bfloat16_rn(x - __bfloat162float(hi));
                                    }
                            } else {
#pragma unroll
                                for (int mb = 0; mb < MB; mb++) {
                                    out[(size_t)q * (DH + 2) + mb * 16 + g8] = o[mb][j];
                                    out[(size_t)q * (DH + 2) + mb * 16 + g8 + 8] = o[mb][2 + j];
                                }
                                if (g8 == 0) {
                                    out[(size_t)q * (DH + 2) + DH] = m_run[j];  // base-2 units
                                    out[(size_t)q * (DH + 2) + DH + 1] = l_run[j];
                                }
                            }
                        }
                    }
                    if (nseg > 1) __threadfence();
                }
            }
        }
        if (sidx == (int)blockIdx.x) DBT_TL_MARK(1);
        // ---- merging a pair's segments.  Up to kAttSingle segments: the last one to arrive merges them
        // all, in segment order, and writes the output.  More: the segments form groups of kAttGroup;
        // the last arrival of a group merges it in place into the group's first slot, and the last
        // group to finish merges the group results: two short merges on several CTAs instead of one
        // long one on a single CTA (a pair of a 32k-token sequence has ~35 segments).
        // merge n partials at slots pbase + j * slot_stride; final: normalise and write the output,
        // else leave the merged (unnormalised) state in the first slot
        auto merge = [&](float *pbase, int slot_stride, int n, bool final) {
            const size_t sstr = (size_t)slot_stride * 16 * (DH + 2);
            for (int idx0 = tid; idx0 < nq_act * DH; idx0 += 2 * 128) {
                // two outputs per thread, eight partials of each in flight
                const float *pq[2];
                float M[2] = {-INFINITY, -INFINITY}, L[2] = {0.f, 0.f}, X[2] = {0.f, 0.f};
                bool act[2];
                int ee[2], qq[2];
#pragma unroll
                for (int a = 0; a < 2; a++) {
                    int idx = idx0 + a * 128;
                    act[a] = idx < nq_act * DH;
                    qq[a] = act[a] ? idx / DH : 0;
                    ee[a] = act[a] ? idx % DH : 0;
                    pq[a] = pbase + (size_t)qq[a] * (DH + 2);
                }
                for (int sb = 0; sb < n; sb += 8) {
                    float mv[2][8], lv[2][8], ov[2][8];
#pragma unroll
                    for (int a = 0; a < 2; a++)
#pragma unroll
                        for (int j = 0; j < 8; j++) {
                            bool on = act[a] && sb + j < n;
                            const float *pp = pq[a] + (size_t)(sb + j) * sstr;
                            mv[a][j] = on ? __ldcg(pp + DH) : -INFINITY;
                            lv[a][j] = on ? __ldcg(pp + DH + 1) : 0.f;
                            ov[a][j] = on ? __ldcg(pp + ee[a]) : 0.f;
                        }
#pragma unroll
                    for (int a = 0; a < 2; a++) {
                        float Mn = M[a];
#pragma unroll
                        for (int j = 0; j < 8; j++) Mn = fmaxf(Mn, mv[a][j]);
                        float sc = M[a] == -INFINITY ? 0.f : exp2f(M[a] - Mn);
                        L[a] *= sc;
                        X[a] *= sc;
#pragma unroll
                        for (int j = 0; j < 8; j++) {
                            float f = mv[a][j] == -INFINITY ? 0.f : exp2f(mv[a][j] - Mn);
                            L[a] = fmaf(lv[a][j], f, L[a]);
                            X[a] = fmaf(ov[a][j], f, X[a]);
                        }
                        M[a] = Mn;
                    }
                }
#pragma unroll
                for (int a = 0; a < 2; a++) {
                    if (!act[a]) continue;
                    if (final) {
                        int row = packed ? item_row0(item) + qq[a] / p.G : (qq[a] / p.G) * Bc + item;
                        int h = g * p.G + qq[a] % p.G;
                        size_t o_idx = (size_t)row * q_dim + (size_t)h * DH + ee[a];
                        float x = X[a] / L[a];
                        __nv_bfloat16 hi = __float2bfloat16_rn(x);
                        p.Ob[o_idx] = hi;
                        if (p.lo_off) p.Ob[o_idx + p.lo_off] = __float2bfloat16_rn(x - __bfloat162float(hi));
                    } else {
                        // this thread is the only reader of the first slot's element (q, e)
                        pbase[(size_t)qq[a] * (DH + 2) + ee[a]] = X[a];
                        if (ee[a] == 0) {
                            sc_m[qq[a]] = M[a];
                            sc_l[qq[a]] = L[a];
                        }
                    }
                }
            }
            if (!final) {
                consumer_sync();  // every thread has read the first slot's (m, l): now they may change
                if (tid < nq_act) {
                    pbase[(size_t)tid * (DH + 2) + DH] = sc_m[tid];
                    pbase[(size_t)tid * (DH + 2) + DH + 1] = sc_l[tid];
                }
                __threadfence();
            }
        };
        auto arrive = [&](int *counter, int arrivals) {  // true in the CTA that arrives last
            consumer_sync();
            if (tid == 0) {
                int tkt = atomicAdd(counter, 1);
                int last = tkt == arrivals - 1;
                if (last) {
                    atomicExch(counter, 0);
                    __threadfence();
                }
                flag[0] = last;
            }
            consumer_sync();
            return flag[0] != 0;
        };
        if (nseg > 1) {
            float *slot0 = p.part + (size_t)first_slot * 16 * (DH + 2);
            if (nseg <= kAttSingle) {
                if (arrive(p.tickets + pair, nseg)) merge(slot0, 1, nseg, true);
            } else {
                int gi = seg / kAttGroup, ngroups = (nseg + kAttGroup - 1) / kAttGroup;
                int gs = min(kAttGroup, nseg - gi * kAttGroup);
                if (arrive(p.tickets2 + (size_t)pair * kAttMaxGroups + gi, gs)) {
                    merge(slot0 + (size_t)gi * kAttGroup * 16 * (DH + 2), 1, gs, false);
                    if (arrive(p.tickets + pair, ngroups)) merge(slot0, kAttGroup, ngroups, true);
                }
            }
        }
        if (sidx == (int)blockIdx.x) DBT_TL_MARK(2);
    }
#ifdef DBT_TL_ATT_ALL
    {  // every CTA leaves a record: mark 3 carries (SM id << 16 | block index)
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        tlx_[3] = ((unsigned long long)smid << 16) | blockIdx.x;
    }
    DBT_TL_END_IF(true, "attall");
#else
    DBT_TL_END("attentio");
#endif
}

// The K/V pool as a 4-D bf16 tensor (64 columns, 64-column piece of a row, row, K|V plane of a
// layer); rows = (layer, K|V, page, head, slot).  One box {64, d_h/64, 16, 2} brings a page's K and V
// of one KV head.  The row extent stops one plane short so that plane 1 of the last layer stays
// inside the allocation.
inline bool make_kv_page_map(CUtensorMap *map, const void *pool, uint64_t total_rows, uint64_t plane_rows, int head_dim) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || total_rows >= (1ull << 31) || total_rows <= plane_rows) return false;
    cuuint64_t dims[4] = {64, (cuuint64_t)head_dim / 64, total_rows - plane_rows, 2};
    cuuint64_t strides[3] = {128, (cuuint64_t)head_dim * 2, plane_rows * (cuuint64_t)head_dim * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)head_dim / 64, 16, 2};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(pool), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace dbt
