// The whole grouped decode step of a dense bf16 model as ONE persistent kernel (sm_100a).
//
// Why: run as separate kernels, a layer is ten launches of a few microseconds each, and the
// dependency latency between them (grid drain, flush, wake-up of the next grid) costs more
// than the kernels themselves at small batch.  Here one CTA per SM stays resident for the
// whole step; the phases of a layer are separated by grid barriers (an arrival counter in
// global memory, every wait bounded), and a single producer warp per CTA streams, through one
// shared-memory ring, everything the step reads from HBM in program order: the weight tiles
// of the Q|K|V GEMM, the K/V pages of the attention, the weight tiles of the O, gate|up and
// down GEMMs, the next layer's..., and finally the output matrix.  Weight tiles do not depend
// on activations, so the producer runs ahead of the barriers and the ring is full when a GEMM
// phase begins; only the (small, L2-resident) activation tiles wait for the barrier.
//
// Roles (320 threads): warp 0 = producer (TMA), warp 1 = tcgen05 MMA issuer and TMEM owner,
// warps 2..9 = workers (GEMM epilogues out of tensor memory, the elementwise phases, the
// attention math with mma.sync: two groups of four warps take alternate 64-token stages).
//
// Every phase is a dependency hop of a few L2 round trips, so the elementwise phases are written
// to put all their loads in flight at once (partials of several outputs gathered together, row
// scales and per-sequence positions staged in shared memory) instead of chasing them one by one.
//
// GEMM phases are split "stream-K": all (tile, k-tile) units of a GEMM are laid end to end
// and CTA c takes units [c*q, (c+1)*q): every SM streams the same number of weight bytes
// whatever the shape.  A CTA's run of units inside one 128-feature tile is a segment; its
// partial tile goes to slot c + tile, and the elementwise phase after the barrier adds a
// tile's segments in CTA order (deterministic, and identical for grouped and primary-only
// steps because q depends on the shape only).  RMSNorm is split around the GEMMs: the gain
// is folded into the GEMM input, sum(S^2) is kept as per-block shares, and the phase after
// the GEMM multiplies by 1/rms.
//
// Phases per layer (Section 4.1, Eq. asymattn, Eq. mlp):
//   G1 Q|K|V  | E1 1/rms, RoPE, Q~_2 = Q_2 + a*Q_1, append K_1,V_1 | A attention (both paths'
//   queries on one pass over the pages) | G2 O | E2 S-bar = S + ., next input | G3 gate|up |
//   E3 SiLU*up, H~_2 = H_2 + b*H_1 | G4 down | E4 M_2 += c*M_1, S += M, next input
// then the output matrix and the readout (Eq. alpha, Eq. mixloss) spread over all CTAs.
#pragma once

#include "dbt_attn_mma.cuh"
#include "dbt_fused.cuh"
#include "dbt_kernels.cuh"

namespace dbt {

constexpr int kMegaMaxLayers = 128;
constexpr int kMegaSlots = 6;
constexpr int kMegaSlotBytes = 32768;
constexpr int kMegaWorkerWarps = 8;
constexpr int kMegaWorkers = kMegaWorkerWarps * 32;
constexpr int kMegaThreads = 64 + kMegaWorkers;
constexpr int kMegaMaxCtas = 160;
constexpr int kMegaAcc = 4;  // independent TMEM accumulators per segment (one per k16 step of a stage)
constexpr unsigned long long kMegaWaitCycles = 4000000000ull;

struct MegaLayer {
    const float *coup_a, *coup_b, *coup_c, *g_mlp, *g_next;  // g_next: gain folded into the input after this layer
};

struct MegaPlan {
    int B, grouped, R, L, d, n_q, n_kv, dh, F, V, Rmax, final_norm;
    int num_pages, pt_stride;
    float eps;
    float *S, *Q, *P, *ss, *Z, *part, *rd_part, *rd_best;
    __nv_bfloat16 *Xb, *Ob, *Hb, *pool;
    size_t lo_x, lo_o, lo_h;  // element offset of the lo plane of each GEMM input
    const float2 *rope;
    int32_t *seq_len;
    const int32_t *page_table;
    int *att_tickets, *status;
    unsigned int *bar_count, *done_count;
    int *err;
    const CUtensorMap *maps;  // per layer wq wk wv wo wg wu wd; then lm_head, K/V pages, and per row-tile width 16/32/64: Xb, Ob, Hb
    const __nv_bfloat16 *E1, *E2;
    const float *g_e, *g_first;
    long long plane_rows;  // rows of one K (or V) plane of one layer in the pool's 2-D view
    MegaLayer layer[kMegaMaxLayers];
};

template <int N_TILE, int DH>
struct MegaCfg {
    static constexpr int kBBytes = N_TILE * kTcK * 2;
    static constexpr int kScratchBytes = 2 * 16 * (DH + 8) * 4 + 12288;  // includes the debug timestamps
    static constexpr int kSmemBytes = kMegaSlots * kMegaSlotBytes + 1024 + 256 + kScratchBytes;
    static_assert(kTcABytes + 2 * kBBytes <= kMegaSlotBytes, "GEMM stage must fit a ring slot");
    static_assert(2 * 4 * 16 * DH * 2 <= kMegaSlotBytes, "attention stage must fit a ring slot");
};

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// stream-K bookkeeping of one GEMM phase
struct MegaGemm {
    const CUtensorMap *w[3], *x;
    int n_out[3], nseg, K, tiles, KT, U, q, lo_row0;
};

// Sums of K outputs' segment partials (each in CTA order), with the loads of all K outputs and of
// NB segments in flight together: one L2 round trip per NB segments instead of one per load.
template <int N_TILE, int K, int NB>
__device__ __forceinline__ void mega_gather(const float *P, const MegaGemm &g, const int (&tile)[K], const int (&row)[K],
                                            const int (&feat)[K], float (&out)[K]) {
    const float *p[K];
    int n[K], nmax = 0;
#pragma unroll
    for (int k = 0; k < K; k++) {
        int first = (tile[k] * g.KT) / g.q, last = ((tile[k] + 1) * g.KT - 1) / g.q;
        p[k] = P + ((size_t)(first + tile[k]) * N_TILE + row[k]) * 128 + feat[k];
        n[k] = last - first + 1;
        nmax = max(nmax, n[k]);
        out[k] = 0.f;
    }
    for (int j = 0; j < nmax; j += NB) {
        float v[NB][K];
#pragma unroll
        for (int jj = 0; jj < NB; jj++)
#pragma unroll
            for (int k = 0; k < K; k++)
                v[jj][k] = (j + jj < n[k]) ? __ldcg(p[k] + (size_t)(j + jj) * (N_TILE * 128)) : 0.f;
#pragma unroll
        for (int jj = 0; jj < NB; jj++)
#pragma unroll
            for (int k = 0; k < K; k++) out[k] += v[jj][k];
    }
}

template <int N_TILE, int DH>
__global__ void __launch_bounds__(kMegaThreads, 1)
mega_decode_kernel(const MegaPlan *__restrict__ pl, const int32_t *tokens, int32_t *next, float *alpha_out) {
    using Cfg = MegaCfg<N_TILE, DH>;
    constexpr int SLOTS = kMegaSlots, HALVES = DH / 64, KS = DH / 16, NB = DH / 8;
    constexpr int PAGE_BYTES = 16 * DH * 2;
    constexpr int SLOT_FLOATS = N_TILE * 128;  // one partial tile [N_TILE rows][128 features]
    constexpr int NW = kMegaWorkers;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t *gen_ring = smem_raw + (ring - raw);
    const uint32_t bars = ring + SLOTS * kMegaSlotBytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (SLOTS + s); };
    auto accf_bar = [&](int b) { return bars + 8u * (2 * SLOTS + b); };
    auto acce_bar = [&](int b) { return bars + 8u * (2 * SLOTS + 2 + b); };
    uint8_t *aux = gen_ring + SLOTS * kMegaSlotBytes;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(aux + 192);
    volatile unsigned *gen_s = reinterpret_cast<volatile unsigned *>(aux + 200);
    volatile int *abort_s = reinterpret_cast<volatile int *>(aux + 204);
    constexpr int FS = DH + 8;                            // row stride of a fold slot (bank-conflict free)
    float *sc_o = reinterpret_cast<float *>(aux + 256);  // two [16][FS] slots
    float *sc_m = sc_o + 2 * 16 * FS, *sc_l = sc_m + 32;
    int *flag = reinterpret_cast<int *>(sc_l + 32);
    int *cum = flag + 8, *nk_s = cum + kAttMaxItems + 1;
    float *red = reinterpret_cast<float *>(nk_s + kAttMaxItems + 1);  // [32] worker reductions
    float *rs_s = red + 32;                                           // [64] 1/rms per row
    int *pos_s = reinterpret_cast<int *>(rs_s + 64), *pg_s = pos_s + 32;  // per sequence: position, page of the append
#ifdef DBT_MEGA_TL
    unsigned long long *tl = reinterpret_cast<unsigned long long *>(pg_s + 32);  // debug: barrier timestamps
    unsigned long long *dbg = tl + 384;                                          // debug: [288] in-phase timestamps
#endif

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_prod = warp == 0, is_mma = warp == 1, is_worker = warp >= 2;
    const int wt = tid - 64, ww = warp - 2;  // worker thread / warp index
    const int C = gridDim.x, cta = blockIdx.x;
    const int B = pl->B, grouped = pl->grouped, R = pl->R, d = pl->d, dh = DH, n_q = pl->n_q, n_kv = pl->n_kv;
    const int F = pl->F, V = pl->V, qd = n_q * dh, kvd = n_kv * dh, G = n_q / n_kv, half = dh / 2;
    const int ss_tiles = (d + 255) / 256, ss_ld = pl->Rmax;
    const float eps = pl->eps;
    float *const P = pl->P;
    const CUtensorMap *maps = pl->maps;
    const CUtensorMap *map_tail = maps + (size_t)pl->L * 7;
    const CUtensorMap *map_act = map_tail + 2 + 3 * (N_TILE == 16 ? 0 : N_TILE == 32 ? 1 : 2);  // Xb, Ob, Hb

    if (tid == 0) {
        for (int s = 0; s < SLOTS; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 4);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(accf_bar(b), 1);
            mbar_init(acce_bar(b), kMegaWorkerWarps);
        }
        *gen_s = 0;
        *abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (is_mma) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)(2 * kMegaAcc * N_TILE))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (is_worker && wt < B) {
        // the step's positions and append pages, once (the lengths move only at the very end)
        int pos = ld_mut(pl->seq_len + wt);
        int page = pl->page_table[(size_t)wt * pl->pt_stride + pos / 16];
        if (page < 0 || page >= pl->num_pages) {
            report(pl->status, kStatusBadPage, page);
            page = -1;
        }
        pos_s[wt] = pos;
        pg_s[wt] = page;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_holder;

    // ---- shared bookkeeping: every role walks the same schedule and keeps the same counters
    unsigned k_bar = 0;  // grid barriers in program order
    int it = 0;          // ring slots in program order
    int seg_it = 0;      // GEMM segments (TMEM buffers) in program order
    bool ok = true;

    auto fail_here = [&](int site) {
        ok = false;
        *abort_s = 1;
        atomicExch(pl->err, 1);
        report(pl->status, kStatusWaitExpired, site);
    };
    // bounded waits that also give up as soon as any role of any CTA has failed
    auto wait_bar = [&](uint32_t bar, uint32_t parity, int site) {
        if (!ok) return;
        uint32_t done = 0;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return;
        long long t0 = clock64();
        unsigned spins = 0;
        while (true) {
            asm volatile(
                "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                : "=r"(done)
                : "r"(bar), "r"(parity)
                : "memory");
            if (done) return;
            if ((++spins & 1023u) == 0) {
                if (*abort_s || (unsigned long long)(clock64() - t0) > kMegaWaitCycles) {
                    fail_here(site);
                    return;
                }
            }
        }
    };
    // Grid barrier.  Workers arrive and wait; the other roles only count it.
    auto grid_barrier = [&]() {
        k_bar++;
        if (!is_worker) return;
        asm volatile("fence.proxy.async;" ::: "memory");  // this phase's stores are read by other SMs' TMA next
        worker_sync();
        if (wt == 0) {
            __threadfence();
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(pl->bar_count) : "memory");
            const unsigned target = k_bar * (unsigned)C;
            long long t0 = clock64();
            unsigned spins = 0;
            while (ok && ld_acquire_u32(pl->bar_count) < target) {
                if ((++spins & 255u) == 0) {
                    if (*abort_s || *(volatile int *)pl->err || (unsigned long long)(clock64() - t0) > kMegaWaitCycles)
                        fail_here(900 + (int)(k_bar & 63));
                }
            }
            *gen_s = k_bar;
#ifdef DBT_MEGA_TL
            if (cta == 0 && k_bar < 380) tl[k_bar] = gtime();
            tl[380] = gtime();
            tl[381] = (unsigned long long)clock64();
#endif
        }
        worker_sync();
        if (*abort_s) ok = false;
    };
    // the producer and the MMA issuer learn from their own CTA's workers that barrier k has been passed
    auto wait_gen = [&](unsigned k, int site) {
        if (!ok) return;
        long long t0 = clock64();
        unsigned spins = 0;
        while (*gen_s < k) {
            if ((++spins & 255u) == 0) {
                if (*abort_s || (unsigned long long)(clock64() - t0) > kMegaWaitCycles) {
                    fail_here(site);
                    return;
                }
            }
        }
        __threadfence_block();
        asm volatile("fence.proxy.async;" ::: "memory");  // other SMs' stores, now visible, are read next by TMA
    };
    // the same without fences, for a role that touches shared and tensor memory only
    auto wait_gen_light = [&](unsigned k, int site) {
        if (!ok) return;
        if (*gen_s >= k) return;
        long long t0 = clock64();
        unsigned spins = 0;
        while (*gen_s < k) {
            if ((++spins & 255u) == 0) {
                if (*abort_s || (unsigned long long)(clock64() - t0) > kMegaWaitCycles) {
                    fail_here(site);
                    return;
                }
            }
        }
    };
    // sums of two values over the worker threads (result to all)
    auto worker_sum2 = [&](float &a, float &b) {
        a = warp_sum(a);
        b = warp_sum(b);
        worker_sync();
        if (lane == 0) {
            red[2 * ww] = a;
            red[2 * ww + 1] = b;
        }
        worker_sync();
        a = b = 0.f;
#pragma unroll
        for (int w = 0; w < kMegaWorkerWarps; w++) {
            a += red[2 * w];
            b += red[2 * w + 1];
        }
    };
    // 1/rms of every row from the shares of sum(S^2): loads first, the rest after the caller's own loads
    auto rs_issue = [&](float (&sh)[16]) {
#pragma unroll
        for (int t = 0; t < 16; t++) sh[t] = (wt < R && t < ss_tiles) ? __ldcg(pl->ss + (size_t)t * ss_ld + wt) : 0.f;
    };
    auto rs_finish = [&](const float (&sh)[16]) {
        float a = 0.f;
#pragma unroll
        for (int t = 0; t < 16; t++) a += sh[t];
        for (int t = 16; t < ss_tiles; t++) a += (wt < R) ? __ldcg(pl->ss + (size_t)t * ss_ld + wt) : 0.f;
        if (wt < R) rs_s[wt] = 1.f / sqrtf(a / (float)d + eps);
        worker_sync();
    };

    auto make_gemm = [&](const CUtensorMap *w0, int n0, const CUtensorMap *w1, int n1, const CUtensorMap *w2, int n2,
                         const CUtensorMap *x, int K) {
        MegaGemm g;
        g.w[0] = w0; g.w[1] = w1; g.w[2] = w2;
        g.n_out[0] = n0; g.n_out[1] = n1; g.n_out[2] = n2;
        g.nseg = w2 ? 3 : w1 ? 2 : 1;
        g.K = K;
        g.tiles = (n0 + 127) / 128 + (w1 ? (n1 + 127) / 128 : 0) + (w2 ? (n2 + 127) / 128 : 0);
        g.KT = (K + kTcK - 1) / kTcK;
        g.U = g.tiles * g.KT;
        g.q = (g.U + C - 1) / C;
        g.lo_row0 = pl->Rmax;
        g.x = x;
        return g;
    };

    // ---- one GEMM phase; the activations are ready once grid barrier `gate` has been passed.
    // The per-unit loops of the producer and the MMA issuer are the serial paths of a phase: no
    // divisions, no state in local memory, slot and k-tile indices advanced incrementally.
    auto gemm_phase = [&](const MegaGemm &g, unsigned gate) {
        const int KT = g.KT, U = g.U, q = g.q;
        const int u0 = min(U, cta * q), u1 = min(U, u0 + q), nun = u1 - u0;
        const int tile0 = u0 / KT, kt0 = u0 - tile0 * KT;
        const int nsegs = nun > 0 ? (u1 - 1) / KT - tile0 + 1 : 0;
        const int it0 = it, seg0 = seg_it;
        const int s0 = it0 % SLOTS, ph0 = (it0 / SLOTS) & 1;
        if (is_prod) {
            // lane 0 waits, arms the barrier and issues the weight tile; the activation boxes of the
            // units parked behind the gate go out from as many lanes at once
            const CUtensorMap *w0 = g.w[0], *w1 = g.w[1], *w2 = g.w[2], *xm = g.x;
            const int t1 = (g.n_out[0] + 127) / 128, t2 = t1 + (g.nseg > 1 ? (g.n_out[1] + 127) / 128 : 0);
            const uint32_t tx = kTcABytes + 2 * Cfg::kBBytes;
            const int npark = min(nun, SLOTS);  // units whose weight tile is issued before the gate opens
            int s = s0, ph = ph0, tile = tile0, kt = kt0;
            if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(xm) : "memory");
            for (int i = 0; i < nun; i++) {
                if (lane == 0) {
                    if (it0 + i >= SLOTS) wait_bar(empty_bar(s), ph ^ 1, 400);
                    if (ok) {
                        const CUtensorMap *wm = tile < t1 ? w0 : (tile < t2 ? w1 : w2);
                        int row0 = (tile - (tile < t1 ? 0 : (tile < t2 ? t1 : t2))) * 128;
                        mbar_expect_tx(full_bar(s), tx);
                        tma_load_2d(ring + s * kMegaSlotBytes, wm, full_bar(s), kt * kTcK, row0);
                        if (i >= npark) tma_load_3d(ring + s * kMegaSlotBytes + kTcABytes, xm, full_bar(s), kt * kTcK, 0, 0);
                    }
                }
                if (i == npark - 1) {
                    if (lane == 0) wait_gen(gate, 410);
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    asm volatile("fence.proxy.async;" ::: "memory");
                    if (ok && lane < npark) {
                        int sp = s0 + lane, ktp = kt0 + lane;
                        if (sp >= SLOTS) sp -= SLOTS;
                        while (ktp >= KT) ktp -= KT;
                        tma_load_3d(ring + sp * kMegaSlotBytes + kTcABytes, xm, full_bar(sp), ktp * kTcK, 0, 0);
                    }
                }
                if (++kt == KT) {
                    kt = 0;
                    tile++;
                }
                if (++s == SLOTS) {
                    s = 0;
                    ph ^= 1;
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
        } else if (is_mma) {
            if (lane == 0) {
                constexpr uint32_t idesc = umma_idesc(N_TILE);
                static_assert(kTcK / 16 == kMegaAcc, "one accumulator per k16 step");
                // Not before this CTA's workers are through the preceding phases: a wait posted on a
                // full barrier while the attention phase still cycles the same slot would be two
                // phases ahead of it and could match the parity of an attention stage.
                wait_gen_light(gate, 415);
                const uint64_t desc_hi = umma_smem_desc(0);
                int s = s0, ph = ph0, kt = kt0, seg = seg0;
                for (int i = 0; i < nun && ok; i++) {
                    const int buf = seg & 1;
                    const bool first = i == 0 || kt == 0, last = i == nun - 1 || kt == KT - 1;
                    if (first && seg >= 2) wait_bar(acce_bar(buf), ((seg >> 1) - 1) & 1, 420);
                    wait_bar(full_bar(s), ph, 421);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = ring + s * kMegaSlotBytes;
                    const uint64_t adesc = desc_hi | (uint64_t)((sa & 0x3FFFFu) >> 4);
                    const uint32_t acc = first ? 0u : 1u, d0 = tmem_base + buf * kMegaAcc * N_TILE;
#pragma unroll
                    for (int part = 0; part < 2; part++) {
                        const uint64_t bdesc = desc_hi | (uint64_t)(((sa + kTcABytes + part * Cfg::kBBytes) & 0x3FFFFu) >> 4);
#pragma unroll
                        for (int k = 0; k < kTcK / 16; k++)  // k16 step k accumulates in its own buffer
                            umma_f16(d0 + k * N_TILE, adesc + 2 * k, bdesc + 2 * k, idesc, part == 0 ? acc : 1u);
                    }
                    // the slot is free when these MMAs have read it: three plain arrivals plus the commit's
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], 3;" ::"r"(empty_bar(s)) : "memory");
                    umma_commit(empty_bar(s));
                    if (last) {
                        umma_commit(accf_bar(buf));
                        seg++;
                    }
                    if (++kt == KT) kt = 0;
                    if (++s == SLOTS) {
                        s = 0;
                        ph ^= 1;
                    }
                }
            }
        } else {
            // workers: each finished segment out of tensor memory into its partial slot; two warps
            // share a TMEM lane quarter and take alternate 16-row chunks; the four accumulators of a
            // segment are added here, in a fixed order
            for (int sgi = 0; sgi < nsegs; sgi++) {
                const int tile = tile0 + sgi, seg = seg0 + sgi, buf = seg & 1;
                wait_bar(accf_bar(buf), (seg >> 1) & 1, 430);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (ok) {
                    float *out = P + (size_t)(cta + tile) * SLOT_FLOATS + (warp & 3) * 32 + lane;
                    const uint32_t t0 = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + buf * kMegaAcc * N_TILE;
#pragma unroll 1
                    for (int c0 = (ww >> 2) * 16; c0 < N_TILE && c0 < R; c0 += 32) {
                        float v[16];
                        tmem_ld16(t0 + c0, v);
#pragma unroll
                        for (int a = 1; a < kMegaAcc; a++) {
                            float t[16];
                            tmem_ld16(t0 + a * N_TILE + c0, t);
#pragma unroll
                            for (int i = 0; i < 16; i++) v[i] += t[i];
                        }
#pragma unroll
                        for (int i = 0; i < 16; i++)
                            if (c0 + i < R) out[(size_t)(c0 + i) * 128] = v[i];
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acce_bar(buf)) : "memory");
            }
        }
        it = it0 + nun;
        seg_it = seg0 + nsegs;
    };

    // ---- attention phase (same decomposition as the stand-alone kernel, CTAs = the grid; the two
    // groups of four worker warps take alternate stages and their states are folded at the end)
    auto attn_phase = [&](int layer, unsigned gate) {
        const int items = B, Bc = B, nq_act = grouped ? 2 * G : G;
        if (is_prod) {
            if (lane == 0) wait_gen(gate, 500);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            asm volatile("fence.proxy.async;" ::: "memory");
        }
        if (warp == 2) {
            int running = 0, longest = 0;
            if (lane == 0) cum[0] = 0;
            for (int base = 0; base < items; base += 32) {
                int i = base + lane, nk = 0, u = 0;
                if (i < items) {
                    nk = pos_s[i] + 1;
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
            if (lane == 0) flag[1] = longest;
        }
        __syncthreads();
        const int U = cum[items] * n_kv;
        const int quota = max(max((U + C - 1) / C, kAttMinUnits), (flag[1] + kAttMaxSeg - 2) / (kAttMaxSeg - 1));
        const int u0 = min(U, cta * quota), u1 = min(U, u0 + quota);
        const int it0 = it;
        const long long k_row0 = (long long)layer * 2 * pl->plane_rows;
        const CUtensorMap *tmKV = map_tail + 1;
        int item = 0;
        if (u0 < u1)
            while (cum[item + 1] * n_kv <= u0) item++;

        if (is_prod) {
            // lane 0 waits for the slot and arms its barrier; up to four lanes then issue one box each
            // (a page's K and V, 8 KB), each after its own page-table lookup
#ifdef DBT_MEGA_TL
            unsigned long long tp0 = gtime(), twait = 0;
#endif
            for (int u = u0; u < u1 && ok;) {
                int ui = cum[item + 1] - cum[item], base = cum[item] * n_kv;
                int g = (u - base) / ui, t0 = (u - base) % ui;
                int pair_end = base + (g + 1) * ui, t1 = t0 + min(u1, pair_end) - u;
                int total_pages = (nk_s[item] + 15) >> 4;
                for (int t = t0; t < t1; t++, it++) {
                    int s = it % SLOTS;
                    int p0 = t * 4, np = min(4, total_pages - p0);
                    if (lane == 0) {
#ifdef DBT_MEGA_TL
                        unsigned long long tw0 = gtime();
#endif
                        if (it >= SLOTS) wait_bar(empty_bar(s), ((it / SLOTS) - 1) & 1, 510);
#ifdef DBT_MEGA_TL
                        twait += gtime() - tw0;
#endif
                        if (ok) mbar_expect_tx(full_bar(s), (uint32_t)np * 2 * PAGE_BYTES);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    if (lane < np) {
                        int page = __ldg(pl->page_table + (size_t)item * pl->pt_stride + p0 + lane);
                        if (page < 0 || page >= pl->num_pages) {
                            report(pl->status, kStatusBadPage, page);
                            page = 0;
                        }
                        int row = (int)(((long long)page * n_kv + g) * 16);
                        tma_load_4d(ring + s * kMegaSlotBytes + lane * 2 * PAGE_BYTES, tmKV, full_bar(s), 0, 0, (int)(k_row0 + row), 0);
                    }
                }
                u += t1 - t0;
                if (u == pair_end && g == n_kv - 1) item++;
            }
            __syncwarp();
#ifdef DBT_MEGA_TL
            if (cta == 1 && layer == 15 && lane == 0)
                printf("ATT prod: tiles %d issue span %llu ns, waiting on empty %llu ns\n", u1 - u0, gtime() - tp0, twait);
#endif
        } else if (is_worker) {
#ifdef DBT_MEGA_TL
            unsigned long long tbar = tl[380];
            unsigned long long tc0 = gtime(), tcw = 0, tfold = 0, tA = 0, tB = 0, tC = 0, tD = 0, tq = 0;
#endif
            const float qscale = kLog2e / sqrtf((float)DH);
            const int grp = ww >> 2, pw = ww & 3;  // stage group, page within the stage
            for (int u = u0; u < u1;) {
                int ui = cum[item + 1] - cum[item], base = cum[item] * n_kv;
                int g = (u - base) / ui, t0 = (u - base) % ui;
                int pair_start = base + g * ui, pair_end = pair_start + ui, t1 = t0 + min(u1, pair_end) - u;
                int nkeys = nk_s[item];
                worker_sync();
                for (int idx = wt; idx < 16 * DH / 4; idx += NW) {
                    int q = idx / (DH / 4), c4 = idx % (DH / 4);
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (q < nq_act) {
                        int row = q < G ? item : Bc + item;
                        int h = g * G + (q < G ? q : q - G);
                        v = __ldcg(reinterpret_cast<const float4 *>(pl->Q + (size_t)row * qd + (size_t)h * DH) + c4);
                    }
                    reinterpret_cast<float4 *>(sc_o)[idx] = v;
                }
                worker_sync();
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
                worker_sync();
                float o[NB][4];
#pragma unroll
                for (int nb = 0; nb < NB; nb++) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
                float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
                for (int t = t0 + grp; t < t1; t += 2) {
                    int iu = it + (t - t0), s = iu % SLOTS;
#ifdef DBT_MEGA_TL
                    unsigned long long tw0 = gtime();
#endif
                    wait_bar(full_bar(s), (iu / SLOTS) & 1, 520);
#ifdef DBT_MEGA_TL
                    tcw += gtime() - tw0;
#endif
                    bool live = __all_sync(0xffffffffu, ok);
                    int valid = min(16, nkeys - (t * kAttTile + pw * 16));
                    if (live && valid > 0) {
                        // a page's box: K then V, each [16 rows][DH] with the 128-byte pieces of a row swizzled
                        uint32_t kpage = ring + s * kMegaSlotBytes + pw * 2 * PAGE_BYTES;
                        uint32_t vpage = kpage + PAGE_BYTES;
                        if (valid < 16) {
                            for (int idx = lane; idx < (16 - valid) * HALVES * 8; idx += 32) {
                                uint32_t a = vpage + valid * HALVES * 128 + idx * 16;
                                asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                            }
                            __syncwarp();
                        }
                        float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                        {
                            int r = (lane & 7) + ((lane >> 4) << 3), cb = (lane >> 3) & 1;
#pragma unroll
                            for (int ks = 0; ks < KS; ks++) {
                                int chunk = ks * 2 + cb;
                                int seg = r * HALVES + (chunk >> 3);
                                uint32_t a = kpage + seg * 128 + (((chunk & 7) ^ (seg & 7)) << 4);
                                uint32_t kb[4];
                                ldsm_x4(a, kb);
                                mma_bf16(sacc[0], qa[ks], kb[0], kb[1]);
                                mma_bf16(sacc[1], qa[ks], kb[2], kb[3]);
                            }
                        }
                        int col = (lane & 3) * 2;
                        float rmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
                        for (int nb = 0; nb < 2; nb++)
#pragma unroll
                            for (int e = 0; e < 4; e++) {
                                int tk = nb * 8 + col + (e & 1);
                                if (tk >= valid) sacc[nb][e] = -INFINITY;
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
                        {
                            int r = (lane & 7) + (((lane >> 3) & 1) << 3), cb = lane >> 4;
#pragma unroll
                            for (int np = 0; np < NB / 2; np++) {
                                int chunk = np * 2 + cb;
                                int seg = r * HALVES + (chunk >> 3);
                                uint32_t a = vpage + seg * 128 + (((chunk & 7) ^ (seg & 7)) << 4);
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
                it += t1 - t0;
#ifdef DBT_MEGA_TL
                unsigned long long tf0 = gtime();
#endif
                // fold the eight warps' states through the two scratch slots, in a fixed order:
                // (0+4) (1+5), (2+6) (3+7), (0+2) (1+3), (0+1)
                int pair = item * n_kv + g;
                int first_cta = pair_start / quota, nseg = (pair_end - 1) / quota - first_cta + 1;
                float *out = pl->part + (size_t)(cta + pair) * 16 * (DH + 2);
                {
                    int r0 = lane >> 2, c = (lane & 3) * 2;
                    auto put = [&](int slot) {
                        float *so = sc_o + (size_t)slot * 16 * FS, *sm = sc_m + slot * 16, *sl = sc_l + slot * 16;
#pragma unroll
                        for (int nb = 0; nb < NB; nb++) {
                            *reinterpret_cast<float2 *>(so + (size_t)r0 * FS + nb * 8 + c) = make_float2(o[nb][0], o[nb][1]);
                            *reinterpret_cast<float2 *>(so + (size_t)(r0 + 8) * FS + nb * 8 + c) = make_float2(o[nb][2], o[nb][3]);
                        }
                        if ((lane & 3) == 0) {
                            sm[r0] = m_run[0];
                            sm[r0 + 8] = m_run[1];
                            sl[r0] = l_run[0];
                            sl[r0 + 8] = l_run[1];
                        }
                    };
                    auto take = [&](int slot) {
                        const float *so = sc_o + (size_t)slot * 16 * FS, *sm = sc_m + slot * 16, *sl = sc_l + slot * 16;
#pragma unroll
                        for (int h = 0; h < 2; h++) {
                            int r = r0 + 8 * h;
                            float mb = sm[r], lb = sl[r];
                            float M = fmaxf(m_run[h], mb);
                            float fa = m_run[h] == -INFINITY ? 0.f : exp2f(m_run[h] - M);
                            float fb = mb == -INFINITY ? 0.f : exp2f(mb - M);
                            l_run[h] = l_run[h] * fa + lb * fb;
                            m_run[h] = M;
#pragma unroll
                            for (int nb = 0; nb < NB; nb++) {
                                float2 ob = *reinterpret_cast<const float2 *>(so + (size_t)r * FS + nb * 8 + c);
                                o[nb][2 * h] = o[nb][2 * h] * fa + ob.x * fb;
                                o[nb][2 * h + 1] = o[nb][2 * h + 1] * fa + ob.y * fb;
                            }
                        }
                    };
                    // step: source warps (two of them), destination warps
                    for (int step = 0; step < 4; step++) {
                        int src0 = step == 0 ? 4 : step == 1 ? 6 : step == 2 ? 2 : 1;
                        int dst0 = step == 1 ? 2 : 0;
                        int width = step == 3 ? 1 : 2;
                        if (ww >= src0 && ww < src0 + width) put(ww - src0);
                        worker_sync();
                        if (ww >= dst0 && ww < dst0 + width) take(ww - dst0);
                        worker_sync();
                    }
#ifdef DBT_MEGA_TL
                    unsigned long long tf1 = gtime();
                    tA += tf1 - tf0;
#endif
                    if (ww == 0) {
#pragma unroll
                        for (int h = 0; h < 2; h++) {
                            int q = r0 + 8 * h;
                            if (q < nq_act) {
                                if (nseg == 1) {
                                    // the pair's only segment: normalise and write the head's output
                                    int row = q < G ? item : Bc + item;
                                    int hq = g * G + (q < G ? q : q - G);
                                    size_t ob = (size_t)row * qd + (size_t)hq * DH;
                                    float inv = 1.f / l_run[h];
#pragma unroll
                                    for (int nb = 0; nb < NB; nb++) {
                                        store_split(pl->Ob, ob + nb * 8 + c, pl->lo_o, o[nb][2 * h] * inv);
                                        store_split(pl->Ob, ob + nb * 8 + c + 1, pl->lo_o, o[nb][2 * h + 1] * inv);
                                    }
                                } else {
#pragma unroll
                                    for (int nb = 0; nb < NB; nb++)
                                        *reinterpret_cast<float2 *>(out + (size_t)q * (DH + 2) + nb * 8 + c) =
                                            make_float2(o[nb][2 * h], o[nb][2 * h + 1]);
                                    if ((lane & 3) == 0) {
                                        out[(size_t)q * (DH + 2) + DH] = m_run[h];
                                        out[(size_t)q * (DH + 2) + DH + 1] = l_run[h];
                                    }
                                }
                            }
                        }
                        if (nseg > 1) __threadfence();
                    }
                }
#ifdef DBT_MEGA_TL
                unsigned long long tf2 = gtime();
#endif
                int is_last = 0;
                if (nseg > 1) {
                    worker_sync();
                    if (wt == 0) {
                        int *tk = pl->att_tickets + pair;
                        int tkt = atomicAdd(tk, 1);
                        int last = tkt == nseg - 1;
                        if (last) {
                            atomicExch(tk, 0);
                            __threadfence();
                        }
                        flag[0] = last;
                    }
                    worker_sync();
                    is_last = flag[0];
                }
#ifdef DBT_MEGA_TL
                unsigned long long tf3 = gtime();
                tC += tf3 - tf2;
#endif
                if (is_last) {
                    const float *pbase = pl->part + (size_t)(first_cta + pair) * 16 * (DH + 2);
                    for (int idx0 = wt; idx0 < nq_act * DH; idx0 += 2 * NW) {
                        // two outputs per thread, eight segments of each in flight
                        const float *pq[2];
                        float M[2] = {-INFINITY, -INFINITY}, L[2] = {0.f, 0.f}, X[2] = {0.f, 0.f};
                        bool act[2];
#pragma unroll
                        for (int a = 0; a < 2; a++) {
                            int idx = idx0 + a * NW;
                            act[a] = idx < nq_act * DH;
                            int q = act[a] ? idx / DH : 0, e = act[a] ? idx % DH : 0;
                            pq[a] = pbase + (size_t)q * (DH + 2) + e;
                        }
                        for (int sb = 0; sb < nseg; sb += 8) {
                            float mv[2][8], lv[2][8], ov[2][8];
#pragma unroll
                            for (int a = 0; a < 2; a++)
#pragma unroll
                                for (int j = 0; j < 8; j++) {
                                    bool on = act[a] && sb + j < nseg;
                                    const float *pp = pq[a] + (size_t)(sb + j) * 16 * (DH + 2);
                                    int e = (idx0 + a * NW) % DH;
                                    mv[a][j] = on ? __ldcg(pp - e + DH) : -INFINITY;
                                    lv[a][j] = on ? __ldcg(pp - e + DH + 1) : 0.f;
                                    ov[a][j] = on ? __ldcg(pp) : 0.f;
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
                            int idx = idx0 + a * NW;
                            if (act[a]) {
                                int q = idx / DH, e = idx % DH;
                                int row = q < G ? item : Bc + item;
                                int h = g * G + (q < G ? q : q - G);
                                store_split(pl->Ob, (size_t)row * qd + (size_t)h * DH + e, pl->lo_o, X[a] / L[a]);
                            }
                        }
                    }
                }
                u += t1 - t0;
                if (u == pair_end && g == n_kv - 1) item++;
#ifdef DBT_MEGA_TL
                tfold += gtime() - tf0;
                tD += gtime() - tf3;
#endif
            }
#ifdef DBT_MEGA_TL
            if (cta == 1 && layer == 15 && (wt == 0 || wt == 128))
                printf("ATT worker %d: span %llu ns, waiting on full %llu ns, fold+merge %llu ns (fold %llu, ticket %llu, merge %llu) entry-after-barrier %llu\n", wt, gtime() - tc0, tcw, tfold, tA, tC, tD, tc0 - tbar);
            if (layer == 2 && wt == 0 && (cta % 16) == 0)
                printf("ATT cta %d: entry %llu end %llu (ns after its barrier pass) units %d\n", cta, tc0 - tbar, gtime() - tbar, u1 - u0);
#endif
        }
        it = it0 + (u1 - u0);
    };

    // =========================== the step ===========================================
    // E0: embeddings (Eq. embeddings), one row per CTA
    if (is_worker) {
        for (int r = cta; r < R; r += C) {
            int path = r >= B;
            int tok = ld_mut(tokens + (r % B));
            if (tok < 0 || tok >= V) {
                if (wt == 0) report(pl->status, kStatusBadToken, tok);
                tok = min(max(tok, 0), V - 1);
            }
            const __nv_bfloat16 *e = (path ? pl->E2 : pl->E1) + (size_t)tok * d;
            float ssq = 0.f, dummy = 0.f;
            for (int i = wt; i < d; i += NW) {
                float x = __bfloat162float(e[i]);
                ssq += x * x;
            }
            worker_sum2(ssq, dummy);
            float inv = 1.f / sqrtf(ssq / (float)d + eps), sq = 0.f;
            for (int i = wt; i < d; i += NW) {
                float s0 = pl->g_e[i] * __bfloat162float(e[i]) * inv;
                pl->S[(size_t)r * d + i] = s0;
                store_split(pl->Xb, (size_t)r * d + i, pl->lo_x, pl->g_first[i] * s0);
                sq += s0 * s0;
            }
            worker_sum2(sq, dummy);
            for (int t = wt; t < ss_tiles; t += NW) pl->ss[(size_t)t * ss_ld + r] = t == 0 ? sq : 0.f;
        }
    }
    grid_barrier();

    const int tQ = (qd + 127) / 128, tK = (kvd + 127) / 128, tG = (F + 127) / 128;
    for (int l = 0; l < pl->L; l++) {
        const MegaLayer &ly = pl->layer[l];
        const CUtensorMap *mp = maps + (size_t)l * 7;
        const long long plane = pl->plane_rows;
        __nv_bfloat16 *kpool = pl->pool + (size_t)l * 2 * plane * DH, *vpool = kpool + (size_t)plane * DH;

        // G1: Q | K | V
        MegaGemm g1 = make_gemm(mp + 0, qd, mp + 1, kvd, mp + 2, kvd, map_act + 0, d);
        gemm_phase(g1, k_bar);
        grid_barrier();
        // E1: 1/rms, RoPE, a coupling, cache append
        if (is_worker) {
            float sh[16];
            rs_issue(sh);
            const int per_row = (n_q + n_kv) * half, total = B * per_row;
            bool rs_done = false;
            for (int idx0 = cta * NW; idx0 < total || !rs_done; idx0 += C * NW) {
                int idx = idx0 + wt;
                bool act = idx < total;
                int b = 0, hh = 0, i = 0;
                if (act) {
                    b = idx / per_row;
                    int rem = idx % per_row;
                    hh = rem / half;
                    i = rem % half;
                }
                float2 t = make_float2(1.f, 0.f);
                float x[4] = {0.f, 0.f, 0.f, 0.f};
                bool isq = hh < n_q;
                if (act) {
                    t = pl->rope[(size_t)pos_s[b] * half + i];
                    if (isq) {
                        int o0 = hh * dh + i, tile = o0 / 128;
                        int tl4[4] = {tile, tile, tile, tile}, rw[4] = {b, b, grouped ? B + b : b, grouped ? B + b : b};
                        int ft[4] = {o0 % 128, (o0 + half) % 128, o0 % 128, (o0 + half) % 128};
                        mega_gather<N_TILE, 4, 3>(P, g1, tl4, rw, ft, x);
                    } else {
                        int c0 = (hh - n_q) * dh + i, tk = tQ + c0 / 128, tv = tQ + tK + c0 / 128;
                        int tl4[4] = {tk, tk, tv, tv}, rw[4] = {b, b, b, b};
                        int ft[4] = {c0 % 128, (c0 + half) % 128, c0 % 128, (c0 + half) % 128};
                        mega_gather<N_TILE, 4, 3>(P, g1, tl4, rw, ft, x);
                    }
                }
                if (!rs_done) {
                    rs_finish(sh);
                    rs_done = true;
                }
                if (!act) continue;
                float rs1 = rs_s[b];
                if (isq) {
                    int o0 = hh * dh + i, o1 = o0 + half;
                    float x0 = rs1 * x[0], x1 = rs1 * x[1];
                    float r0 = x0 * t.x - x1 * t.y, r1 = x1 * t.x + x0 * t.y;
                    pl->Q[(size_t)b * qd + o0] = r0;
                    pl->Q[(size_t)b * qd + o1] = r1;
                    if (grouped) {
                        float rs2 = rs_s[B + b];
                        float y0 = rs2 * x[2], y1 = rs2 * x[3];
                        pl->Q[(size_t)(B + b) * qd + o0] = (y0 * t.x - y1 * t.y) + ly.coup_a[o0] * r0;
                        pl->Q[(size_t)(B + b) * qd + o1] = (y1 * t.x + y0 * t.y) + ly.coup_a[o1] * r1;
                    }
                } else if (pg_s[b] >= 0) {
                    int gk = hh - n_q;
                    size_t base = (((size_t)pg_s[b] * n_kv + gk) * 16 + (pos_s[b] & 15)) * dh;
                    float x0 = rs1 * x[0], x1 = rs1 * x[1];
                    kpool[base + i] = __float2bfloat16_rn(x0 * t.x - x1 * t.y);
                    kpool[base + i + half] = __float2bfloat16_rn(x1 * t.x + x0 * t.y);
                    vpool[base + i] = __float2bfloat16_rn(rs1 * x[2]);
                    vpool[base + i + half] = __float2bfloat16_rn(rs1 * x[3]);
                }
            }
        }
        grid_barrier();
        // A: attention of both paths over the primary cache
        attn_phase(l, k_bar);
        grid_barrier();
        // G2: O projection
        MegaGemm g2 = make_gemm(mp + 3, d, nullptr, 0, nullptr, 0, map_act + 1, qd);
        gemm_phase(g2, k_bar);
        grid_barrier();
        // E2 / E4 share this: residual update, next GEMM input, shares of sum(S^2)
        auto resid = [&](const MegaGemm &g, int mode, const float *coup_c, const float *g_next) {
            if (!is_worker) return;
            for (int unit = cta; unit < B * ss_tiles; unit += C) {
                int b = unit / ss_tiles, blk = unit % ss_tiles;
                float q1 = 0.f, q2 = 0.f;
                int i = blk * 256 + wt;
                if (i < d) {
                    size_t o1 = (size_t)b * d + i, o2 = (size_t)(B + b) * d + i;
                    float s1 = __ldcg(pl->S + o1), s2 = grouped ? __ldcg(pl->S + o2) : 0.f;
                    float gn = g_next ? g_next[i] : 1.f, cc = mode == 2 ? coup_c[i] : 0.f;
                    int tl2[2] = {i / 128, i / 128}, rw[2] = {b, grouped ? B + b : b}, ft[2] = {i % 128, i % 128};
                    float mm[2];
                    mega_gather<N_TILE, 2, 5>(P, g, tl2, rw, ft, mm);
                    s1 += mm[0];
                    pl->S[o1] = s1;
                    store_split(pl->Xb, o1, pl->lo_x, gn * s1);
                    q1 = s1 * s1;
                    if (grouped) {
                        float m2 = mm[1];
                        if (mode == 2) m2 += cc * mm[0];
                        s2 += m2;
                        pl->S[o2] = s2;
                        store_split(pl->Xb, o2, pl->lo_x, gn * s2);
                        q2 = s2 * s2;
                    }
                }
                worker_sum2(q1, q2);
                if (wt == 0) {
                    pl->ss[(size_t)blk * ss_ld + b] = q1;
                    if (grouped) pl->ss[(size_t)blk * ss_ld + B + b] = q2;
                }
            }
        };
        resid(g2, 1, nullptr, ly.g_mlp);
        grid_barrier();
        // G3: gate | up
        MegaGemm g3 = make_gemm(mp + 4, F, mp + 5, F, nullptr, 0, map_act + 0, d);
        gemm_phase(g3, k_bar);
        grid_barrier();
        // E3: SwiGLU and the b coupling
        if (is_worker) {
            float sh[16];
            rs_issue(sh);
            bool rs_done = false;
            const int total = B * F;
            for (int idx0 = cta * NW; idx0 < total || !rs_done; idx0 += C * NW) {
                int idx = idx0 + wt;
                bool act = idx < total;
                int b = act ? idx / F : 0, f = act ? idx % F : 0;
                float x[4] = {0.f, 0.f, 0.f, 0.f};
                if (act) {
                    int tg = f / 128, tu = tG + f / 128, r2 = grouped ? B + b : b;
                    int tl4[4] = {tg, tu, tg, tu}, rw[4] = {b, b, r2, r2}, ft[4] = {f % 128, f % 128, f % 128, f % 128};
                    mega_gather<N_TILE, 4, 3>(P, g3, tl4, rw, ft, x);
                }
                if (!rs_done) {
                    rs_finish(sh);
                    rs_done = true;
                }
                if (!act) continue;
                float rs1 = rs_s[b];
                float h1 = silu(rs1 * x[0]) * (rs1 * x[1]);
                store_split(pl->Hb, (size_t)b * F + f, pl->lo_h, h1);
                if (grouped) {
                    float rs2 = rs_s[B + b];
                    float h2 = silu(rs2 * x[2]) * (rs2 * x[3]);
                    store_split(pl->Hb, (size_t)(B + b) * F + f, pl->lo_h, h2 + ly.coup_b[f] * h1);
                }
            }
        }
        grid_barrier();
        // G4: down
        MegaGemm g4 = make_gemm(mp + 6, d, nullptr, 0, nullptr, 0, map_act + 2, F);
        gemm_phase(g4, k_bar);
        grid_barrier();
        resid(g4, 2, ly.coup_c, ly.g_next);
        grid_barrier();
    }

    // ---- output matrix and readout (Eq. alpha, Eq. mixloss)
    MegaGemm g5 = make_gemm(map_tail + 0, V, nullptr, 0, nullptr, 0, map_act + 0, d);
    gemm_phase(g5, k_bar);
    grid_barrier();
    const int chunk = (V + C - 1) / C, v0 = min(V, cta * chunk), v1 = min(V, v0 + chunk);
    if (is_worker) {
        // logits of this CTA's vocabulary chunk; per row the chunk's (max, sum exp, sum exp^2), one
        // warp per row, eight columns' partials gathered at a time
        float sh[16];
        rs_issue(sh);
        rs_finish(sh);
        for (int r = ww; r < R; r += kMegaWorkerWarps) {
            float rs = pl->final_norm ? rs_s[r] : 1.f;
            float m = -INFINITY, s1 = 0.f, c1 = 0.f;
            for (int vb = v0 + lane; vb < v1; vb += 256) {
                int tl8[8], rw[8], ft[8];
                float z[8];
#pragma unroll
                for (int k = 0; k < 8; k++) {
                    int v = min(vb + 32 * k, V - 1);
                    tl8[k] = v / 128;
                    rw[k] = r;
                    ft[k] = v % 128;
                }
                mega_gather<N_TILE, 8, 2>(P, g5, tl8, rw, ft, z);
#pragma unroll
                for (int k = 0; k < 8; k++) {
                    int v = vb + 32 * k;
                    if (v < v1) {
                        float zz = rs * z[k];
                        pl->Z[(size_t)r * V + v] = zz;
                        if (zz > m) {
                            float f = m == -INFINITY ? 0.f : expf(m - zz);
                            s1 *= f;
                            c1 *= f * f;
                            m = zz;
                        }
                        float e1 = expf(zz - m);
                        s1 += e1;
                        c1 += e1 * e1;
                    }
                }
            }
            float M = warp_max(m);
            float f = m == -INFINITY ? 0.f : expf(m - M);
            s1 = warp_sum(s1 * f);
            c1 = warp_sum(c1 * f * f);
            if (lane == 0) {
                float *o = pl->rd_part + ((size_t)cta * 64 + r) * 4;
                o[0] = M;
                o[1] = s1;
                o[2] = c1;
            }
        }
    }
    grid_barrier();
    if (is_worker) {
        // global softmax statistics per row from the chunk partials (CTA order), then this chunk's
        // best candidate of the mixture per sequence
        for (int b = ww; b < B; b += kMegaWorkerWarps) {
            float M[2] = {0.f, 0.f}, D[2] = {1.f, 1.f}, alpha = 1.f;
            // the chunk's logits, in flight while the statistics are combined
            float z1[8], z2[8];
#pragma unroll
            for (int k = 0; k < 8; k++) {
                int v = v0 + lane + 32 * k;
                z1[k] = v < v1 ? __ldcg(pl->Z + (size_t)b * V + v) : 0.f;
                z2[k] = (grouped && v < v1) ? __ldcg(pl->Z + (size_t)(B + b) * V + v) : 0.f;
            }
            if (grouped) {
                float Cq = 0.f;
                float pm[2][5], ps[2][5], pc[5];
#pragma unroll
                for (int p = 0; p < 2; p++)
#pragma unroll
                    for (int j = 0; j < 5; j++) {
                        int c = lane + 32 * j;
                        const float *o = pl->rd_part + ((size_t)min(c, C - 1) * 64 + p * B + b) * 4;
                        pm[p][j] = c < C ? __ldcg(o) : -INFINITY;
                        ps[p][j] = c < C ? __ldcg(o + 1) : 0.f;
                        if (p == 0) pc[j] = c < C ? __ldcg(o + 2) : 0.f;
                    }
#pragma unroll
                for (int p = 0; p < 2; p++) {
                    float mx = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 5; j++) mx = fmaxf(mx, pm[p][j]);
                    mx = warp_max(mx);
                    float s = 0.f, cq = 0.f;
#pragma unroll
                    for (int j = 0; j < 5; j++)
                        if (pm[p][j] != -INFINITY) {
                            float f = expf(pm[p][j] - mx);
                            s += ps[p][j] * f;
                            if (p == 0) cq += pc[j] * f * f;
                        }
                    M[p] = mx;
                    D[p] = warp_sum(s);
                    if (p == 0) Cq = warp_sum(cq);
                }
                alpha = fminf(1.f, fmaxf(0.5f, Cq / (D[0] * D[0])));
            }
            ArgBest best = {-INFINITY, 0x7fffffff};
            for (int vb = v0 + lane; vb < v1; vb += 256) {
#pragma unroll
                for (int k = 0; k < 8; k++) {
                    int v = vb + 32 * k;
                    if (v < v1) {
                        float a1 = vb == v0 + lane ? z1[k] : __ldcg(pl->Z + (size_t)b * V + v);
                        float val = a1;
                        if (grouped) {
                            float a2 = vb == v0 + lane ? z2[k] : __ldcg(pl->Z + (size_t)(B + b) * V + v);
                            val = alpha * (expf(a1 - M[0]) / D[0]) + (1.f - alpha) * (expf(a2 - M[1]) / D[1]);
                        }
                        best = better(best, ArgBest{val, v});
                    }
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                ArgBest other = {__shfl_xor_sync(0xffffffffu, best.v, o), __shfl_xor_sync(0xffffffffu, best.i, o)};
                best = better(best, other);
            }
            if (lane == 0) {
                float *o = pl->rd_best + ((size_t)cta * 64 + b) * 2;
                o[0] = best.v;
                o[1] = __int_as_float(best.i);
                if (cta == 0 && grouped && alpha_out) alpha_out[b] = alpha;
            }
        }
    }
    grid_barrier();
    if (is_worker && cta == 0) {
        for (int b = ww; b < B; b += kMegaWorkerWarps) {
            ArgBest best = {-INFINITY, 0x7fffffff};
            for (int c = lane; c < C; c += 32) {
                const float *o = pl->rd_best + ((size_t)c * 64 + b) * 2;
                best = better(best, ArgBest{__ldcg(o), __float_as_int(__ldcg(o + 1))});
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                ArgBest other = {__shfl_xor_sync(0xffffffffu, best.v, o), __shfl_xor_sync(0xffffffffu, best.i, o)};
                best = better(best, other);
            }
            if (lane == 0) {
                if (next) next[b] = best.i;
                pl->seq_len[b] = pos_s[b] + 1;
            }
        }
    }

#ifdef DBT_MEGA_TL
    if (cta == 0 && wt == 0) {
        for (unsigned k = 2; k <= k_bar && k < 380; k++) printf("TL %u %llu\n", k, tl[k] - tl[k - 1]);
    }
    __syncthreads();
    if (cta == 1 && wt == 0) {
        const char *nm[3] = {"G3", "G2", "G4"};
        for (int ph = 0; ph < 3; ph++) {
            int base = ph == 0 ? 0 : ph == 1 ? 96 : 192;
            printf("DBG %s gate %llu done %llu | stored %llu %llu\n", nm[ph], dbg[base + 60], dbg[base + 61], dbg[base + 56], dbg[base + 57]);
            for (int u = 0; u < 24; u++) printf("DBG %s unit %d prewait %llu full %llu issued %llu\n", nm[ph], u, dbg[base + 64 + u], dbg[base + u], dbg[base + 32 + u]);
        }
    }
#endif
    // ---- teardown: nothing of this CTA may still be in flight
    if (is_prod && lane == 0 && !ok) {
        // give copies that were issued a bounded time to land before the shared memory goes away
        long long t0 = clock64();
        while ((unsigned long long)(clock64() - t0) < 200000ull) {
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (is_mma)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)(2 * kMegaAcc * N_TILE))
                     : "memory");
    if (tid == 0) {
        // the last CTA out re-arms the barrier counters for the next launch
        __threadfence();
        unsigned n = atomicAdd(pl->done_count, 1u);
        if (n == (unsigned)C - 1) {
            atomicExch(pl->bar_count, 0u);
            atomicExch(pl->done_count, 0u);
        }
    }
}

}  // namespace dbt
