// Per-expert grouped GEMM with persistent CTAs (Eq. moe_layer: every selected expert's matrices are
// streamed once for the rows of all paths that chose it; sm_100a).
//
// gemm_tc_kernel in its per-expert mode launches one CTA per (expert, feature tile, row tile), most of
// which belong to experts nobody selected and leave at once.  Here two CTAs per SM stay resident and pull
// the units that have work -- (selected expert, row tile of its list, feature tile), enumerated from the
// per-expert counts -- round robin; the TMA ring runs on across units, and the accumulator is double
// buffered in tensor memory so that the epilogue of one unit overlaps the MMAs of the next.
//
// Roles in the 192-thread CTA: warp 0 lane 0 issues TMA, warp 1 lane 0 issues MMAs (warp 1 owns the TMEM
// allocation), warps 2..5 run the epilogue (warp w reads TMEM lanes 32 (w mod 4) ..).  Every wait is bounded.
#pragma once

#include "dbt_gemm_tc.cuh"

namespace dbt {

constexpr int kPersistMaxGroups = 1024;

// The gate|up launch may also do the SwiGLU (Eq. moe_layer's expert MLP): FUSE = a unit takes the gate tile and the
// up tile of the same 128 features (two accumulators), and its epilogue -- which overlaps the next unit's MMAs --
// writes H = SiLU(rs * gate) * (rs * up) as the down projection's two bf16 planes: no kernel in between.
struct SwigluEpi {
    __nv_bfloat16 *Hs;  // [rows][Fe] hi plane (+ lo plane at lo_off)
    size_t lo_off;
    const float *rs;    // per sorted row: 1/rms of the row the GEMM input was not yet divided by (nullptr: 1)
    int Fe;
};

template <int N_TILE, bool FUSE = false>
struct TcPersistCfg {
    using Base = TcCfg<N_TILE>;
    static constexpr int kWTiles = FUSE ? 2 : 1;
    static constexpr int kStageBytes = kWTiles * kTcABytes + 2 * Base::kBBytes;
    static constexpr int kStages = FUSE ? 3 : Base::kStages;  // both forms keep two CTAs per SM
    static constexpr int kAccCols = kWTiles * Base::kAccCols;  // accumulator columns of one unit
    static constexpr int kTmemCols = 2 * kAccCols < 32 ? 32 : 2 * kAccCols;  // two units' accumulators
    // ring + alignment slack + barriers + three tables of E (+1) ints: counts, row offsets, tile offsets
    static constexpr int smem_bytes(int n_groups) { return kStages * kStageBytes + 1024 + 256 + (3 * n_groups + 8) * 4; }
};

template <int N_TILE, bool FUSE = false>
__global__ void __launch_bounds__(192, 2)
gemm_tc_persist_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                       const __grid_constant__ CUtensorMap tmX, TcParams p, int n_groups, int tiles, SwigluEpi se) {
    using Cfg = TcCfg<N_TILE>;
    using PCfg = TcPersistCfg<N_TILE, FUSE>;
    static_assert(N_TILE <= 32, "the epilogue holds a whole accumulator row in registers");
    constexpr int STAGES = PCfg::kStages;
    constexpr int kXOff = PCfg::kWTiles * kTcABytes;  // the activation box follows the weight tile(s) of a stage
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_s = (raw + 1023u) & ~1023u;  // 1024-byte aligned operand tiles
    uint8_t *gen = smem_raw + (tiles_s - raw);
    const uint32_t bars = tiles_s + STAGES * PCfg::kStageBytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto acc_full = [&](int b) { return bars + 8u * (2 * STAGES + b); };
    auto acc_empty = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(gen + STAGES * PCfg::kStageBytes + 8 * (2 * STAGES + 4));
    int *cnt_s = reinterpret_cast<int *>(gen + STAGES * PCfg::kStageBytes + 256);  // [E]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, E = n_groups;
    int *roff = cnt_s + E;      // [E + 1] first sorted row of an expert
    int *toff = roff + E + 1;   // [E + 1] row tiles before an expert
    if (tid == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(acc_full(b), 1);
            mbar_init(acc_empty(b), 4);  // one arrival per epilogue warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)PCfg::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // the experts' row counts (final before this launch can be resident when grp_prewait is set)
    if (!p.grp_prewait) pdl_wait();
    for (int e = tid; e < E; e += blockDim.x) cnt_s[e] = ld_mut(p.grp_cnt + e);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_holder;
    if (warp == 0) {  // exclusive prefixes of the rows and of the row tiles, 32 experts per round
        int run_r = 0, run_t = 0;
        for (int base = 0; base < E; base += 32) {
            const int e = base + lane, c = e < E ? cnt_s[e] : 0, t = (c + N_TILE - 1) / N_TILE;
            int ir = c, itl = t;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int a = __shfl_up_sync(0xffffffffu, ir, o), b = __shfl_up_sync(0xffffffffu, itl, o);
                if (lane >= o) {
                    ir += a;
                    itl += b;
                }
            }
            if (e < E) {
                roff[e] = run_r + ir - c;
                toff[e] = run_t + itl - t;
            }
            run_r += __shfl_sync(0xffffffffu, ir, 31);
            run_t += __shfl_sync(0xffffffffu, itl, 31);
        }
        if (lane == 0) {
            roff[E] = run_r;
            toff[E] = run_t;
        }
    }
    __syncthreads();
    pdl_launch_dependents();

    const int U = tiles * toff[E];  // units with work
    const int total_kt = (p.K + kTcK - 1) / kTcK;
    struct Unit {
        int x_row0, rows, w_row, sg, f0;
    };
    auto decode = [&](int u) {
        const int rtg = u / tiles, ft = u % tiles;
        int lo = 0, hi = E - 1;
        while (lo < hi) {  // the expert whose row tiles hold rtg: the largest e with toff[e] <= rtg
            const int mid = (lo + hi + 1) >> 1;
            if (toff[mid] <= rtg) lo = mid; else hi = mid - 1;
        }
        const int rt = rtg - toff[lo];
        Unit un;
        un.x_row0 = roff[lo] + rt * N_TILE;
        un.rows = min(N_TILE, cnt_s[lo] - rt * N_TILE);
        un.sg = (!FUSE && p.nseg > 1 && ft >= p.seg[1].tile0) ? 1 : 0;  // FUSE: `tiles` counts one segment's tiles
        un.f0 = (ft - p.seg[un.sg].tile0) * kTcM;
        un.w_row = lo * p.grp_w_rows + un.f0;
        return un;
    };

    bool ok = true;
    if (warp == 0 && lane == 0) {
        // ---- TMA producer: the ring runs on from one unit to the next
        tma_prefetch_desc(&tmW0);
        tma_prefetch_desc(&tmW1);
        tma_prefetch_desc(&tmX);
        const uint32_t tx = PCfg::kWTiles * kTcABytes + 2 * Cfg::kBBytes;
        const uint64_t pol = l2_evict_first_policy();
        auto load_w = [&](int s, int kt, const Unit &un) {
#pragma unroll
            for (int wt = 0; wt < PCfg::kWTiles; wt++) {  // FUSE: the gate tile, then the up tile of the same features
                const CUtensorMap *tmW = (FUSE ? wt : un.sg) == 0 ? &tmW0 : &tmW1;
                const uint32_t dst = tiles_s + s * PCfg::kStageBytes + wt * kTcABytes;
                if (p.evict_first)
                    tma_load_2d_hint(dst, tmW, full_bar(s), kt * kTcK, un.w_row, pol);
                else
                    tma_load_2d(dst, tmW, full_bar(s), kt * kTcK, un.w_row);
            }
        };
        auto load_x = [&](int s, int kt, const Unit &un) {
            tma_load_3d(tiles_s + s * PCfg::kStageBytes + kXOff, &tmX, full_bar(s), kt * kTcK, un.x_row0, 0);
        };
        int it = 0;
        bool first = true;
        for (int u = blockIdx.x; u < U && ok; u += gridDim.x) {
            const Unit un = decode(u);
            int kt = 0;
            if (first) {
                // weight tiles do not depend on the previous kernel: the first ring of them goes out before the wait
                first = false;
                const int npre = min(STAGES, total_kt);
                for (int i = 0; i < npre; i++) {
                    mbar_expect_tx(full_bar(i), tx);
                    load_w(i, i, un);
                }
                pdl_wait();
                for (int i = 0; i < npre; i++) load_x(i, i, un);
                kt = npre;
                it = npre;
            }
            for (; kt < total_kt; kt++, it++) {
                const int s = it % STAGES;
                if (it >= STAGES) ok = mbar_wait(empty_bar(s), ((it / STAGES) - 1) & 1);
                if (!ok) break;
                mbar_expect_tx(full_bar(s), tx);
                load_w(s, kt, un);
                load_x(s, kt, un);
            }
        }
        if (!ok) report(p.status, kStatusWaitExpired, 500);
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer: unit j accumulates into buffer j mod 2 once the epilogue has drained it
        constexpr uint32_t idesc2 = umma_idesc(2 * N_TILE);  // both activation planes as one B operand
        int it = 0, j = 0;
        for (int u = blockIdx.x; u < U && ok; u += gridDim.x, j++) {
            const int buf = j & 1;
            ok = mbar_wait(acc_empty(buf), ((j >> 1) & 1) ^ 1);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t acc = tmem_base + buf * PCfg::kAccCols;
            for (int kt = 0; kt < total_kt; kt++, it++) {
                const int s = it % STAGES;
                ok = mbar_wait(full_bar(s), (it / STAGES) & 1);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t bdesc = umma_smem_desc(tiles_s + s * PCfg::kStageBytes + kXOff);
#pragma unroll
                for (int wt = 0; wt < PCfg::kWTiles; wt++) {
                    const uint64_t adesc = umma_smem_desc(tiles_s + s * PCfg::kStageBytes + wt * kTcABytes);
#pragma unroll
                    for (int k = 0; k < kTcK / 16; k++)
                        umma_f16(acc + wt * Cfg::kAccCols, adesc + 2 * k, bdesc + 2 * k, idesc2, (kt | k) != 0);
                }
                umma_commit(empty_bar(s));
            }
            if (ok) umma_commit(acc_full(buf));
        }
        if (!ok) report(p.status, kStatusWaitExpired, 501);
    } else if (warp >= 2) {
        // ---- epilogue: TMEM lane = weight row (feature), TMEM column = activation row
        const int q = warp & 3;
        pdl_wait();
        int j = 0;
        for (int u = blockIdx.x; u < U && ok; u += gridDim.x, j++) {
            const Unit un = decode(u);
            const int buf = j & 1;
            ok = mbar_wait(acc_full(buf), (j >> 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t base = tmem_base + ((uint32_t)(q * 32) << 16) + buf * PCfg::kAccCols;
            float v[N_TILE], vu[FUSE ? N_TILE : 1];
#pragma unroll
            for (int c0 = 0; c0 < N_TILE; c0 += 16) {
                uint32_t a[16], b[16];
                tmem_ld16_issue(base + c0, a);
                tmem_ld16_issue(base + N_TILE + c0, b);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; i++) v[c0 + i] = __uint_as_float(a[i]) + __uint_as_float(b[i]);
                if constexpr (FUSE) {  // the up tile's accumulator
                    tmem_ld16_issue(base + Cfg::kAccCols + c0, a);
                    tmem_ld16_issue(base + Cfg::kAccCols + N_TILE + c0, b);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; i++) vu[c0 + i] = __uint_as_float(a[i]) + __uint_as_float(b[i]);
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty(buf)) : "memory");
            const TcSeg seg = p.seg[un.sg];
            const int f = un.f0 + q * 32 + lane;
            if constexpr (FUSE) {
                if (f < se.Fe) {
#pragma unroll
                    for (int i = 0; i < N_TILE; i++)
                        if (i < un.rows) {
                            const int row = un.x_row0 + i;
                            const float sc = se.rs ? __ldcg(se.rs + row) : 1.f;
                            store_split(se.Hs, (size_t)row * se.Fe + f, se.lo_off, silu(sc * v[i]) * (sc * vu[i]));
                        }
                }
            } else if (f < seg.n_out) {
                float *out = p.P + (size_t)un.x_row0 * p.ldp + seg.col0 + f;
#pragma unroll
                for (int i = 0; i < N_TILE; i++)
                    if (i < un.rows) out[(size_t)i * p.ldp] = v[i];
            }
        }
        if (!ok && lane == 0) report(p.status, kStatusWaitExpired, 502 + q);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)PCfg::kTmemCols)
                     : "memory");
}

}  // namespace dbt
