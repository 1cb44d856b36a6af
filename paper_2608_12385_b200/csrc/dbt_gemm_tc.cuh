// Grouped skinny GEMM on the 5th-generation tensor cores (sm_100a): Y[r][f] = sum_k W[f][k] X[r][k].
//
// "Swap-AB": the bf16 weight tile is the 128-row A operand (it is the big, streamed side), the
// stacked [primary; branch] activation rows are the N side (16..256 columns).  Each weight
// tile is brought from HBM exactly once by TMA (128B-swizzled, K-major) into a shared-memory
// ring, multiplied by tcgen05.mma into an fp32 accumulator in tensor memory, and read back
// with tcgen05.ld for the epilogue.  One CTA = one 128-feature tile x one K range (split-K
// partials are written to global memory and summed, in split order, by the consumer kernel;
// the shared output matrix runs unsplit and writes logits, times the row's 1/rms, directly).
//
// Roles inside the 128-thread CTA: warp 0 lane 0 issues TMA, warp 1 lane 0 issues MMAs and
// owns the TMEM allocation, all four warps run the epilogue (warp w owns TMEM lanes 32w..).
// Every wait is bounded: on expiry the CTA records kStatusWaitExpired, skips its stores,
// frees its TMEM and returns.
#pragma once

#include <cuda.h>

#include "dbt_common.cuh"
#include "dbt_fused.cuh"

namespace dbt {

constexpr int kTcM = 128;       // weight rows per tile (MMA M)
constexpr int kTcK = 64;        // K elements per stage (one 128-byte swizzle row of bf16)
constexpr int kTcABytes = kTcM * kTcK * 2;
constexpr uint64_t kWaitCycles = 4000000000ull;  // ~2 s at 1.9 GHz
constexpr uint64_t kTestWaitCycles = 2000000ull;  // ~1 ms: the limit under TcParams::test_skip_load

struct TcSeg {
    int tile0;   // first tile index of this segment
    int n_out;   // features in this segment
    int rows;    // activation rows whose outputs are kept (K/V: primary rows only)
    int col0;    // first output column of this segment in P
};

// Prompt chunks, gate|up launch with two weight tiles per CTA: the two tiles are the gate tile and the up tile of
// the same 128 features, and the epilogue applies the SwiGLU (Eq. mlp: H = SiLU(m W_g) * (m W_u), with the row's
// 1/rms from its shares of sum(S^2)) and writes the down projection's input planes: no partials, no kernel between.
struct GuEpi {
    int on;
    __nv_bfloat16 *Hb;  // [rows][F] hi plane (+ lo plane at lo_off)
    size_t lo_off;
    const float *ss;    // nullptr: the GEMM input was already normalised
    int ss_tiles, ss_ld, d_norm, F;
    float eps;
};

struct TcParams {
    GuEpi gu;
    int evict_first;  // weight tiles carry the evict-first L2 hint
    int x3d;  // tmX is the 3-D {64, N_TILE, 2} view of a two-plane input: one box per stage
    int stacked;  // with x3d: one MMA per k16 step over both planes (N = 2 * N_TILE), halves added in the epilogue
    TcSeg seg[3];
    int nseg;
    int K;
    int kt_per_split;  // k-tiles (of 64) per split
    int ldp;           // row stride of P (total output features)
    int R;             // activation rows
    int parts;         // 1: X is plain bf16; 2: X = hi + lo (two bf16 terms), lo rows at lo_row0
    int lo_row0;       // row offset of the lo term inside the activation buffer
    float *P;          // [splits][R][ldp] fp32 partials
    int *status;
    // grouped (per-expert) mode: blockIdx.z = expert; its rows are grp_cnt[e] consecutive rows of
    // X and P starting at grp_off[e]; its weight rows start at e * grp_w_rows.  nullptr = off.
    const int *grp_cnt, *grp_off;
    int grp_w_rows;
    // grouped mode with row tiles: blockIdx.y = which N_TILE rows of the expert's list (CTAs past the
    // list's end leave at once); 0: the whole list fits one tile and blockIdx.y is the split as usual
    int grp_row_tiles;
    // grouped mode: 1 = the row lists were written at least three kernels before this one (by a kernel that the
    // launch chain guarantees complete before any CTA of this launch can be resident), so they may be read, and
    // the first ring of weight tiles requested, before the dependency wait
    int grp_prewait;
    // dense mode with more rows than one tile holds (prompt chunks): blockIdx.x = weight tile * row_tiles + row
    // tile, so that the CTAs sharing a weight tile are neighbours in launch order and all but the first find it
    // in L2; 0 or 1: blockIdx.x is the weight tile
    int row_tiles;
    // test hook (dbt_op_gemm_tc only): 1 = CTA (0,0,0) never requests the weight tile of its first stage
    // and every wait gives up after kTestWaitCycles, so that the expired-wait path can be exercised:
    // the kernel records kStatusWaitExpired, skips its stores, frees its TMEM and returns
    int test_skip_load;
};

// Epilogue of the shared output matrix (Section 4.2: z_i from the final states): logits = accumulator
// times the row's 1/rms (the final RMSNorm's gain is folded into the GEMM input), written to Z.
struct LmEpi {
    float *Z;             // nullptr: the ordinary split-K partial store
    const float *ss_in;   // per-tile shares of sum(S^2): [ss_tiles][ss_ld]
    int ss_tiles, ss_ld, d_norm, use_scale;
    float eps;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on a phase parity; false when the limit expired.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint64_t limit = kWaitCycles) {
    uint32_t done = 0;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;  // the common case costs one probe and no clock read
    long long t0 = clock64();
    while (true) {
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if ((unsigned long long)(clock64() - t0) > limit) return false;
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
// L2 eviction policy for data that is read once per step (weight tiles, K/V pages): evict first, so
// that the stream does not push the small reused data (activations, partials, gains, tables) out.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                                 uint64_t hint) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, "
        "%4}], [%2], %5;" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "l"(hint)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}


// K-major, 128B-swizzled operand tile: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address
    d |= (uint64_t)0 << 16;                    // leading byte offset: unused for swizzled K-major
    d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                    // SWIZZLE_128B
    return d;
}
// kind::f16, bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// The same without waiting for the data: several loads can be in flight before one tmem_ld_wait().
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; i++) v[i] = __uint_as_float(r[i]);
}

// Activations may arrive as two bf16 terms, x = hi + lo (hi = bf16(x), lo = bf16(x - hi)): the
// weight tile is then multiplied by both and the two products land in the same fp32
// accumulator, which restores fp32-level accuracy of the activations at no extra HBM traffic.
// MT: weight tiles per CTA.  A prompt chunk's GEMM (256-row activation tiles, no split-K) is bound by the
// bytes its CTAs pull from L2 per MMA; with two weight tiles (two accumulators, 2 x 256 TMEM columns) sharing
// every activation box, a stage carries 96 KB for twice the MMAs of the 80 KB stage of one tile.
template <int N_TILE, int MT = 1>
struct TcCfg {
    static constexpr int kBBytes = N_TILE * kTcK * 2;        // one term of the activation tile
    static constexpr int kStageBytes = MT * kTcABytes + 2 * kBBytes;
    // small row counts: keep one CTA near 100 KB so that a dependent kernel's CTA can become
    // resident beside it; large row counts take the whole SM
    // (64-row tiles with two weight tiles per CTA -- the per-expert GEMMs of a prompt chunk -- keep two CTAs per SM
    // with two stages of 48 KB each)
    static constexpr int kStages = N_TILE <= 16 ? 5 : N_TILE <= 32 ? 4 : N_TILE <= 64 ? (MT == 2 ? 2 : 3) : N_TILE <= 128 ? 4 : 2;
    // room for the two planes' accumulators side by side (see `stacked` in the kernel)
    static constexpr int kStackable = N_TILE <= 128;
    static constexpr int kAccCols = kStackable ? 2 * N_TILE : N_TILE;  // accumulator columns of one weight tile
    static constexpr int kTmemCols = MT * kAccCols < 32 ? 32 : MT * kAccCols;
    static_assert(MT * kAccCols <= 512, "tensor memory has 512 columns");
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int N_TILE, int MT = 1>
__global__ void __launch_bounds__(128, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
               const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmX, TcParams p,
               LmEpi e) {
    using Cfg = TcCfg<N_TILE, MT>;
    constexpr int STAGES = Cfg::kStages;
    constexpr int kBOff = MT * kTcABytes;  // the activation box follows the weight tiles of a stage
    extern __shared__ uint8_t smem_raw[];
    uint32_t raw = smem_u32(smem_raw);
    uint32_t tiles = (raw + 1023u) & ~1023u;  // 1024-byte aligned operand tiles
    uint8_t *gen_tiles = smem_raw + (tiles - raw);
    uint32_t bars = tiles + STAGES * Cfg::kStageBytes;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(gen_tiles + STAGES * Cfg::kStageBytes + 8 * (2 * STAGES + 1));
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    uint32_t accum_bar = bars + 8u * (2 * STAGES);

    DBT_TL_DECL;
    int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int tile = blockIdx.x, split = p.grp_row_tiles ? 0 : blockIdx.y;
    int x_row0 = 0, w_row0 = 0, grp_n = -1;
    if (p.row_tiles > 1) {
        x_row0 = (int)(blockIdx.x % p.row_tiles) * N_TILE;
        tile = blockIdx.x / p.row_tiles;
    }
    if (p.grp_cnt) {
        // the expert's row list comes from an earlier kernel: nothing can start before it is known
        if (!p.grp_prewait) pdl_wait();
        grp_n = ld_mut(p.grp_cnt + blockIdx.z);
        if (grp_n == 0) return;  // expert not selected by any row of either path: its weights are not read
        x_row0 = ld_mut(p.grp_off + blockIdx.z);
        w_row0 = blockIdx.z * p.grp_w_rows;
        if (p.grp_row_tiles) {
            const int r0 = (int)blockIdx.y * N_TILE;
            if (r0 >= grp_n) return;  // the expert's rows end before this tile
            x_row0 += r0;
            grp_n -= r0;
        }
    }
    int sg = 0;
    if (p.nseg > 1 && tile >= p.seg[1].tile0) sg = 1;
    if (p.nseg > 2 && tile >= p.seg[2].tile0) sg = 2;
    const TcSeg seg = p.seg[sg];
    const CUtensorMap *tmW = sg == 0 ? &tmW0 : sg == 1 ? &tmW1 : &tmW2;
    const bool gu_pair = MT == 2 && p.gu.on;
    int f0 = (tile - seg.tile0) * kTcM * (gu_pair ? 1 : MT);
    int total_kt = (p.K + kTcK - 1) / kTcK;
    int kt0 = split * p.kt_per_split;
    int nkt = min(p.kt_per_split, total_kt - kt0);

    if (tid == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(accum_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    uint32_t tmem_base = *tmem_holder;
    pdl_launch_dependents();

    bool ok = true;
    const uint64_t wait_limit = p.test_skip_load ? kTestWaitCycles : kWaitCycles;
    const bool skip_first_w = p.test_skip_load && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
    if (warp == 0 && lane == 0) {
        // ---- TMA producer.  Weight tiles do not depend on the previous kernel: the first
        // ring-full of them is requested before waiting for it.
        tma_prefetch_desc(tmW);
        tma_prefetch_desc(&tmX);
        int npre = min(STAGES, nkt);
        const uint32_t tx = MT * kTcABytes + p.parts * Cfg::kBBytes;
        auto load_x = [&](int s, int kt) {
            if (p.x3d) {
                tma_load_3d(tiles + s * Cfg::kStageBytes + kBOff, &tmX, full_bar(s), kt * kTcK, x_row0, 0);
                return;
            }
            for (int part = 0; part < p.parts; part++)
                for (int j = 0; j < N_TILE / 16; j++)
                    tma_load_2d(tiles + s * Cfg::kStageBytes + kBOff + part * Cfg::kBBytes + j * 2048, &tmX,
                                full_bar(s), kt * kTcK, part * p.lo_row0 + x_row0 + j * 16);
        };
        const uint64_t pol = l2_evict_first_policy();
        auto load_w = [&](int s, int kt) {
#pragma unroll
            for (int mt = 0; mt < MT; mt++) {  // a tile past the matrix's last row arrives as zeros
                // (gate|up pairs: tile 0 from the gate matrix, tile 1 the same rows of the up matrix)
                const CUtensorMap *tw = gu_pair ? (mt == 0 ? &tmW0 : &tmW1) : tmW;
                const int wrow = w_row0 + f0 + (gu_pair ? 0 : mt * kTcM);
                if (p.evict_first)
                    tma_load_2d_hint(tiles + s * Cfg::kStageBytes + mt * kTcABytes, tw, full_bar(s), kt * kTcK, wrow, pol);
                else
                    tma_load_2d(tiles + s * Cfg::kStageBytes + mt * kTcABytes, tw, full_bar(s), kt * kTcK, wrow);
            }
        };
        for (int i = 0; i < npre; i++) {
            mbar_expect_tx(full_bar(i), tx);
            if (!(skip_first_w && i == 0)) load_w(i, kt0 + i);
        }
        pdl_wait();
        DBT_TL_MARK(0);
        for (int i = 0; i < npre; i++) load_x(i, kt0 + i);
        for (int i = npre; i < nkt && ok; i++) {
            int s = i % STAGES;
            ok = mbar_wait(empty_bar(s), ((i / STAGES) - 1) & 1, wait_limit);
            if (!ok) break;
            mbar_expect_tx(full_bar(s), tx);
            load_w(s, kt0 + i);
            load_x(s, kt0 + i);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer
        constexpr uint32_t idesc = umma_idesc(N_TILE);
        // Stacked form: the 3-D box leaves the hi rows and the lo rows of a k-tile next to each other,
        // so they can serve as ONE B operand of 2 * N_TILE rows: hi and lo products land in separate
        // accumulator columns (added in the epilogue) and the narrow MMAs, whose cost is mostly
        // fixed, are issued once per k16 step instead of twice.
        constexpr uint32_t idesc2 = umma_idesc(Cfg::kStackable ? 2 * N_TILE : N_TILE);
        const bool stacked = Cfg::kStackable && p.stacked;
        for (int i = 0; i < nkt && ok; i++) {
            int s = i % STAGES;
            ok = mbar_wait(full_bar(s), (i / STAGES) & 1, wait_limit);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int mt = 0; mt < MT; mt++) {
                const uint32_t acc = tmem_base + mt * Cfg::kAccCols;
                uint64_t adesc = umma_smem_desc(tiles + s * Cfg::kStageBytes + mt * kTcABytes);
                if (stacked) {
                    uint64_t bdesc = umma_smem_desc(tiles + s * Cfg::kStageBytes + kBOff);
#pragma unroll
                    for (int k = 0; k < kTcK / 16; k++) umma_f16(acc, adesc + 2 * k, bdesc + 2 * k, idesc2, (i | k) != 0);
                } else {
                    for (int part = 0; part < p.parts; part++) {
                        uint64_t bdesc = umma_smem_desc(tiles + s * Cfg::kStageBytes + kBOff + part * Cfg::kBBytes);
#pragma unroll
                        for (int k = 0; k < kTcK / 16; k++)  // advance 16 elements = 32 bytes inside the swizzle row
                            umma_f16(acc, adesc + 2 * k, bdesc + 2 * k, idesc, (i | k | part) != 0);
                    }
                }
            }
            umma_commit(empty_bar(s));
        }
        if (ok) umma_commit(accum_bar);
    }
    if (warp == 0 && lane == 0) DBT_TL_MARK(1);
    if (!ok) report(p.status, kStatusWaitExpired, 100 + warp);
    __syncwarp();

    // ---- epilogue: TMEM lane = weight row (feature), TMEM column = activation row
    pdl_wait();
    DBT_TL_WAITED;
    bool got = ok && mbar_wait(accum_bar, 0, wait_limit);  // the issuing lane knows already when the accumulator will never complete
    DBT_TL_MARK(2);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (!got && lane == 0) report(p.status, kStatusWaitExpired, 200 + warp);
    got = __syncthreads_and(got);  // the ring is idle from here on: its memory serves as scratch
    float *scratch = reinterpret_cast<float *>(gen_tiles);
    int rows = grp_n >= 0 ? min(grp_n, N_TILE) : min(min(seg.rows, p.R) - x_row0, N_TILE);
    const bool stacked_acc = Cfg::kStackable && p.stacked;
    auto ld_acc = [&](int mt, int c0, float (&v)[16]) {  // 16 accumulator columns of this thread's feature
        uint32_t a[16], b[16];
        const uint32_t base = tmem_base + ((uint32_t)(warp * 32) << 16) + mt * Cfg::kAccCols;
        tmem_ld16_issue(base + c0, a);
        if (stacked_acc) tmem_ld16_issue(base + N_TILE + c0, b);
        tmem_ld_wait();  // both halves travel together
#pragma unroll
        for (int i = 0; i < 16; i++) v[i] = __uint_as_float(a[i]) + (stacked_acc ? __uint_as_float(b[i]) : 0.f);
    };
    if (got && e.Z) {
        // 1/rms per row (or 1 when the input was not normalised) into shared memory
        for (int r = tid; r < p.R; r += blockDim.x) {
            float v = 1.f;
            if (e.use_scale) {
                float ss = 0.f;
                for (int t = 0; t < e.ss_tiles; t++) ss += __ldcg(e.ss_in + (size_t)t * e.ss_ld + r);
                v = 1.f / sqrtf(ss / (float)e.d_norm + e.eps);
            }
            scratch[r] = v;
        }
        __syncthreads();
        int f = f0 + warp * 32 + lane;
#pragma unroll 1
        for (int c0 = 0; c0 < N_TILE && c0 < rows; c0 += 16) {
            float v[16];
            ld_acc(0, c0, v);
            if (f < seg.n_out) {
#pragma unroll
                for (int i = 0; i < 16; i++)
                    if (c0 + i < rows) e.Z[(size_t)(c0 + i) * p.ldp + seg.col0 + f] = v[i] * scratch[c0 + i];
            }
        }
    } else if (got && gu_pair) {
        if constexpr (MT == 2) {
            // H goes through shared memory (the idle ring: [row][128 features] per plane) so that it leaves in
            // 16-byte pieces of a row instead of 2-byte elements of a column.  F % 8 == 0.
            __nv_bfloat16 *st_hi = reinterpret_cast<__nv_bfloat16 *>(gen_tiles), *st_lo = st_hi + N_TILE * kTcM;
            float *rs_s = reinterpret_cast<float *>(st_lo + N_TILE * kTcM);
            for (int r = tid; r < rows; r += blockDim.x)
                rs_s[r] = row_scale(p.gu.ss, p.gu.ss_tiles, p.gu.ss_ld, x_row0 + r, p.gu.d_norm, p.gu.eps);
            __syncthreads();
            const int fl = warp * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < N_TILE && c0 < rows; c0 += 16) {
                float vg[16], vu[16];
                ld_acc(0, c0, vg);
                ld_acc(1, c0, vu);
#pragma unroll
                for (int i = 0; i < 16; i++) {
                    const float rs = rs_s[min(c0 + i, N_TILE - 1)];
                    const float h = silu(rs * vg[i]) * (rs * vu[i]);
                    const __nv_bfloat16 hi = __float2bfloat16_rn(h);
                    st_hi[(c0 + i) * kTcM + fl] = hi;
                    st_lo[(c0 + i) * kTcM + fl] = __float2bfloat16_rn(h - __bfloat162float(hi));
                }
            }
            __syncthreads();
            const int nf8 = max(0, min(kTcM, p.gu.F - f0)) / 8;  // 16-byte pieces of this tile's features
            for (int idx = tid; idx < rows * (kTcM / 8); idx += blockDim.x) {
                const int r = idx / (kTcM / 8), c8 = idx % (kTcM / 8);
                if (c8 < nf8) {
                    const size_t o = (size_t)(x_row0 + r) * p.gu.F + f0 + c8 * 8;
                    *reinterpret_cast<uint4 *>(p.gu.Hb + o) = *reinterpret_cast<const uint4 *>(st_hi + r * kTcM + c8 * 8);
                    if (p.gu.lo_off)
                        *reinterpret_cast<uint4 *>(p.gu.Hb + o + p.gu.lo_off) =
                            *reinterpret_cast<const uint4 *>(st_lo + r * kTcM + c8 * 8);
                }
            }
        }
    } else if (got) {
#pragma unroll 1
        for (int mt = 0; mt < MT; mt++) {
            int f = f0 + mt * kTcM + warp * 32 + lane;
            float *out = p.P + ((size_t)split * p.R + x_row0) * p.ldp + seg.col0 + f;
#pragma unroll 1
            for (int c0 = 0; c0 < N_TILE && c0 < rows; c0 += 16) {
                float v[16];
                ld_acc(mt, c0, v);
                if (f < seg.n_out) {
#pragma unroll
                    for (int i = 0; i < 16; i++)
                        if (c0 + i < rows) out[(size_t)(c0 + i) * p.ldp] = v[i];
                }
            }
        }
    }
    DBT_TL_MARK(3);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
#ifdef DBT_TL_GEMM_ALL
    if (p.grp_cnt) tlx_[3] = blockIdx.z * 1000 + blockIdx.x;  // every per-expert CTA leaves a record
    DBT_TL_END_IF(p.grp_cnt != nullptr, "gemmall");
#else
    DBT_TL_END("gemm");
#endif
}

// ---- host side: tensor maps -------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 matrix [rows][K] (K contiguous), box = 64 x box_rows, 128B swizzle, zero fill outside.
inline bool make_bf16_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t K, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {K, rows};
    cuuint64_t strides[1] = {K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kTcK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// A GEMM input held as two bf16 planes [2][plane_rows][K]: one box {64, n_tile, 2} brings a k-tile
// of n_tile rows of both planes.
inline bool make_act_map(CUtensorMap *map, const void *base, uint64_t plane_rows, uint64_t K, uint32_t n_tile) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {K, plane_rows, 2};
    cuuint64_t strides[2] = {K * 2, plane_rows * K * 2};
    cuuint32_t box[3] = {(cuuint32_t)kTcK, n_tile, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace dbt
