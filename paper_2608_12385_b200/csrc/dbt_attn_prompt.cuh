// Causal attention of a prompt chunk over the bf16 paged cache (Section 4.4 item 1: the primary path
// alone walks the prompt and writes the cache; sm_100a).
//
// The decode kernel gives a (sequence, KV head) pair one 16-row query tile and splits its keys over
// CTAs: right for one position per sequence, wasteful for a chunk of a few thousand positions, where
// every tile of 16 / G positions would stream all its keys again (from L2: ~1 GB per layer for 2048
// positions of the 1B model).  Here a CTA owns 8 such tiles -- 8 consumer warps, each with the 16 / G
// consecutive positions x G heads of one m16 tile in registers -- and the K/V pages it brings in
// (one 4-D TMA box per page, 64 tokens per stage, the same ring as the decode kernel) serve all of
// them: an eighth of the traffic.  Each warp runs the whole online softmax of its own rows over the
// pages up to its causal limit (mma.sync m16n8k16, bf16 in, fp32 accumulate), so there is no fold
// between warps, no split, no partials; the output goes straight to the O projection's input
// planes.  Blocks are ordered longest first.  All waits are bounded.
#pragma once

#include "dbt_attn_mma.cuh"

namespace dbt {

struct PromptAttnParams {
    const float *Q;  // [B * cn][q_dim] fp32, post-RoPE
    int B, cn;       // sequences; positions per sequence in this chunk (their K, V are in the cache already)
    int G, n_kv, num_pages, pt_stride;
    long long k_row0;  // first row of this layer's K plane in the pool's row numbering
    const int32_t *page_table, *seq_len;  // seq_len: positions before this chunk
    __nv_bfloat16 *Ob;  // [B * cn][q_dim] attention output, hi plane (+ lo plane at lo_off)
    size_t lo_off;
    int *status;
    int nqb;  // query blocks per sequence: ceil(cn / (8 * 16 / G))
};

constexpr int kPaWarps = 8;  // consumer warps = query tiles per CTA

template <int DH>
struct PromptAttCfg {
    static constexpr int kPageBytes = 16 * DH * 2;
    static constexpr int kStageBytes = 2 * 4 * kPageBytes;
    static constexpr int kStages = DH == 128 ? 6 : 12;  // 192 KB ring, one CTA per SM
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;
};

template <int DH>
__global__ void __launch_bounds__((kPaWarps + 1) * 32, 1) attn_prompt_kernel(const __grid_constant__ CUtensorMap tmKV,
                                                                            PromptAttnParams p) {
    using Cfg = PromptAttCfg<DH>;
    constexpr int STAGES = Cfg::kStages, HALVES = DH / 64, KS = DH / 16, NB = DH / 8;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t bars = tiles + STAGES * Cfg::kStageBytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int PW = 16 / p.G, PB = kPaWarps * PW;  // positions per warp, per block
    // block -> (query block, sequence, KV head): the last query blocks (most keys) are scheduled first
    const int per_j = p.B * p.n_kv;
    const int j = p.nqb - 1 - (int)blockIdx.x / per_j, rest = (int)blockIdx.x % per_j;
    const int b = rest / p.n_kv, g = rest % p.n_kv;
    if (tid == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), kPaWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();  // the chunk's Q rows and its K, V rows in the cache come from the kernel before
    const int len0 = ld_mut(p.seq_len + b);
    const int c0 = j * PB, c_last = min(c0 + PB, p.cn) - 1;  // chunk positions of this block
    const int nkeys_max = len0 + c_last + 1;                 // keys visible to the block's last position
    const int T = (nkeys_max + kAttTile - 1) / kAttTile, total_pages = (nkeys_max + 15) >> 4;

    if (warp == kPaWarps) {
        // ---- producer: one box per page (K and V of this KV head), page ids fetched 32 at a time
        if (lane == 0) tma_prefetch_desc(&tmKV);
        bool ok = true;
        int pt_base = -(1 << 30), my_page = 0;
        for (int t = 0; t < T; t++) {
            const int s = t % STAGES, p0 = t * 4, np = min(4, total_pages - p0);
            if (p0 + 4 > pt_base + 32) {
                pt_base = p0;
                my_page = p0 + lane < total_pages ? __ldg(p.page_table + (size_t)b * p.pt_stride + p0 + lane) : 0;
            }
            if (lane == 0) {
                if (t >= STAGES) ok = mbar_wait(empty_bar(s), ((t / STAGES) - 1) & 1);
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
                const int row = (int)(((long long)page * p.n_kv + g) * 16);
                tma_load_4d(tiles + s * Cfg::kStageBytes + lane * 2 * Cfg::kPageBytes, &tmKV, full_bar(s), 0, 0,
                            (int)(p.k_row0 + row), 0);
            }
        }
        if (!ok && lane == 0) report(p.status, kStatusWaitExpired, 400);
        return;
    }

    // ---- consumers: warp w holds chunk positions cw0 .. cw0 + npos_w - 1 (x G heads) as one m16 tile
    const int q_dim = p.n_kv * p.G * DH;
    const int cw0 = c0 + warp * PW, npos_w = max(0, min(PW, p.cn - cw0));
    const int pos_last_w = len0 + cw0 + npos_w - 1;  // the last key this warp's rows may see
    const int r0 = lane >> 2, c = (lane & 3) * 2;
    const float qscale = kLog2e / sqrtf((float)DH);
    uint32_t qa[KS][4];
    int pl[2];  // chunk position (relative to cw0) of this lane's two rows, clamped to the valid ones
    {
        const float *qrow[2];
        bool on[2];
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const int r = r0 + 8 * h, pr = r / p.G;
            on[h] = pr < npos_w;
            pl[h] = min(pr, max(npos_w - 1, 0));
            qrow[h] = p.Q + (size_t)(b * p.cn + cw0 + pl[h]) * q_dim + (size_t)(g * p.G + r % p.G) * DH;
        }
#pragma unroll
        for (int ks = 0; ks < KS; ks++) {
            const int k = ks * 16 + c;
            float2 z = make_float2(0.f, 0.f);
            float2 a0 = on[0] ? __ldcg(reinterpret_cast<const float2 *>(qrow[0] + k)) : z;
            float2 a1 = on[1] ? __ldcg(reinterpret_cast<const float2 *>(qrow[1] + k)) : z;
            float2 a2 = on[0] ? __ldcg(reinterpret_cast<const float2 *>(qrow[0] + k + 8)) : z;
            float2 a3 = on[1] ? __ldcg(reinterpret_cast<const float2 *>(qrow[1] + k + 8)) : z;
            qa[ks][0] = pack_bf16(a0.x * qscale, a0.y * qscale);
            qa[ks][1] = pack_bf16(a1.x * qscale, a1.y * qscale);
            qa[ks][2] = pack_bf16(a2.x * qscale, a2.y * qscale);
            qa[ks][3] = pack_bf16(a3.x * qscale, a3.y * qscale);
        }
    }
    float o[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; nb++) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    // keys visible to each of this lane's two rows: 0 .. len0 + cw0 + pl
    const int lim[2] = {len0 + cw0 + pl[0] + 1, len0 + cw0 + pl[1] + 1};

    bool ok = true;
    for (int t = 0; t < T; t++) {
        const int s = t % STAGES;
        ok = mbar_wait(full_bar(s), (t / STAGES) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (npos_w > 0) {
            for (int pg = 0; pg < 4; pg++) {
                const int key0 = t * kAttTile + pg * 16;
                if (key0 > pos_last_w) break;  // this page and the later ones lie behind the warp's causal limit
                const uint32_t kpage = tiles + s * Cfg::kStageBytes + pg * 2 * Cfg::kPageBytes;
                const uint32_t vpage = kpage + Cfg::kPageBytes;
                const int valid = min(16, nkeys_max - key0);
                if (valid < 16) {
                    // slots past the block's last key hold stale pool contents: their scores are masked below and
                    // their V rows are zeroed so that 0 * garbage cannot produce a NaN (every warp that reads the
                    // page writes the same zeros before its own reads)
                    for (int idx = lane; idx < (16 - valid) * HALVES * 8; idx += 32) {
                        uint32_t a = vpage + valid * HALVES * 128 + idx * 16;
                        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
                // S = Q K^T for the page's 16 tokens: two 8-token column blocks
                float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                {
                    const int r = (lane & 7) + ((lane >> 4) << 3);  // token row this lane addresses
                    const int cb = (lane >> 3) & 1;                 // which 8-dim chunk of the k-step
#pragma unroll
                    for (int ks = 0; ks < KS; ks++) {
                        const int chunk = ks * 2 + cb;
                        const int sg = r * HALVES + (chunk >> 3);
                        const uint32_t a = kpage + sg * 128 + (((chunk & 7) ^ (sg & 7)) << 4);
                        uint32_t kb[4];
                        ldsm_x4(a, kb);
                        mma_bf16(sacc[0], qa[ks], kb[0], kb[1]);
                        mma_bf16(sacc[1], qa[ks], kb[2], kb[3]);
                    }
                }
                // causal mask per row, online softmax (base 2), P packed as the A operand of P V
                float rmax[2] = {-INFINITY, -INFINITY};
                if (key0 + 16 > min(lim[0], lim[1])) {  // only pages that cross a row's limit need the mask
#pragma unroll
                    for (int nb = 0; nb < 2; nb++)
#pragma unroll
                        for (int e = 0; e < 4; e++)
                            if (key0 + nb * 8 + c + (e & 1) >= lim[e >> 1]) sacc[nb][e] = -INFINITY;
                }
#pragma unroll
                for (int nb = 0; nb < 2; nb++)
#pragma unroll
                    for (int e = 0; e < 4; e++) rmax[e >> 1] = fmaxf(rmax[e >> 1], sacc[nb][e]);
                float corr[2], msub[2];
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    rmax[h] = fmaxf(rmax[h], __shfl_xor_sync(0xffffffffu, rmax[h], 1));
                    rmax[h] = fmaxf(rmax[h], __shfl_xor_sync(0xffffffffu, rmax[h], 2));
                    const float mnew = fmaxf(m_run[h], rmax[h]);
                    msub[h] = mnew == -INFINITY ? 0.f : mnew;
                    corr[h] = m_run[h] == -INFINITY ? 0.f : exp2f(m_run[h] - msub[h]);
                    m_run[h] = mnew;
                }
                float rsum[2] = {0.f, 0.f};
                uint32_t pa[4];
#pragma unroll
                for (int nb = 0; nb < 2; nb++) {
                    const float p0 = exp2f(sacc[nb][0] - msub[0]), p1 = exp2f(sacc[nb][1] - msub[0]);
                    const float p2 = exp2f(sacc[nb][2] - msub[1]), p3 = exp2f(sacc[nb][3] - msub[1]);
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
                if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
                    for (int nb = 0; nb < NB; nb++) {
                        o[nb][0] *= corr[0];
                        o[nb][1] *= corr[0];
                        o[nb][2] *= corr[1];
                        o[nb][3] *= corr[1];
                    }
                }
                // O += P V: V read transposed, two 8-dim column blocks per ldmatrix
                {
                    const int r = (lane & 7) + (((lane >> 3) & 1) << 3);  // token row
                    const int cb = lane >> 4;                              // which of the two dim blocks
#pragma unroll
                    for (int np = 0; np < NB / 2; np++) {
                        const int chunk = np * 2 + cb;
                        const int sg = r * HALVES + (chunk >> 3);
                        const uint32_t a = vpage + sg * 128 + (((chunk & 7) ^ (sg & 7)) << 4);
                        uint32_t vb[4];
                        ldsm_x4_trans(a, vb);
                        mma_bf16(o[np * 2], pa, vb[0], vb[1]);
                        mma_bf16(o[np * 2 + 1], pa, vb[2], vb[3]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(s)) : "memory");
    }
    if (!ok) {
        if (lane == 0) report(p.status, kStatusWaitExpired, 410 + warp);
        return;
    }
    // ---- normalise and write the rows of this warp's positions (two bf16 planes)
#pragma unroll
    for (int h = 0; h < 2; h++) {
        const int r = r0 + 8 * h, pr = r / p.G;
        if (pr >= npos_w) continue;
        const size_t ob = (size_t)(b * p.cn + cw0 + pr) * q_dim + (size_t)(g * p.G + r % p.G) * DH + c;
        const float inv = 1.f / l_run[h];
#pragma unroll
        for (int nb = 0; nb < NB; nb++) {
            const float x0 = o[nb][2 * h] * inv, x1 = o[nb][2 * h + 1] * inv;
            const __nv_bfloat162 hi = __floats2bfloat162_rn(x0, x1);
            *reinterpret_cast<__nv_bfloat162 *>(p.Ob + ob + nb * 8) = hi;
            if (p.lo_off)
                *reinterpret_cast<__nv_bfloat162 *>(p.Ob + ob + nb * 8 + p.lo_off) =
                    __floats2bfloat162_rn(x0 - __low2float(hi), x1 - __high2float(hi));
        }
    }
}

}  // namespace dbt
