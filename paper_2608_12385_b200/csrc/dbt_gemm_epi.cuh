// Epilogues fused into the grouped skinny GEMM (bf16 dense path).
//
// Every CTA of a GEMM writes its split-K partial tile; the last CTA to arrive for an output
// tile (an arrival ticket per tile, self-resetting) sums the partials in split order and
// applies the step's elementwise work for that tile, so no separate kernel runs between two
// GEMMs of a layer:
//   FE_QKV     RoPE on Q (both paths) and K (primary), Q~_2 = Q_2 + a*Q_1 (Eq. asymattn),
//              append of K_1,V_1 to the paged cache
//   FE_RESID   S-bar_i = S_i + Attn_i W_O, next GEMM input g*S-bar as two bf16 planes, and this
//              tile's share of sum(S-bar^2) per row (the RMSNorm statistic)
//   FE_GATEUP  H = SiLU(gate)*up, H~_2 = H_2 + b*H_1 (Eq. mlp), two bf16 planes
//   FE_DOWN    M_2 += c*M_1, S_i += M_i (Eq. mlp), next input and RMSNorm statistic as FE_RESID
//   FE_LMHEAD  logits = row scale * accumulator, straight from tensor memory
// RMSNorm is split around the GEMM: its gain is folded into the GEMM input and the per-row
// factor 1/rms multiplies the GEMM output (the GEMM is linear), with sum(S^2) assembled from
// the per-tile shares in tile order.
#pragma once

#include "dbt_common.cuh"

namespace dbt {

enum : int { FE_NONE = 0, FE_QKV = 1, FE_RESID = 2, FE_GATEUP = 3, FE_DOWN = 4, FE_LMHEAD = 5 };

struct FusedEpi {
    int mode;
    int cluster;      // FE_RESID / FE_DOWN: the splits of a tile form a thread-block cluster and reduce through
                      // distributed shared memory (no tickets, no partials in global memory)
    int Bc, grouped;  // primary rows; branch rows Bc..2Bc-1 present
    RowMap rm;
    int *tickets;     // one counter per output tile (zero between launches)
    int arrivals;     // CTAs per ticket: splits, or 2*splits for gate|up
    // per-row 1/rms of the GEMM input, from per-tile shares ss_in[t][ss_ld]
    const float *ss_in;
    int ss_tiles, ss_ld, d_norm, use_scale;
    float eps;
    // residual stream and the next GEMM's input
    float *S;                 // [R][n_out]
    const float *g_next;      // gain folded into the next input (nullptr: none)
    __nv_bfloat16 *Xout;      // hi plane [.][ld_out], lo plane at lo_off
    size_t lo_off;
    int ld_out;
    float *ss_out;            // [tiles][ss_ld] this GEMM's shares of sum(S^2)
    const float *coup;        // a (QKV), b (GATEUP), c (DOWN); nullptr = none
    // QKV
    float *Q;                 // [R][q_dim] fp32
    const float2 *rope;
    const int32_t *seq_len, *page_table;
    int pt_stride, num_pages, n_q, n_kv, dh;
    __nv_bfloat16 *kpool, *vpool;
    // LM head
    float *Z;
};

__device__ __forceinline__ void epi_store_split(__nv_bfloat16 *dst, size_t idx, size_t lo_off, float x) {
    __nv_bfloat16 hi = __float2bfloat16_rn(x);
    dst[idx] = hi;
    if (lo_off) dst[idx + lo_off] = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// 1/rms per row into shared memory (or 1 when the input was not normalised).
__device__ __forceinline__ void epi_row_scales(const FusedEpi &e, int R, float *rs) {
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        float v = 1.f;
        if (e.use_scale) {
            float ss = 0.f;
            for (int t = 0; t < e.ss_tiles; t++) ss += __ldcg(e.ss_in + (size_t)t * e.ss_ld + r);
            v = 1.f / sqrtf(ss / (float)e.d_norm + e.eps);
        }
        rs[r] = v;
    }
    __syncthreads();
}

// Sum the split-K partials of a [rows x 128] tile into shared memory with wide, independent
// loads (float4 slots, all splits of a slot in flight together): T[rl][f] for local rows
// rl < nb (primary rows b0..) and, in grouped mode, 32 + rl (their branch twins).
constexpr int kEpiRows = 32;  // primary rows per chunk (and as many branch rows)

__device__ __forceinline__ void epi_gather(const float *__restrict__ P, size_t sstride, int nsplit, int ldp, int colbase,
                                           int ncols, int b0, int nb, int Bc, int grouped, float *__restrict__ T) {
    const int nrl = grouped ? 2 * kEpiRows : kEpiRows;
    constexpr int UNR = 4;
    for (int slot0 = threadIdx.x; slot0 < nrl * 32; slot0 += 128 * UNR) {
        float4 acc[UNR];
        const float *src[UNR];
#pragma unroll
        for (int u = 0; u < UNR; u++) {
            int slot = slot0 + u * 128, rl = slot >> 5, c4 = slot & 31;
            int lr = rl & (kEpiRows - 1);
            bool ok = slot < nrl * 32 && lr < nb && c4 * 4 < ncols;
            int row = (rl < kEpiRows ? 0 : Bc) + b0 + lr;
            src[u] = ok ? P + (size_t)row * ldp + colbase + c4 * 4 : nullptr;
            acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int sp = 0; sp < nsplit; sp++) {
#pragma unroll
            for (int u = 0; u < UNR; u++) {
                if (src[u]) {
                    float4 v = __ldcg(reinterpret_cast<const float4 *>(src[u] + (size_t)sp * sstride));
                    acc[u].x += v.x; acc[u].y += v.y; acc[u].z += v.z; acc[u].w += v.w;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNR; u++) {
            int slot = slot0 + u * 128;
            if (slot < nrl * 32) reinterpret_cast<float4 *>(T)[slot] = acc[u];
        }
    }
}

// The work of the last-arriving CTA of an output tile.  P: [nsplit][R][ldp] partials; f0: first
// feature of the tile inside its segment; col0: first column of the segment in P; seg_kind:
// 0 Q, 1 K, 2 V for FE_QKV.  smem: 72 KB of scratch (the idle operand ring).
__device__ __forceinline__ void fused_epilogue(const FusedEpi &e, const float *P, int nsplit, int R, int ldp, int f0,
                                               int col0, int n_out, int seg_kind, int tile_index, float *smem) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t sstride = (size_t)R * ldp;
    const int Bc = e.Bc, grouped = e.grouped;
    float *rs = smem, *wsum = smem + 256;                    // [256], [4][64]
    int *posv = reinterpret_cast<int *>(smem + 512);         // [32] position of each primary row of the chunk
    int *pagev = posv + 32;                                  // [32] its physical page
    float *T0 = smem + 640, *T1 = T0 + 2 * kEpiRows * 128;   // two [64][128] tiles
    const int ncols = min(128, n_out - f0);

    if (e.mode != FE_RESID && e.mode != FE_DOWN) epi_row_scales(e, R, rs);

    for (int b0 = 0; b0 < Bc; b0 += kEpiRows) {
        const int nb = min(kEpiRows, Bc - b0);
        __syncthreads();  // the previous chunk's tiles are no longer read
        if (e.mode == FE_GATEUP) {
            epi_gather(P, sstride, nsplit, ldp, f0, ncols, b0, nb, Bc, grouped, T0);          // gate columns
            epi_gather(P, sstride, nsplit, ldp, n_out + f0, ncols, b0, nb, Bc, grouped, T1);  // up columns
        } else {
            epi_gather(P, sstride, nsplit, ldp, col0 + f0, ncols, b0, nb, Bc, grouped, T0);
            if (e.mode == FE_RESID || e.mode == FE_DOWN)  // the residual rows, same shape (one "split")
                epi_gather(e.S, 0, 1, n_out, f0, ncols, b0, nb, Bc, grouped, T1);
            if (e.mode == FE_QKV && tid < nb) {
                int seq = e.rm.seq(b0 + tid), pos = ld_mut(e.seq_len + seq) + e.rm.off(b0 + tid);
                posv[tid] = pos;
                int page = e.page_table[(size_t)seq * e.pt_stride + pos / 16];
                pagev[tid] = (page < 0 || page >= e.num_pages) ? -1 : page;  // reported by the attention walk
            }
        }
        __syncthreads();

        if (e.mode == FE_RESID || e.mode == FE_DOWN) {
            int col = f0 + tid;
            bool fv = tid < ncols;
            float cf = (e.mode == FE_DOWN && grouped && e.coup && fv) ? e.coup[col] : 0.f;
            float gn = (e.g_next && fv) ? e.g_next[col] : 1.f;
            for (int rl = 0; rl < nb; rl++) {
                float q1 = 0.f, q2 = 0.f;
                if (fv) {
                    int b = b0 + rl;
                    float m1 = T0[rl * 128 + tid];
                    float s1 = T1[rl * 128 + tid] + m1;
                    e.S[(size_t)b * n_out + col] = s1;
                    epi_store_split(e.Xout, (size_t)b * e.ld_out + col, e.lo_off, gn * s1);
                    q1 = s1 * s1;
                    if (grouped) {
                        float m2 = T0[(kEpiRows + rl) * 128 + tid] + cf * m1;
                        float s2 = T1[(kEpiRows + rl) * 128 + tid] + m2;
                        e.S[(size_t)(Bc + b) * n_out + col] = s2;
                        epi_store_split(e.Xout, (size_t)(Bc + b) * e.ld_out + col, e.lo_off, gn * s2);
                        q2 = s2 * s2;
                    }
                }
                q1 = warp_sum(q1);
                q2 = warp_sum(q2);
                if (lane == 0) {
                    wsum[warp * 64 + rl] = q1;
                    wsum[warp * 64 + kEpiRows + rl] = q2;
                }
            }
            __syncthreads();
            for (int rl = tid; rl < (grouped ? 2 : 1) * kEpiRows; rl += blockDim.x) {
                int lr = rl & (kEpiRows - 1);
                if (lr < nb) {
                    int row = (rl < kEpiRows ? 0 : Bc) + b0 + lr;
                    e.ss_out[(size_t)tile_index * e.ss_ld + row] = wsum[rl] + wsum[64 + rl] + wsum[128 + rl] + wsum[192 + rl];
                }
            }
        } else if (e.mode == FE_GATEUP) {
            int col = f0 + tid;
            if (tid < ncols) {
                float bf = (grouped && e.coup) ? e.coup[col] : 0.f;
                for (int rl = 0; rl < nb; rl++) {
                    int b = b0 + rl;
                    float sc1 = rs[b];
                    float h1 = silu(T0[rl * 128 + tid] * sc1) * (T1[rl * 128 + tid] * sc1);
                    epi_store_split(e.Xout, (size_t)b * e.ld_out + col, e.lo_off, h1);
                    if (grouped) {
                        float sc2 = rs[Bc + b];
                        float h2 = silu(T0[(kEpiRows + rl) * 128 + tid] * sc2) * (T1[(kEpiRows + rl) * 128 + tid] * sc2);
                        epi_store_split(e.Xout, (size_t)(Bc + b) * e.ld_out + col, e.lo_off, h2 + bf * h1);
                    }
                }
            }
        } else if (e.mode == FE_QKV) {
            const int dh = e.dh, half = dh / 2, q_dim = e.n_q * dh;
            int j = tid & 63, rp = tid >> 6;  // rotation pair inside the tile, row parity
            int fa = (j / half) * dh + (j % half), fb = fa + half, i = j % half;
            int ca = f0 + fa, cb = ca + half;  // feature indices inside the segment
            if (fa < ncols) {
                for (int rl = rp; rl < nb; rl += 2) {
                    int b = b0 + rl, pos = posv[rl];
                    float2 t = __ldg(e.rope + (size_t)pos * half + i);
                    float sc1 = rs[b];
                    float x0 = T0[rl * 128 + fa] * sc1, x1 = T0[rl * 128 + fb] * sc1;
                    if (seg_kind == 0) {
                        float r0 = x0 * t.x - x1 * t.y, r1 = x1 * t.x + x0 * t.y;
                        e.Q[(size_t)b * q_dim + ca] = r0;
                        e.Q[(size_t)b * q_dim + cb] = r1;
                        if (grouped) {
                            float sc2 = rs[Bc + b];
                            float y0 = T0[(kEpiRows + rl) * 128 + fa] * sc2, y1 = T0[(kEpiRows + rl) * 128 + fb] * sc2;
                            e.Q[(size_t)(Bc + b) * q_dim + ca] = (y0 * t.x - y1 * t.y) + e.coup[ca] * r0;
                            e.Q[(size_t)(Bc + b) * q_dim + cb] = (y1 * t.x + y0 * t.y) + e.coup[cb] * r1;
                        }
                    } else if (pagev[rl] >= 0) {
                        int gk = ca / dh;
                        size_t base = (((size_t)pagev[rl] * e.n_kv + gk) * 16 + (pos & 15)) * dh;
                        if (seg_kind == 1) {
                            e.kpool[base + i] = __float2bfloat16_rn(x0 * t.x - x1 * t.y);
                            e.kpool[base + i + half] = __float2bfloat16_rn(x1 * t.x + x0 * t.y);
                        } else {
                            e.vpool[base + i] = __float2bfloat16_rn(x0);
                            e.vpool[base + i + half] = __float2bfloat16_rn(x1);
                        }
                    }
                }
            }
        }
    }
}

}  // namespace dbt
