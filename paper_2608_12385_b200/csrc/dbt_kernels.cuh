// Generic kernels of the Decode-Branch step, templated on the storage type (fp32 / bf16).
// These cover every operation of the step with fp32 arithmetic on the CUDA cores: they are
// the fp32-model path and the fallback for shapes the tensor-core kernels do not take.
// All reductions use fixed trees and fixed orders: results are run-to-run deterministic and
// a primary row's value never depends on whether branch rows are present.
#pragma once

#include "dbt_common.cuh"

namespace dbt {

// ---------------------------------------------------------------------------------------
// Eq. embeddings: S_1^0 = RMSNorm(E_1[x]), S_2^0 = RMSNorm(E_2[x]).  One block per row.
template <typename WT>
__global__ void embed_norm_kernel(const int32_t *tokens, int n, int p0, RowMap rm,
                                  const WT *__restrict__ E1, const WT *__restrict__ E2,
                                  const float *__restrict__ g, float eps, int d, int V,
                                  float *S, int *status) {
    pdl_enter();
    __shared__ float scratch[32];
    int r = blockIdx.x;
    int path = r / rm.Bc();  // 0 primary; j >= 1: decode branch j with its own table E2[j-1] (Appendix C.1)
    int tok = ld_mut(tokens + (size_t)rm.seq(r) * n + p0 + rm.off(r));
    if (tok < 0 || tok >= V) {
        if (threadIdx.x == 0) report(status, kStatusBadToken, tok);
        tok = min(max(tok, 0), V - 1);
    }
    const WT *e = (path ? E2 + (size_t)(path - 1) * V * d : E1) + (size_t)tok * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float x = load1(e + i);
        ss += x * x;
    }
    ss = block_sum(ss, scratch);
    float inv = 1.f / sqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) S[(size_t)r * d + i] = g[i] * load1(e + i) * inv;
}

// N = RMSNorm(S) (gain g, or no gain when g == nullptr: plain copy scaled by 1).
// Output row r reads input row r * src_mul + src_add (a gather for "last position" rows).
__global__ void rmsnorm_kernel(const float *S, const float *__restrict__ g, float eps, int d,
                               int src_mul, int src_add, int apply, float *N) {
    pdl_enter();
    __shared__ float scratch[32];
    int r = blockIdx.x;
    const float *x = S + ((size_t)r * src_mul + src_add) * d;
    float inv = 1.f;
    if (apply) {
        float ss = 0.f;
        for (int i = threadIdx.x; i < d; i += blockDim.x) ss += x[i] * x[i];
        ss = block_sum(ss, scratch);
        inv = 1.f / sqrtf(ss / (float)d + eps);
    }
    for (int i = threadIdx.x; i < d; i += blockDim.x)
        N[(size_t)r * d + i] = apply ? g[i] * x[i] * inv : x[i];
}

// ---------------------------------------------------------------------------------------
// Skinny linear layer on the CUDA cores: Y[r][f] = sum_k W[f][k] X[r][k].
// One warp per output feature; the warp walks the weight row once per group of RT rows with
// 128-bit loads.  Up to three weight segments share one launch (Q|K|V).

enum : int { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_DOWN = 3, EPI_RESID_GATED = 4 };

struct LinArgs {
    const void *W[3];
    float *Y[3];
    int n_out[3];
    int rows[3];
    int nseg;
    const float *X;  // [rows][K]
    int K;
    int epi;
    int Bc;       // primary rows in this launch
    int grouped;  // paths present: 0 or 1 = the primary alone; P >= 2 = branch rows j*Bc .. (j+1)*Bc-1, j = 1..P-1
    const float *coup;  // b (EPI_SWIGLU), c (EPI_DOWN) or g_A (EPI_RESID_GATED); nullptr = no coupling
    float *S;     // residual rows [.][n_out[0]] for EPI_RESID / EPI_DOWN
};

constexpr int kLinWarps = 8;
constexpr int kLinRT = 8;

template <typename WT, int RT>
__device__ __forceinline__ void warp_dots(const WT *__restrict__ wrow, const float *const (&xp)[RT], int K,
                                          float (&acc)[RT]) {
    int lane = threadIdx.x & 31;
#pragma unroll
    for (int r = 0; r < RT; r++) acc[r] = 0.f;
    for (int k = lane * 8; k < K; k += 256) {
        float w[8];
        load8(wrow + k, w);
#pragma unroll
        for (int r = 0; r < RT; r++) {
            if (xp[r] != nullptr) {
                float x[8];
                load8(xp[r] + k, x);
#pragma unroll
                for (int i = 0; i < 8; i++) acc[r] = fmaf(w[i], x[i], acc[r]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < RT; r++) acc[r] = warp_sum(acc[r]);
}

template <typename WT>
__global__ void __launch_bounds__(kLinWarps * 32) linear_kernel(LinArgs a) {
    pdl_enter();
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int f = blockIdx.x * kLinWarps + warp;
    int seg = 0;
    if (a.epi != EPI_SWIGLU) {
        while (seg < a.nseg && f >= a.n_out[seg]) {
            f -= a.n_out[seg];
            seg++;
        }
        if (seg >= a.nseg) return;
    } else if (f >= a.n_out[0]) {
        return;
    }
    int K = a.K, rows = a.rows[seg], n_out = a.n_out[seg];
    const WT *w0 = reinterpret_cast<const WT *>(a.W[seg]) + (size_t)f * K;
    float *Y = a.Y[seg];
    for (int r0 = 0; r0 < rows; r0 += kLinRT) {
        const float *xp[kLinRT];
#pragma unroll
        for (int r = 0; r < kLinRT; r++) xp[r] = (r0 + r < rows) ? a.X + (size_t)(r0 + r) * K : nullptr;
        float acc[kLinRT];
        warp_dots<WT, kLinRT>(w0, xp, K, acc);
        if (a.epi == EPI_SWIGLU) {
            float up[kLinRT];
            const WT *w1 = reinterpret_cast<const WT *>(a.W[1]) + (size_t)f * K;
            warp_dots<WT, kLinRT>(w1, xp, K, up);
#pragma unroll
            for (int r = 0; r < kLinRT; r++) acc[r] = silu(acc[r]) * up[r];
        }
#pragma unroll
        for (int r = 0; r < kLinRT; r++) {
            if (lane == r && r0 + r < rows) {
                size_t o = (size_t)(r0 + r) * n_out + f;
                if (a.epi == EPI_RESID) {
                    a.S[o] += acc[r];
                } else if (a.epi == EPI_RESID_GATED) {
                    // S-bar_1 = S_1 + A_1 ; S-bar_2 = S_2 + g_A * A_1 (Eq. matched_attention): primary rows only
                    a.S[o] += acc[r];
                    for (int j = 1; j < a.grouped; j++) a.S[(size_t)(j * a.Bc + r0 + r) * n_out + f] += a.coup[f] * acc[r];
                } else
                    Y[o] = acc[r];
            }
        }
    }
    if (a.epi == EPI_SWIGLU && a.grouped > 1 && a.coup != nullptr) {
        // H~_j = H_j + b * H_1 (Eq. mlp), feature f of every sequence and branch
        __syncwarp();
        float bf = a.coup[f];
        for (int b = lane; b < a.Bc; b += 32)
            for (int j = 1; j < a.grouped; j++) Y[(size_t)(j * a.Bc + b) * n_out + f] += bf * Y[(size_t)b * n_out + f];
    } else if (a.epi == EPI_DOWN) {
        // M_j += c * M_1 ; S_i^{l+1} = S-bar_i + M_i (Eq. mlp)
        __syncwarp();
        float cf = (a.grouped > 1 && a.coup != nullptr) ? a.coup[f] : 0.f;
        for (int b = lane; b < a.Bc; b += 32) {
            float m1 = Y[(size_t)b * n_out + f];
            a.S[(size_t)b * n_out + f] += m1;
            for (int j = 1; j < a.grouped; j++)
                a.S[(size_t)(j * a.Bc + b) * n_out + f] += Y[(size_t)(j * a.Bc + b) * n_out + f] + cf * m1;
        }
    }
}

// ---------------------------------------------------------------------------------------
// RoPE on Q (both paths) and K (primary), the a coupling Q~_2 = Q_2 + a*Q_1 (Eq. asymattn)
// and the append of K_1,V_1 to the paged cache (Section 4.4 item 3).  One block per primary
// row, which also handles its branch twin.
template <typename KT>
__global__ void rope_couple_append_kernel(float *Q, const float *Kn,
                                          const float *Vn, RowMap rm, int grouped, int n_q,
                                          int n_kv, int dh, const float *__restrict__ coup_a,
                                          const float2 *__restrict__ rope_tab, const int32_t *seq_len,
                                          const int32_t *__restrict__ page_table, int pt_stride, int num_pages,
                                          int page_size, KT *kpool, KT *vpool, int *status) {
    pdl_enter();
    int item = blockIdx.x, Bc = rm.Bc();
    int seq = rm.seq(item), pos = ld_mut(seq_len + seq) + rm.off(item);
    int half = dh / 2, q_dim = n_q * dh, kv_dim = n_kv * dh;
    const float2 *cs = rope_tab + (size_t)pos * half;
    float *q1 = Q + (size_t)item * q_dim;
    for (int idx = threadIdx.x; idx < n_q * half; idx += blockDim.x) {
        int h = idx / half, i = idx % half;
        float2 t = cs[i];
        int o0 = h * dh + i, o1 = o0 + half;
        float x0 = q1[o0], x1 = q1[o1];
        float r0 = x0 * t.x - x1 * t.y, r1 = x1 * t.x + x0 * t.y;
        q1[o0] = r0;
        q1[o1] = r1;
        for (int j = 1; j < grouped; j++) {  // `grouped` counts the paths present: every branch row, the same a
            float *q2 = Q + (size_t)(j * Bc + item) * q_dim;
            float y0 = q2[o0], y1 = q2[o1];
            q2[o0] = (y0 * t.x - y1 * t.y) + coup_a[o0] * r0;
            q2[o1] = (y1 * t.x + y0 * t.y) + coup_a[o1] * r1;
        }
    }
    int page = page_table[(size_t)seq * pt_stride + pos / page_size];
    if (page < 0 || page >= num_pages) {
        if (threadIdx.x == 0) report(status, kStatusBadPage, page);
        return;
    }
    int slot = pos % page_size;
    const float *kn = Kn + (size_t)item * kv_dim, *vn = Vn + (size_t)item * kv_dim;
    for (int idx = threadIdx.x; idx < n_kv * half; idx += blockDim.x) {
        int g = idx / half, i = idx % half;
        float2 t = cs[i];
        size_t base = (((size_t)page * n_kv + g) * page_size + slot) * dh;
        float x0 = kn[g * dh + i], x1 = kn[g * dh + i + half];
        store1(kpool + base + i, x0 * t.x - x1 * t.y);
        store1(kpool + base + i + half, x1 * t.x + x0 * t.y);
        store1(vpool + base + i, vn[g * dh + i]);
        store1(vpool + base + i + half, vn[g * dh + i + half]);
    }
}

// ---------------------------------------------------------------------------------------
// Grouped decode attention, CUDA-core version.  One block per (primary row, KV head, split):
// the G primary query heads of that KV head and, in grouped mode, the G coupled branch
// heads read each K/V position once.  Keys 0..pos inclusive (the K/V appended this step is
// already in its page).  Partial (m, l, acc) per split; a second kernel merges in split
// order.
template <typename KT, int NQ, int DH>
__global__ void __launch_bounds__(128) attn_partial_kernel(
    const float *Q, RowMap rm, int grouped, int G, int n_kv, const KT *kpool,
    const KT *vpool, const int32_t *__restrict__ page_table, int pt_stride, int num_pages,
    const int32_t *seq_len, int nsplit, float *part, int *status) {
    pdl_enter();
    constexpr int TPB = 128, CH = 128, PS = 16, SUB = TPB / DH;
    __shared__ float qs[NQ][DH];
    __shared__ float sc[NQ][CH];
    __shared__ float m_s[NQ], l_s[NQ], corr_s[NQ];
    __shared__ int pg[CH / PS];
    int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int item = blockIdx.x, g = blockIdx.y, sp = blockIdx.z;
    int Bc = rm.Bc(), seq = rm.seq(item);
    int nkeys = ld_mut(seq_len + seq) + rm.off(item) + 1;
    int nq_act = (grouped > 1 ? grouped : 1) * G, q_dim = n_kv * G * DH;  // `grouped`: paths present
    float scale = 1.f / sqrtf((float)DH);
    for (int idx = tid; idx < NQ * DH; idx += TPB) {
        int q = idx / DH, e = idx % DH;
        float v = 0.f;
        if (q < nq_act) {
            int row = (q / G) * Bc + item;
            int h = g * G + q % G;
            v = Q[(size_t)row * q_dim + h * DH + e] * scale;
        }
        qs[q][e] = v;
    }
    if (tid < NQ) {
        m_s[tid] = -INFINITY;
        l_s[tid] = 0.f;
    }
    int total_pages = (nkeys + PS - 1) / PS;
    int pps = (total_pages + nsplit - 1) / nsplit;
    int pb = sp * pps, pe = min(total_pages, pb + pps);
    int jbeg = pb * PS, jend = min(nkeys, pe * PS);
    float acc[NQ];
#pragma unroll
    for (int q = 0; q < NQ; q++) acc[q] = 0.f;
    __syncthreads();
    for (int j0 = jbeg; j0 < jend; j0 += CH) {
        if (tid < CH / PS) {
            int p = j0 / PS + tid, page = 0;
            if (p < pe) {
                page = page_table[(size_t)seq * pt_stride + p];
                if (page < 0 || page >= num_pages) {
                    report(status, kStatusBadPage, page);
                    page = 0;
                }
            }
            pg[tid] = page;
        }
        __syncthreads();
        bool valid = j0 + tid < jend;
        float dots[NQ];
#pragma unroll
        for (int q = 0; q < NQ; q++) dots[q] = 0.f;
        if (valid) {
            const KT *kp = kpool + (((size_t)pg[tid / PS] * n_kv + g) * PS + (tid % PS)) * DH;
            for (int e = 0; e < DH; e += 8) {
                float kv[8];
                load8(kp + e, kv);
#pragma unroll
                for (int q = 0; q < NQ; q++)
#pragma unroll
                    for (int i = 0; i < 8; i++) dots[q] = fmaf(kv[i], qs[q][e + i], dots[q]);
            }
        }
#pragma unroll
        for (int q = 0; q < NQ; q++) sc[q][tid] = valid ? dots[q] : -INFINITY;
        __syncthreads();
        for (int q = warp; q < NQ; q += TPB / 32) {
            float mx = -INFINITY;
#pragma unroll
            for (int i = 0; i < CH / 32; i++) mx = fmaxf(mx, sc[q][lane + 32 * i]);
            mx = warp_max(mx);
            float mold = m_s[q], mnew = fmaxf(mold, mx), s = 0.f;
#pragma unroll
            for (int i = 0; i < CH / 32; i++) {
                float x = sc[q][lane + 32 * i];
                float p = (x == -INFINITY) ? 0.f : expf(x - mnew);
                sc[q][lane + 32 * i] = p;
                s += p;
            }
            s = warp_sum(s);
            __syncwarp();
            if (lane == 0) {
                float c = (mold == -INFINITY) ? 0.f : expf(mold - mnew);
                corr_s[q] = c;
                l_s[q] = l_s[q] * c + s;
                m_s[q] = mnew;
            }
        }
        __syncthreads();
        int e = tid % DH, sub = tid / DH, cnt = min(CH, jend - j0);
#pragma unroll
        for (int q = 0; q < NQ; q++) acc[q] *= corr_s[q];
        for (int jj = sub; jj < cnt; jj += SUB) {
            float v = load1(vpool + (((size_t)pg[jj / PS] * n_kv + g) * PS + (jj % PS)) * DH + e);
#pragma unroll
            for (int q = 0; q < NQ; q++) acc[q] = fmaf(sc[q][jj], v, acc[q]);
        }
        __syncthreads();
    }
    if (SUB > 1) {  // fold the token subsets in a fixed order
#pragma unroll
        for (int q = 0; q < NQ; q++) sc[q][tid] = acc[q];
        __syncthreads();
        if (tid < DH) {
#pragma unroll
            for (int q = 0; q < NQ; q++) {
                float t = sc[q][tid];
                for (int s2 = 1; s2 < SUB; s2++) t += sc[q][s2 * DH + tid];
                acc[q] = t;
            }
        }
    }
    float *out = part + (((size_t)item * n_kv + g) * nsplit + sp) * NQ * (DH + 2);
    if (tid < DH) {
#pragma unroll
        for (int q = 0; q < NQ; q++) out[(size_t)q * (DH + 2) + tid] = acc[q];
    }
    if (tid < NQ) {
        out[(size_t)tid * (DH + 2) + DH] = m_s[tid];
        out[(size_t)tid * (DH + 2) + DH + 1] = l_s[tid];
    }
}

// Merge the split partials in split order (log-sum-exp), write O [rows][q_dim].
__global__ void attn_merge_kernel(const float *part, int nsplit, int NQ, int DH, int Bc, int grouped,
                                  int G, int n_kv, float *O, __nv_bfloat16 *Ob,
                                  size_t lo_off) {
    pdl_enter();
    int item = blockIdx.x, g = blockIdx.y, e = threadIdx.x;
    int nq_act = (grouped > 1 ? grouped : 1) * G, q_dim = n_kv * G * DH;  // `grouped`: paths present
    const float *base = part + ((size_t)item * n_kv + g) * nsplit * NQ * (DH + 2);
    for (int q = 0; q < nq_act; q++) {
        float M = -INFINITY;
        for (int s = 0; s < nsplit; s++) M = fmaxf(M, base[((size_t)s * NQ + q) * (DH + 2) + DH]);
        float L = 0.f, o = 0.f;
        for (int s = 0; s < nsplit; s++) {
            const float *p = base + ((size_t)s * NQ + q) * (DH + 2);
            float ms = p[DH];
            float w = (ms == -INFINITY) ? 0.f : expf(ms - M);
            L += p[DH + 1] * w;
            o += p[e] * w;
        }
        int row = (q / G) * Bc + item;
        int h = g * G + q % G;
        if (O) O[(size_t)row * q_dim + h * DH + e] = o / L;
        if (Ob) {
            float x = o / L;
            __nv_bfloat16 hi = __float2bfloat16_rn(x);
            Ob[(size_t)row * q_dim + h * DH + e] = hi;
            if (lo_off) Ob[(size_t)row * q_dim + h * DH + e + lo_off] = __float2bfloat16_rn(x - __bfloat162float(hi));
        }
    }
}

// ---------------------------------------------------------------------------------------
// Readout (Eq. alpha, Eq. mixloss): p = softmax(z_1), q_j = softmax(z_j) for the decode branches
// j = 2..P (one in the main text; Appendix C.1 averages several: qbar = mean_j q_j),
// alpha = clip_[0.5,1](sum p^2), next = argmax(alpha p + (1-alpha) qbar), lowest index on ties.
// Primary-only (P = 1): next = argmax z_1.  Z rows are path-major: row j*B + b.  One block per
// sequence; the block also advances its sequence's length when asked to (the last kernel of a step).
struct ArgBest {
    float v;
    int i;
};
__device__ __forceinline__ ArgBest better(ArgBest a, ArgBest b) {
    if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
    return a;
}
constexpr int kMaxBranches = 7;  // decode branches per model (P <= 8 paths)

__global__ void __launch_bounds__(1024) readout_kernel(const float *Z, int B, int V, int P,
                                                       int32_t *next, float *alpha_out, int32_t *seq_len, int advance) {
    pdl_enter();
    __shared__ float scratch[32];
    __shared__ float bv[32];
    __shared__ int bi[32];
    int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
    const bool grouped = P > 1;
    const int nb = grouped ? P - 1 : 0;
    const float *z1 = Z + (size_t)b * V;
    float m1 = -INFINITY, d1 = 1.f, alpha = 1.f;
    float mb[kMaxBranches], db[kMaxBranches];
    if (grouped) {
        for (int v = tid; v < V; v += blockDim.x) m1 = fmaxf(m1, z1[v]);
        m1 = block_max(m1, scratch);
        float s1 = 0.f, c1 = 0.f;
        for (int v = tid; v < V; v += blockDim.x) {
            float e1 = expf(z1[v] - m1);
            s1 += e1;
            c1 += e1 * e1;
        }
        d1 = block_sum(s1, scratch);
        c1 = block_sum(c1, scratch);
        alpha = fminf(1.f, fmaxf(0.5f, c1 / (d1 * d1)));
#pragma unroll
        for (int jb = 0; jb < kMaxBranches; jb++) {
            mb[jb] = 0.f;
            db[jb] = 1.f;
            if (jb < nb) {
                const float *zj = Z + (size_t)((jb + 1) * B + b) * V;
                float mj = -INFINITY, sj = 0.f;
                for (int v = tid; v < V; v += blockDim.x) mj = fmaxf(mj, zj[v]);
                mj = block_max(mj, scratch);
                for (int v = tid; v < V; v += blockDim.x) sj += expf(zj[v] - mj);
                mb[jb] = mj;
                db[jb] = block_sum(sj, scratch);
            }
        }
    }
    const float inv_nb = grouped ? 1.f / (float)nb : 0.f;
    ArgBest best = {-INFINITY, 0x7fffffff};
    for (int v = tid; v < V; v += blockDim.x) {
        float val = z1[v];
        if (grouped) {
            float qs = 0.f;
#pragma unroll
            for (int jb = 0; jb < kMaxBranches; jb++)
                if (jb < nb) qs += expf(Z[(size_t)((jb + 1) * B + b) * V + v] - mb[jb]) / db[jb];
            val = alpha * (expf(z1[v] - m1) / d1) + (1.f - alpha) * (qs * inv_nb);
        }
        best = better(best, ArgBest{val, v});
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ArgBest other = {__shfl_xor_sync(0xffffffffu, best.v, o), __shfl_xor_sync(0xffffffffu, best.i, o)};
        best = better(best, other);
    }
    __syncthreads();
    if (lane == 0) {
        bv[warp] = best.v;
        bi[warp] = best.i;
    }
    __syncthreads();
    if (warp == 0) {
        ArgBest t = lane < nw ? ArgBest{bv[lane], bi[lane]} : ArgBest{-INFINITY, 0x7fffffff};
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ArgBest other = {__shfl_xor_sync(0xffffffffu, t.v, o), __shfl_xor_sync(0xffffffffu, t.i, o)};
            t = better(t, other);
        }
        if (lane == 0) {
            if (next) next[b] = t.i;
            if (alpha_out && grouped) alpha_out[b] = alpha;
            if (seq_len) seq_len[b] += advance;  // the step's last use of the lengths was the last layer's attention
        }
    }
}

// ---- the readout on many CTAs -----------------------------------------------------------------
// readout_kernel walks a row three times with one CTA.  Here a row is cut into NC chunks of at most
// kRoChunk logits, a CTA per (row, chunk), each logit staged in registers:
//   readout_stats_kernel: per chunk a record (m1, sum e^(z1-m1), sum e^(2(z1-m1)), and per decode branch
//     (m_j, sum e^(z_j-m_j))) with the chunk's own maxima;
//   readout_pick_kernel: every CTA folds the row's NC records in chunk order into p's and the q_j's
//     normalisers and alpha (Eq. alpha), evaluates alpha p + (1 - alpha) mean_j q_j (Eq. mixloss;
//     Appendix C.1 for several branches) over its chunk, and leaves its best (value, index); the last
//     CTA of the row to arrive picks among the NC candidates (lowest index on ties), writes the token and
//     alpha and advances the sequence length.
// Primary-only steps skip the first kernel: the pick is the argmax of z1.
// Record layout (kRoRec floats): [0] m1, [1] s1, [2] sum of squares, [3] best value, [4] best index,
// [5 + 2j] m of branch j, [6 + 2j] s of branch j.
constexpr int kRoChunk = 2048, kRoThreads = 256, kRoPer = kRoChunk / kRoThreads, kRoMaxChunks = 128;
constexpr int kRoRec = 5 + 2 * kMaxBranches + 1;

__global__ void __launch_bounds__(kRoThreads) readout_stats_kernel(const float *Z, int B, int V, int P, int chunk, float *stats) {
    pdl_enter();
    __shared__ float scratch[32];
    const int b = blockIdx.x, ck = blockIdx.y, tid = threadIdx.x;
    const int v0 = ck * chunk, v1 = min(V, v0 + chunk);
    const float *z1 = Z + (size_t)b * V, *z2 = Z + (size_t)(B + b) * V;
    float a[kRoPer], c[kRoPer];
    float m1 = -INFINITY, m2 = -INFINITY;
#pragma unroll
    for (int j = 0; j < kRoPer; j++) {
        const int v = v0 + j * kRoThreads + tid;
        a[j] = v < v1 ? __ldcg(z1 + v) : -INFINITY;
        c[j] = v < v1 ? __ldcg(z2 + v) : -INFINITY;
    }
#pragma unroll
    for (int j = 0; j < kRoPer; j++) {
        m1 = fmaxf(m1, a[j]);
        m2 = fmaxf(m2, c[j]);
    }
    m1 = block_max(m1, scratch);
    m2 = block_max(m2, scratch);
    float s1 = 0.f, q1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int j = 0; j < kRoPer; j++) {
        const float e1 = a[j] == -INFINITY ? 0.f : expf(a[j] - m1);
        s1 += e1;
        q1 += e1 * e1;
        s2 += c[j] == -INFINITY ? 0.f : expf(c[j] - m2);
    }
    s1 = block_sum(s1, scratch);
    q1 = block_sum(q1, scratch);
    s2 = block_sum(s2, scratch);
    float *o = stats + ((size_t)b * gridDim.y + ck) * kRoRec;
    if (tid == 0) {
        o[0] = m1; o[1] = s1; o[2] = q1; o[5] = m2; o[6] = s2;
    }
    for (int jb = 1; jb < P - 1; jb++) {  // further decode branches, one after the other
        const float *zj = Z + (size_t)((jb + 1) * B + b) * V;
        float mj = -INFINITY, sj = 0.f;
#pragma unroll
        for (int j = 0; j < kRoPer; j++) {
            const int v = v0 + j * kRoThreads + tid;
            c[j] = v < v1 ? __ldcg(zj + v) : -INFINITY;
            mj = fmaxf(mj, c[j]);
        }
        mj = block_max(mj, scratch);
#pragma unroll
        for (int j = 0; j < kRoPer; j++) sj += c[j] == -INFINITY ? 0.f : expf(c[j] - mj);
        sj = block_sum(sj, scratch);
        if (tid == 0) {
            o[5 + 2 * jb] = mj;
            o[6 + 2 * jb] = sj;
        }
    }
}

__global__ void __launch_bounds__(kRoThreads) readout_pick_kernel(const float *Z, int B, int V, int chunk, int P,
                                                                  float *stats, int32_t *tickets, int32_t *next,
                                                                  float *alpha_out, int32_t *seq_len, int advance) {
    pdl_enter();
    __shared__ float bv[32];
    __shared__ int bi[32];
    __shared__ float glob[4 + 2 * kMaxBranches];  // m1, d1, alpha, -, then (m_j, d_j) per branch
    __shared__ int last_s;
    const int b = blockIdx.x, ck = blockIdx.y, nc = gridDim.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int v0 = ck * chunk, v1 = min(V, v0 + chunk);
    const bool grouped = P > 1;
    const int nb = grouped ? P - 1 : 0;
    const float *z1 = Z + (size_t)b * V, *z2 = Z + (size_t)(B + b) * V;
    float a[kRoPer], c[kRoPer];
#pragma unroll
    for (int j = 0; j < kRoPer; j++) {  // the chunk's logits, requested before the row's records are folded
        const int v = v0 + j * kRoThreads + tid;
        a[j] = v < v1 ? __ldcg(z1 + v) : -INFINITY;
        c[j] = (grouped && v < v1) ? __ldcg(z2 + v) : -INFINITY;
    }
    if (grouped && warp == 0) {
        // fold the row's records: maxima first, then the sums rescaled to them, in chunk order (lane 0)
        const float *rec = stats + (size_t)b * nc * kRoRec;
        float m1 = -INFINITY;
        for (int k = lane; k < nc; k += 32) m1 = fmaxf(m1, __ldcg(rec + (size_t)k * kRoRec));
        m1 = warp_max(m1);
        if (lane == 0) {
            float d1 = 0.f, c1 = 0.f;
            for (int k = 0; k < nc; k++) {
                const float f1 = expf(__ldcg(rec + (size_t)k * kRoRec) - m1);
                d1 += __ldcg(rec + (size_t)k * kRoRec + 1) * f1;
                c1 += __ldcg(rec + (size_t)k * kRoRec + 2) * f1 * f1;
            }
            glob[0] = m1; glob[1] = d1;
            glob[2] = fminf(1.f, fmaxf(0.5f, c1 / (d1 * d1)));
        }
        for (int jb = 0; jb < nb; jb++) {
            float mj = -INFINITY;
            for (int k = lane; k < nc; k += 32) mj = fmaxf(mj, __ldcg(rec + (size_t)k * kRoRec + 5 + 2 * jb));
            mj = warp_max(mj);
            if (lane == 0) {
                float dj = 0.f;
                for (int k = 0; k < nc; k++)
                    dj += __ldcg(rec + (size_t)k * kRoRec + 6 + 2 * jb) * expf(__ldcg(rec + (size_t)k * kRoRec + 5 + 2 * jb) - mj);
                glob[4 + 2 * jb] = mj;
                glob[5 + 2 * jb] = dj;
            }
        }
    }
    __syncthreads();
    const float m1 = glob[0], d1 = glob[1], alpha = glob[2];
    const float inv_nb = grouped ? 1.f / (float)nb : 0.f;
    float qs[kRoPer];
    if (grouped) {
        const float m2 = glob[4], d2 = glob[5];
#pragma unroll
        for (int j = 0; j < kRoPer; j++) qs[j] = c[j] == -INFINITY ? 0.f : expf(c[j] - m2) / d2;
        for (int jb = 1; jb < nb; jb++) {
            const float *zj = Z + (size_t)((jb + 1) * B + b) * V;
            const float mj = glob[4 + 2 * jb], dj = glob[5 + 2 * jb];
#pragma unroll
            for (int j = 0; j < kRoPer; j++) {
                const int v = v0 + j * kRoThreads + tid;
                if (v < v1) qs[j] += expf(__ldcg(zj + v) - mj) / dj;
            }
        }
    }
    ArgBest best = {-INFINITY, 0x7fffffff};
#pragma unroll
    for (int j = 0; j < kRoPer; j++) {
        const int v = v0 + j * kRoThreads + tid;
        if (v < v1) {
            float val = grouped ? alpha * (expf(a[j] - m1) / d1) + (1.f - alpha) * (qs[j] * inv_nb) : a[j];
            best = better(best, ArgBest{val, v});
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ArgBest other = {__shfl_xor_sync(0xffffffffu, best.v, o), __shfl_xor_sync(0xffffffffu, best.i, o)};
        best = better(best, other);
    }
    if (lane == 0) {
        bv[warp] = best.v;
        bi[warp] = best.i;
    }
    __syncthreads();
    if (warp == 0) {
        ArgBest t = lane < (kRoThreads >> 5) ? ArgBest{bv[lane], bi[lane]} : ArgBest{-INFINITY, 0x7fffffff};
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ArgBest other = {__shfl_xor_sync(0xffffffffu, t.v, o), __shfl_xor_sync(0xffffffffu, t.i, o)};
            t = better(t, other);
        }
        if (lane == 0) {
            float *o2 = stats + ((size_t)b * nc + ck) * kRoRec;
            o2[3] = t.v;
            o2[4] = __int_as_float(t.i);
            __threadfence();
            const int tk = atomicAdd(tickets + b, 1);
            last_s = tk == nc - 1;
            if (last_s) atomicExch(tickets + b, 0);
        }
    }
    __syncthreads();
    if (last_s && warp == 0) {
        __threadfence();
        const float *rec = stats + (size_t)b * nc * kRoRec;
        ArgBest t = {-INFINITY, 0x7fffffff};
        for (int k = lane; k < nc; k += 32)
            t = better(t, ArgBest{__ldcg(rec + (size_t)k * kRoRec + 3), __float_as_int(__ldcg(rec + (size_t)k * kRoRec + 4))});
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ArgBest other = {__shfl_xor_sync(0xffffffffu, t.v, o), __shfl_xor_sync(0xffffffffu, t.i, o)};
            t = better(t, other);
        }
        if (lane == 0) {
            if (next) next[b] = t.i;
            if (alpha_out && grouped) alpha_out[b] = alpha;
            if (seq_len) seq_len[b] += advance;  // the step's last use of the lengths was the last layer's attention
        }
    }
}

// dbt_kv_export / dbt_kv_import: one K or V plane of one layer, [num_pages][n_kv][16][row_bytes], against a staging
// buffer in logical order [nb][nt][n_kv][row_bytes] for sequences seq_ids[s0..s0+nb) and positions t0..t0+nt-1,
// through the page table (Background, KV cache: the cache is addressed by position; paging is this library's).
__global__ void kv_copy_kernel(char *plane, const int32_t *page_table, int pt_stride, int num_pages, int n_kv, int row_bytes,
                               const int32_t *seq_ids, int s0, int nb, int t0, int nt, char *stage, int to_pool, int *status) {
    pdl_enter();
    const int vpr = row_bytes / 16;
    const size_t total = (size_t)nb * nt * n_kv * vpr;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int v = (int)(i % vpr);
    size_t r = i / vpr;
    const int h = (int)(r % n_kv);
    r /= n_kv;
    const int ti = (int)(r % nt), bi = (int)(r / nt);
    const int t = t0 + ti, seq = ld_mut(seq_ids + s0 + bi);
    int page = ld_mut(page_table + (size_t)seq * pt_stride + t / 16);
    if (page < 0 || page >= num_pages) {
        report(status, kStatusBadPage, page);
        return;
    }
    uint4 *pool_p = reinterpret_cast<uint4 *>(plane + (((size_t)page * n_kv + h) * 16 + (t & 15)) * row_bytes) + v;
    uint4 *stage_p = reinterpret_cast<uint4 *>(stage + (((size_t)bi * nt + ti) * n_kv + h) * row_bytes) + v;
    if (to_pool)
        *pool_p = *stage_p;
    else
        *stage_p = *pool_p;
}

__global__ void advance_len_kernel(int32_t *seq_len, int B, int n) {
    pdl_enter();
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) seq_len[b] += n;
}

// ---------------------------------------------------------------------------------------
// MoE (Eq. moe_layer, Eq. moe_budget, Section 4.3).

// Router: softmax over E logits, top-k by repeated "largest remaining, lowest index first",
// weights renormalised over the selection.  Replay: the branch row takes its primary twin's
// selection and weighs it with its own probabilities.  One warp per row; logits may arrive
// as split-K partials [nsplit][R][E] (summed in split order).
// ss != nullptr: the router GEMM ran on g * S (not yet divided by rms(S)); the row's factor comes
// from its per-tile shares of sum(S^2) and multiplies the logits here (the GEMM is linear).
__global__ void __launch_bounds__(32) route_kernel(const float *logits, int nsplit, size_t split_stride, int E, int Bc,
                                                   int k_p, int k_b, int kmax, int replay, int32_t *idx, float *wts,
                                                   int32_t *last, int last_stride_path, const float *ss, int ss_tiles,
                                                   int ss_ld, int d_norm, float eps) {
    DBT_TL_DECL;
    pdl_enter();
    DBT_TL_WAITED;
    extern __shared__ float smem[];
    float *own = smem, *sel = smem + E;  // own-row logits -> probabilities; selection-row logits
    int r = blockIdx.x, lane = threadIdx.x;
    int path = r / Bc;  // 0 primary, j >= 1 decode branch j (each branch routes for itself, fan-out k_b)
    int sel_row = (path && replay) ? r % Bc : r;
    int k = (path && !replay) ? k_b : k_p;
    // One round of loads: the row's norm shares and every split of this lane's experts are requested before
    // anything is added (16 splits x 2 experts in flight; the sums still run in split order).  Replay reads the
    // primary twin's logits too; otherwise the selection row is the row itself.
    const bool twin = sel_row != r;
    float ssa = 0.f, ssb = 0.f;
    if (ss)
        for (int t = lane; t < ss_tiles; t += 32) {
            ssa += __ldcg(ss + (size_t)t * ss_ld + r);
            if (twin) ssb += __ldcg(ss + (size_t)t * ss_ld + sel_row);
        }
    for (int e0 = 0; e0 < E; e0 += 64) {
        float a[2] = {0.f, 0.f}, b2[2] = {0.f, 0.f};
        for (int s0 = 0; s0 < nsplit; s0 += 16) {
            float va[2][16], vb[2][16];
#pragma unroll
            for (int u = 0; u < 2; u++)
#pragma unroll
                for (int j = 0; j < 16; j++) {
                    const int e = e0 + u * 32 + lane;
                    const bool on = e < E && s0 + j < nsplit;
                    va[u][j] = on ? __ldcg(logits + (size_t)(s0 + j) * split_stride + (size_t)r * E + e) : 0.f;
                    vb[u][j] = on && twin ? __ldcg(logits + (size_t)(s0 + j) * split_stride + (size_t)sel_row * E + e) : 0.f;
                }
#pragma unroll
            for (int u = 0; u < 2; u++)
#pragma unroll
                for (int j = 0; j < 16; j++) {
                    a[u] += va[u][j];
                    b2[u] += vb[u][j];
                }
        }
#pragma unroll
        for (int u = 0; u < 2; u++) {
            const int e = e0 + u * 32 + lane;
            if (e < E) {
                own[e] = a[u];
                sel[e] = twin ? b2[u] : a[u];
            }
        }
    }
    DBT_TL_MARK(0);
    float inv_own = 1.f, inv_sel = 1.f;
    if (ss) {
        inv_own = 1.f / sqrtf(warp_sum(ssa) / (float)d_norm + eps);
        inv_sel = twin ? 1.f / sqrtf(warp_sum(ssb) / (float)d_norm + eps) : inv_own;
    }
    float mx = -INFINITY;
    for (int e = lane; e < E; e += 32) {
        const float x = own[e] * inv_own;
        own[e] = x;
        sel[e] *= inv_sel;
        mx = fmaxf(mx, x);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int e = lane; e < E; e += 32) {
        float x = expf(own[e] - mx);
        own[e] = x;
        sum += x;
    }
    sum = warp_sum(sum);
    __syncwarp();
    DBT_TL_MARK(1);
    float tot = 0.f;
    int mine = -1;  // lane j keeps the j-th selection (k <= 64: two rounds of lanes at most)
    int mine2 = -1;
    for (int j = 0; j < k; j++) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int e = lane; e < E; e += 32) {
            float v = sel[e];
            if (v > bv || (v == bv && e < bi)) {  // NaN-free: taken entries are -inf
                bv = v;
                bi = e;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) {
                bv = ov;
                bi = oi;
            }
        }
        if (lane == 0) sel[bi] = -INFINITY;
        __syncwarp();
        tot += own[bi] / sum;
        if (j == lane) mine = bi;
        if (j == lane + 32) mine2 = bi;
    }
    DBT_TL_MARK(2);
    for (int j = lane; j < kmax; j += 32) {
        int e = j < k ? (j < 32 ? mine : mine2) : -1;
        idx[(size_t)r * kmax + j] = e;
        wts[(size_t)r * kmax + j] = j < k ? (own[e] / sum) / tot : 0.f;
        if (last) last[(size_t)path * last_stride_path + (size_t)(r - path * Bc) * kmax + j] = e;
    }
    DBT_TL_END("route");
}

// Per-expert lists of (row, slot) entries in ascending order, and the size of the union.
__global__ void moe_lists_kernel(const int32_t *idx, int R, int kmax, int E, int cap,
                                 int32_t *cnt, int32_t *list, int32_t *union_count) {
    pdl_enter();
    int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= E) return;
    int c = 0;
    for (int r = 0; r < R; r++)
        for (int j = 0; j < kmax; j++)
            if (idx[(size_t)r * kmax + j] == e) list[(size_t)e * cap + c++] = r * kmax + j;
    cnt[e] = c;
    if (c > 0 && union_count) atomicAdd(union_count, 1);
}

// Routed experts, gate/up + SwiGLU: every expert with a non-empty list streams its gate and up
// matrices once for all its entries of both paths.  grid (ceil(Fe/warps), E).
template <typename WT>
__global__ void __launch_bounds__(kLinWarps * 32) expert_gateup_kernel(
    const WT *__restrict__ Wg, const WT *__restrict__ Wu, int Fe, int d, const float *X, int kmax,
    const int32_t *cnt, const int32_t *list, int cap, float *Hexp) {
    pdl_enter();
    int e = blockIdx.y, n = cnt[e];
    if (n == 0) return;
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int f = blockIdx.x * kLinWarps + warp;
    if (f >= Fe) return;
    const WT *wg = Wg + ((size_t)e * Fe + f) * d, *wu = Wu + ((size_t)e * Fe + f) * d;
    const int32_t *li = list + (size_t)e * cap;
    for (int r0 = 0; r0 < n; r0 += kLinRT) {
        const float *xp[kLinRT];
        int ent[kLinRT];
#pragma unroll
        for (int r = 0; r < kLinRT; r++) {
            ent[r] = (r0 + r < n) ? li[r0 + r] : -1;
            xp[r] = ent[r] >= 0 ? X + (size_t)(ent[r] / kmax) * d : nullptr;
        }
        float ga[kLinRT], up[kLinRT];
        warp_dots<WT, kLinRT>(wg, xp, d, ga);
        warp_dots<WT, kLinRT>(wu, xp, d, up);
#pragma unroll
        for (int r = 0; r < kLinRT; r++)
            if (lane == r && ent[r] >= 0) Hexp[(size_t)ent[r] * Fe + f] = silu(ga[r]) * up[r];
    }
}

// Routed experts, down projection: Yexp[entry] = W_D[e] Hexp[entry].  grid (ceil(d/warps), E).
template <typename WT>
__global__ void __launch_bounds__(kLinWarps * 32) expert_down_kernel(
    const WT *__restrict__ Wd, int Fe, int d, const float *Hexp, const int32_t *cnt,
    const int32_t *list, int cap, float *Yexp) {
    pdl_enter();
    int e = blockIdx.y, n = cnt[e];
    if (n == 0) return;
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int f = blockIdx.x * kLinWarps + warp;
    if (f >= d) return;
    const WT *w = Wd + ((size_t)e * d + f) * Fe;
    const int32_t *li = list + (size_t)e * cap;
    for (int r0 = 0; r0 < n; r0 += kLinRT) {
        const float *xp[kLinRT];
        int ent[kLinRT];
#pragma unroll
        for (int r = 0; r < kLinRT; r++) {
            ent[r] = (r0 + r < n) ? li[r0 + r] : -1;
            xp[r] = ent[r] >= 0 ? Hexp + (size_t)ent[r] * Fe : nullptr;
        }
        float acc[kLinRT];
        warp_dots<WT, kLinRT>(w, xp, Fe, acc);
#pragma unroll
        for (int r = 0; r < kLinRT; r++)
            if (lane == r && ent[r] >= 0) Yexp[(size_t)ent[r] * d + f] = acc[r];
    }
}

// M_1 = sum_j w_1j Expert_j(m_1) + G(m_1);  M_2 = sum_j w_2j Expert_j(m_2) + G~(m_2) + c*M_1;
// S_i += M_i.  Slots are summed in slot order.  One block per primary row.
// gate_g != nullptr (Eq. matched_shared_expert): M_2 = sum_j w_2j Expert_j(m_2) + g_G * G(m_1), no c term.
__global__ void moe_combine_kernel(const float *Yexp, const float *Msh,
                                   const int32_t *idx, const float *wts, int kmax, int Bc,
                                   int grouped, const float *__restrict__ coup_c,
                                   const float *__restrict__ gate_g, int d, float *S) {
    pdl_enter();
    int b = blockIdx.x;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float m1 = 0.f;
        for (int j = 0; j < kmax; j++)
            if (idx[(size_t)b * kmax + j] >= 0) m1 = fmaf(wts[(size_t)b * kmax + j], Yexp[((size_t)b * kmax + j) * d + i], m1);
        float sh1 = Msh ? Msh[(size_t)b * d + i] : 0.f;
        if (Msh) m1 += sh1;
        S[(size_t)b * d + i] += m1;
        for (int jp = 1; jp < grouped; jp++) {  // `grouped` counts the paths present
            int r = jp * Bc + b;
            float m2 = 0.f;
            for (int j = 0; j < kmax; j++)
                if (idx[(size_t)r * kmax + j] >= 0)
                    m2 = fmaf(wts[(size_t)r * kmax + j], Yexp[((size_t)r * kmax + j) * d + i], m2);
            if (gate_g)
                m2 += gate_g[i] * sh1;
            else {
                if (Msh) m2 += Msh[(size_t)r * d + i];
                m2 += coup_c[i] * m1;
            }
            S[(size_t)r * d + i] += m2;
        }
    }
}

}  // namespace dbt
