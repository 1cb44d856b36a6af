// Elementwise kernels that sit between the tensor-core GEMMs of the bf16 path.  Each one also
// sums the split-K partials of the GEMM before it, in split order (deterministic).
//
// Rows are path-major: Bc primary rows, then Bc rows per decode branch (one branch in the main text, K-1 with
// more decode branches, Appendix C.1).  A kernel that couples a branch row to its primary twin runs one block
// per (primary row, ..., branch): blockIdx.z is the branch, its row is (blockIdx.z + 1) * Bc + b.  Every block
// recomputes what it needs of the primary row from the partials (a pure function of them); only the blocks of
// the first branch store the primary row's results.
#pragma once

#include "dbt_common.cuh"

namespace dbt {

// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): the two-term form the GEMM consumes.
// lo_off is the element offset of the lo plane (0: store hi only).
__device__ __forceinline__ void store_split(__nv_bfloat16 *dst, size_t idx, size_t lo_off, float x) {
    __nv_bfloat16 hi = __float2bfloat16_rn(x);
    dst[idx] = hi;
    if (lo_off) dst[idx + lo_off] = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// Sum of one output's split-K partials, in split order; the loads go out four at a time so that
// the sum costs one or two L2 round trips instead of one per split.
__device__ __forceinline__ float sum_splits(const float *P, size_t split_stride, int nsplit, size_t off) {
    const float *p = P + off;
    float m = 0.f;
    int s = 0;
    for (; s + 4 <= nsplit; s += 4) {
        float a = __ldcg(p), b = __ldcg(p + split_stride), c = __ldcg(p + 2 * split_stride), e = __ldcg(p + 3 * split_stride);
        m += a;
        m += b;
        m += c;
        m += e;
        p += 4 * split_stride;
    }
    if (s + 2 <= nsplit) {
        float a = __ldcg(p), b = __ldcg(p + split_stride);
        m += a;
        m += b;
        p += 2 * split_stride;
        s += 2;
    }
    if (s < nsplit) m += __ldcg(p);
    return m;
}

// The same for K outputs at once: the loads of all K outputs (two splits of each) are in flight
// together.  Each output is still added in split order.
template <int K, int NB = (K <= 2 ? 4 : 2)>  // NB splits per batch: K * NB loads in flight
__device__ __forceinline__ void sum_splits_k(const float *P, size_t split_stride, int nsplit, const size_t (&off)[K],
                                             float (&out)[K]) {
#pragma unroll
    for (int k = 0; k < K; k++) out[k] = 0.f;
    for (int s = 0; s < nsplit; s += NB) {
        float v[NB][K];
#pragma unroll
        for (int j = 0; j < NB; j++)
#pragma unroll
            for (int k = 0; k < K; k++) v[j][k] = s + j < nsplit ? __ldcg(P + (size_t)(s + j) * split_stride + off[k]) : 0.f;
#pragma unroll
        for (int j = 0; j < NB; j++)
#pragma unroll
            for (int k = 0; k < K; k++) out[k] += v[j][k];
    }
}

// 1/rms of a row from its per-tile shares of sum(x^2) (ss[t][ss_ld], summed in tile order);
// 1 when ss == nullptr (the GEMM input was already normalised).
__device__ __forceinline__ float row_scale(const float *ss, int ss_tiles, int ss_ld, int row, int d_norm, float eps) {
    if (!ss) return 1.f;
    float a = 0.f;
    for (int t0 = 0; t0 < ss_tiles; t0 += 8) {  // eight shares in flight at a time, added in tile order
        float v[8];
#pragma unroll
        for (int j = 0; j < 8; j++) v[j] = t0 + j < ss_tiles ? __ldcg(ss + (size_t)(t0 + j) * ss_ld + row) : 0.f;
#pragma unroll
        for (int j = 0; j < 8; j++) a += v[j];
    }
    return 1.f / sqrtf(a / (float)d_norm + eps);
}

// The same for two rows at once (a primary row and its branch twin), their loads in flight together.
__device__ __forceinline__ void row_scale2(const float *ss, int ss_tiles, int ss_ld, int row_a, int row_b, int d_norm,
                                           float eps, float &rs_a, float &rs_b) {
    rs_a = rs_b = 1.f;
    if (!ss) return;
    float a = 0.f, b = 0.f;
    for (int t0 = 0; t0 < ss_tiles; t0 += 8) {
        float va[8], vb[8];
#pragma unroll
        for (int j = 0; j < 8; j++) {
            va[j] = t0 + j < ss_tiles ? __ldcg(ss + (size_t)(t0 + j) * ss_ld + row_a) : 0.f;
            vb[j] = t0 + j < ss_tiles ? __ldcg(ss + (size_t)(t0 + j) * ss_ld + row_b) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 8; j++) {
            a += va[j];
            b += vb[j];
        }
    }
    rs_a = 1.f / sqrtf(a / (float)d_norm + eps);
    rs_b = 1.f / sqrtf(b / (float)d_norm + eps);
}

// Residual update without the row-wide reduction: S += sum_s P[s] (mode 1) or, with the c
// coupling, M_2 += c*M_1 first (mode 2); the next GEMM's input is g * S (un-normalised, two bf16
// planes) and each 256-column block leaves its share of sum(S^2) per row in ss_out[tile][row].
// The consumer of that GEMM multiplies by 1/rms (the GEMM is linear), see row_scale.
// grid (primary rows, d / 256, branches): every thread owns one column of a row and of its branch twin.
// MULTI = false (at most one decode branch): the block index of the branch is a compile-time zero -- with it
// a run-time value the compiler orders this kernel's loads worse and a launch takes 3.5 us longer.
template <bool MULTI>
__global__ void __launch_bounds__(256) resid_wide_kernel(float *S, const float *P, int nsplit, size_t split_stride,
                                                         int mode, const float *__restrict__ coup_c, int Bc, int grouped,
                                                         const float *__restrict__ g_next, int d, __nv_bfloat16 *Xb,
                                                         size_t lo_off, float *ss_out, int ss_ld) {
    DBT_TL_DECL;
    pdl_launch_dependents();
    __shared__ float scratch[64];
    int b = blockIdx.x, i = blockIdx.y * blockDim.x + threadIdx.x;
    // The gain and the coupling are weights: they are read once per step, so they come from HBM, not from L2.
    // Requested before the dependency wait, that latency passes while the GEMM before this kernel still runs.
    float gn = 1.f, cc = 0.f;
    if (i < d) {
        gn = g_next ? g_next[i] : 1.f;
        cc = mode >= 2 ? coup_c[i] : 0.f;
    }
    pdl_wait();
    DBT_TL_WAITED;
    const bool first = MULTI ? blockIdx.z == 0 : true;  // the first branch's blocks also own the primary row
    const int r2 = MULTI ? ((int)blockIdx.z + 1) * Bc + b : Bc + b;
    float q1 = 0.f, q2 = 0.f;
    if (i < d) {
        // every load of this thread goes out before the first use: S of both rows and all splits of both
        // rows' partials (up to 16 splits in one round)
        size_t o1 = (size_t)b * d + i, o2 = (size_t)r2 * d + i;
        // (the primary row is loaded by every branch's block, stored by the first: a predicate on the load would
        // split this round of loads)
        float s1 = __ldcg(S + o1), s2 = grouped ? __ldcg(S + o2) : 0.f;
        const size_t offs[2] = {o1, grouped && mode != 3 ? o2 : o1};
        float mm[2];
        sum_splits_k<2, 16>(P, split_stride, nsplit, offs, mm);
        s1 += mm[0];
        if (first) {
            S[o1] = s1;
            store_split(Xb, o1, lo_off, gn * s1);
        }
        q1 = s1 * s1;
        if (grouped) {
            float m2 = mm[1];
            if (mode == 2) m2 += cc * mm[0];
            if (mode == 3) m2 = cc * mm[0];  // Eq. matched_attention: coup_c carries g_A
            s2 += m2;
            S[o2] = s2;
            store_split(Xb, o2, lo_off, gn * s2);
            q2 = s2 * s2;
        }
    }
    // both rows' shares in one pass over the block
    q1 = warp_sum(q1);
    q2 = warp_sum(q2);
    int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if (lane == 0) {
        scratch[warp] = q1;
        scratch[32 + warp] = q2;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float a1 = 0.f, a2 = 0.f;
        for (int w2 = 0; w2 < nw; w2++) {
            a1 += scratch[w2];
            a2 += scratch[32 + w2];
        }
        if (first) ss_out[(size_t)blockIdx.y * ss_ld + b] = a1;
        if (grouped) ss_out[(size_t)blockIdx.y * ss_ld + r2] = a2;
    }
    DBT_TL_END("resid_wide");
}

// Residual update + RMSNorm feeding the next GEMM.
//   mode 0: S unchanged                                   (after the embedding, after an MoE layer)
//   mode 1: S += sum_s P[s]                               (S-bar_i = S_i + Attn_i W_O)
//   mode 2: M = sum_s P[s]; M_2 += c * M_1; S += M        (Eq. mlp: M_2 = H~_2 W_D + c*M_1)
//   mode 3: M_1 = sum_s P[s]; M_2 = g * M_1; S += M        (Eq. matched_attention; coup_c carries g_A)
// then Xb = bf16(g * S / rms(S)) (apply_norm) or bf16(S).  Block (j, 0, z) handles primary source row
// j*src_mul + src_add and, in grouped mode, its twin of branch z; outputs go to rows j and (z+1)*n_out + j.
__global__ void __launch_bounds__(1024) resid_norm_kernel(float *S, const float *P, int nsplit,
                                                         size_t split_stride, int mode,
                                                         const float *__restrict__ coup_c, int Bc, int grouped,
                                                         const float *__restrict__ g, float eps, int d, int apply_norm,
                                                         int src_mul, int src_add, __nv_bfloat16 *Xb,
                                                         size_t lo_off, float *Xf) {
    DBT_TL_DECL;
    pdl_enter();
    DBT_TL_WAITED;
    __shared__ float scratch[32];
    int j = blockIdx.x, n_out = gridDim.x;
    const bool first = blockIdx.z == 0;
    const int zb = (int)blockIdx.z + 1;
    int r1 = j * src_mul + src_add, r2 = zb * Bc + r1;
    float ss1 = 0.f, ss2 = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v1 = first ? S[(size_t)r1 * d + i] : 0.f, m1 = 0.f;
        float v2 = grouped ? S[(size_t)r2 * d + i] : 0.f;
        float sm[2] = {0.f, 0.f};
        if (mode != 0) {
            const size_t offs[2] = {(size_t)r1 * d + i, (size_t)(grouped && mode != 3 ? r2 : r1) * d + i};
            sum_splits_k<2, 8>(P, split_stride, nsplit, offs, sm);  // (1024 threads per block: 64 registers each)
            m1 = sm[0];
            v1 += m1;
            if (first) S[(size_t)r1 * d + i] = v1;
        }
        ss1 += v1 * v1;
        if (grouped) {
            if (mode != 0) {
                float m2 = sm[1];
                if (mode == 2) m2 += coup_c[i] * m1;
                if (mode == 3) m2 = coup_c[i] * m1;
                v2 += m2;
                S[(size_t)r2 * d + i] = v2;
            }
            ss2 += v2 * v2;
        }
    }
    float inv1 = 1.f, inv2 = 1.f;
    if (apply_norm) {
        ss1 = block_sum(ss1, scratch);
        inv1 = 1.f / sqrtf(ss1 / (float)d + eps);
        if (grouped) {
            ss2 = block_sum(ss2, scratch);
            inv2 = 1.f / sqrtf(ss2 / (float)d + eps);
        }
    }
    // each thread re-reads only the elements of S it wrote itself (same index stride)
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float gi = apply_norm ? g[i] : 1.f;
        if (first) {
            float x1 = gi * S[(size_t)r1 * d + i] * inv1;
            store_split(Xb, (size_t)j * d + i, lo_off, x1);
            if (Xf) Xf[(size_t)j * d + i] = x1;
        }
        if (grouped) {
            float x2 = gi * S[(size_t)r2 * d + i] * inv2;
            store_split(Xb, (size_t)(zb * n_out + j) * d + i, lo_off, x2);
            if (Xf) Xf[(size_t)(zb * n_out + j) * d + i] = x2;
        }
    }
    DBT_TL_END("resid_norm");
}

// After the Q|K|V GEMM: sum the splits, RoPE on Q (both paths) and K (primary), the a coupling
// Q~_2 = Q_2 + a*Q_1 (Eq. asymattn), append K_1,V_1 to the paged cache.  P rows are
// [q_dim | kv_dim (K) | kv_dim (V)].  grid (primary rows, n_q + n_kv heads), one thread per
// rotation pair of the head.
template <typename KT>
__global__ void __launch_bounds__(64) qkv_epilogue_kernel(
    const float *P, int nsplit, size_t split_stride, float *Q, RowMap rm, int grouped,
    int n_q, int n_kv, int dh, const float *__restrict__ coup_a, const float2 *__restrict__ rope_tab,
    const int32_t *seq_len, const int32_t *__restrict__ page_table, int pt_stride, int num_pages,
    int page_size, KT *kpool, KT *vpool, int *status, const float *ss, int ss_tiles, int ss_ld, int d_norm,
    float eps) {
    DBT_TL_DECL;
    pdl_enter();
    DBT_TL_WAITED;
    int item = blockIdx.x, hh = blockIdx.y, i = threadIdx.x, Bc = rm.Bc();
    const bool first = blockIdx.z == 0;
    const int twin = ((int)blockIdx.z + 1) * Bc + item;
    int half = dh / 2;
    if (i >= half) return;
    int seq = rm.seq(item), pos = ld_mut(seq_len + seq) + rm.off(item);
    int q_dim = n_q * dh, kv_dim = n_kv * dh, ldp = q_dim + 2 * kv_dim;
    float2 t = rope_tab[(size_t)pos * half + i];
    size_t p1 = (size_t)item * ldp, p2 = (size_t)twin * ldp;
    float rs1, rs2;  // 1/rms when the GEMM input was g*S
    row_scale2(ss, ss_tiles, ss_ld, item, grouped ? twin : item, d_norm, eps, rs1, rs2);
    if (hh < n_q) {
        int o0 = hh * dh + i, o1 = o0 + half;
        const size_t offs[4] = {p1 + o0, p1 + o1, grouped ? p2 + o0 : p1 + o0, grouped ? p2 + o1 : p1 + o1};
        float sm[4];
        sum_splits_k<4>(P, split_stride, nsplit, offs, sm);
        float x0 = rs1 * sm[0], x1 = rs1 * sm[1];
        float r0 = x0 * t.x - x1 * t.y, r1 = x1 * t.x + x0 * t.y;
        float *q1 = Q + (size_t)item * q_dim;
        if (first) {
            q1[o0] = r0;
            q1[o1] = r1;
        }
        if (grouped) {
            float y0 = rs2 * sm[2], y1 = rs2 * sm[3];
            float *q2 = Q + (size_t)twin * q_dim;
            q2[o0] = (y0 * t.x - y1 * t.y) + coup_a[o0] * r0;
            q2[o1] = (y1 * t.x + y0 * t.y) + coup_a[o1] * r1;
        }
        DBT_TL_END("qkv_epilogue");
        return;
    }
    if (!first) return;  // K_1, V_1 exist once: the branches have none
    int gk = hh - n_q;
    int page = page_table[(size_t)seq * pt_stride + pos / page_size];
    if (page < 0 || page >= num_pages) {
        if (i == 0) report(status, kStatusBadPage, page);
        return;
    }
    int slot = pos % page_size;
    size_t base = (((size_t)page * n_kv + gk) * page_size + slot) * dh;
    size_t ko = p1 + q_dim + gk * dh + i, vo = ko + kv_dim;
    const size_t offs[4] = {ko, ko + half, vo, vo + half};
    float sm[4];
    sum_splits_k<4>(P, split_stride, nsplit, offs, sm);
    float x0 = rs1 * sm[0], x1 = rs1 * sm[1];
    store1(kpool + base + i, x0 * t.x - x1 * t.y);
    store1(kpool + base + i + half, x1 * t.x + x0 * t.y);
    store1(vpool + base + i, rs1 * sm[2]);
    store1(vpool + base + i + half, rs1 * sm[3]);
}

// After the gate|up GEMM: H = SiLU(gate) * up; H~_2 = H_2 + b * H_1 (Eq. mlp); bf16 out for
// the down projection.  P rows are [F gate | F up].  grid (primary rows, F / 256).
__global__ void __launch_bounds__(256) swiglu_couple_kernel(const float *P, int nsplit,
                                                            size_t split_stride, int F, int Bc, int grouped,
                                                            const float *__restrict__ coup_b,
                                                            __nv_bfloat16 *Hb, size_t lo_off, const float *ss,
                                                            int ss_tiles, int ss_ld, int d_norm, float eps) {
    DBT_TL_DECL;
    pdl_launch_dependents();
    __shared__ float sh[34];
    int b = blockIdx.x, f = blockIdx.y * blockDim.x + threadIdx.x;
    const bool act = f < F;
    const float cb = (act && grouped && coup_b) ? coup_b[f] : 0.f;  // a weight, from HBM: requested before the wait
    pdl_wait();
    DBT_TL_WAITED;
    const bool first = blockIdx.z == 0;
    const int rb = grouped ? ((int)blockIdx.z + 1) * Bc + b : b, lane = threadIdx.x & 31;
    // The norm shares of the block's two rows are fetched once, by the first warp (lanes 0..15 the
    // primary row, 16..31 its twin), requested before the partials so that they travel together,
    // and handed to the block through shared memory: a few hundred blocks would otherwise all
    // hammer the same few lines.
    float myss = 0.f;
    if (ss && threadIdx.x < 32)
        for (int t = lane & 15; t < ss_tiles; t += 16) myss += __ldcg(ss + (size_t)t * ss_ld + (lane < 16 ? b : rb));
    size_t p1 = (size_t)b * 2 * F + (act ? f : 0);
    size_t p2 = grouped ? (size_t)rb * 2 * F + (act ? f : 0) : p1;
    const size_t offs[4] = {p1, p1 + F, p2, p2 + F};
    float sm[4] = {0.f, 0.f, 0.f, 0.f};
    if (act) sum_splits_k<4, 4>(P, split_stride, nsplit, offs, sm);
    if (threadIdx.x < 32) {
        sh[lane] = myss;
        __syncwarp();
        if ((lane & 15) == 0) {
            float a = 0.f;
            for (int j = 0; j < 16; j++) a += sh[lane + j];
            sh[32 + (lane >> 4)] = ss ? 1.f / sqrtf(a / (float)d_norm + eps) : 1.f;
        }
    }
    __syncthreads();
    if (act) {
        float rs1 = sh[32], rs2 = sh[33];
        float h1 = silu(rs1 * sm[0]) * (rs1 * sm[1]);
        if (first) store_split(Hb, (size_t)b * F + f, lo_off, h1);
        if (grouped) {
            float h2 = silu(rs2 * sm[2]) * (rs2 * sm[3]);
            h2 += cb * h1;
            store_split(Hb, (size_t)rb * F + f, lo_off, h2);
        }
    }
    DBT_TL_END("swiglu");
}

// ---- prompt chunks: many primary rows, no branch --------------------------------------------------
// The three kernels above give every thread one output element (latency counts there: a decode step has a
// few dozen rows).  A prompt chunk has up to a few thousand rows and these kernels become streams of
// 10..140 MB: here every thread takes four consecutive elements (16-byte loads, 8-byte bf16 stores) of a
// primary row.  Same arithmetic per element; the partial sums of sum(S^2) are added in another order.

__device__ __forceinline__ float4 ldcg4(const float *p) { return __ldcg(reinterpret_cast<const float4 *>(p)); }

// Four values as two bf16 planes (see store_split), 8 bytes per plane.
__device__ __forceinline__ void store_split4(__nv_bfloat16 *dst, size_t idx, size_t lo_off, float4 x) {
    __nv_bfloat162 h0 = __floats2bfloat162_rn(x.x, x.y), h1 = __floats2bfloat162_rn(x.z, x.w);
    uint2 hv = make_uint2(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1));
    *reinterpret_cast<uint2 *>(dst + idx) = hv;
    if (lo_off) {
        __nv_bfloat162 l0 = __floats2bfloat162_rn(x.x - __low2float(h0), x.y - __high2float(h0));
        __nv_bfloat162 l1 = __floats2bfloat162_rn(x.z - __low2float(h1), x.w - __high2float(h1));
        *reinterpret_cast<uint2 *>(dst + idx + lo_off) =
            make_uint2(*reinterpret_cast<uint32_t *>(&l0), *reinterpret_cast<uint32_t *>(&l1));
    }
}

__device__ __forceinline__ float4 sum_splits4(const float *P, size_t split_stride, int nsplit, size_t off) {
    float4 m = ldcg4(P + off);
    for (int s = 1; s < nsplit; s++) {
        float4 v = ldcg4(P + (size_t)s * split_stride + off);
        m.x += v.x, m.y += v.y, m.z += v.z, m.w += v.w;
    }
    return m;
}

// resid_wide_kernel for R primary rows: S += sum_s P[s]; Xb = g_next * S as two planes; the share of
// sum(S^2) of every (row, 256-column tile).  grid (ceil(R / 4), d / 256), 64 threads per row.  d % 4 == 0.
__global__ void __launch_bounds__(256) resid_rows_kernel(float *S, const float *P, int nsplit, size_t split_stride,
                                                         const float *__restrict__ g_next, int R, int d,
                                                         __nv_bfloat16 *Xb, size_t lo_off, float *ss_out, int ss_ld) {
    pdl_launch_dependents();
    __shared__ float scratch[8];
    const int sub = threadIdx.x >> 6, row = blockIdx.x * 4 + sub, i = blockIdx.y * 256 + (threadIdx.x & 63) * 4;
    const bool act = row < R && i < d;
    float4 gn = make_float4(1.f, 1.f, 1.f, 1.f);
    if (act && g_next) gn = *reinterpret_cast<const float4 *>(g_next + i);
    pdl_wait();
    float q = 0.f;
    if (act) {
        size_t o = (size_t)row * d + i;
        float4 s = ldcg4(S + o), m = sum_splits4(P, split_stride, nsplit, o);
        s.x += m.x, s.y += m.y, s.z += m.z, s.w += m.w;
        *reinterpret_cast<float4 *>(S + o) = s;
        store_split4(Xb, o, lo_off, make_float4(gn.x * s.x, gn.y * s.y, gn.z * s.z, gn.w * s.w));
        q = s.x * s.x + s.y * s.y + s.z * s.z + s.w * s.w;
    }
    q = warp_sum(q);
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = q;
    __syncthreads();
    if ((threadIdx.x & 63) == 0 && row < R) ss_out[(size_t)blockIdx.y * ss_ld + row] = scratch[2 * sub] + scratch[2 * sub + 1];
}

// swiglu_couple_kernel for R primary rows: H = SiLU(rs * gate) * (rs * up) as two planes.
// grid (R, ceil(F / 1024)).  F % 4 == 0.
__global__ void __launch_bounds__(256) swiglu_rows_kernel(const float *P, int nsplit, size_t split_stride, int F,
                                                          __nv_bfloat16 *Hb, size_t lo_off, const float *ss, int ss_tiles,
                                                          int ss_ld, int d_norm, float eps) {
    pdl_launch_dependents();
    __shared__ float rs_s;
    const int row = blockIdx.x, f = (blockIdx.y * 256 + threadIdx.x) * 4;
    pdl_wait();
    float a = 0.f;
    if (ss && threadIdx.x < 32)
        for (int t = threadIdx.x; t < ss_tiles; t += 32) a += __ldcg(ss + (size_t)t * ss_ld + row);
    float4 gt = make_float4(0.f, 0.f, 0.f, 0.f), up = gt;
    if (f < F) {
        size_t o = (size_t)row * 2 * F + f;
        gt = sum_splits4(P, split_stride, nsplit, o);
        up = sum_splits4(P, split_stride, nsplit, o + F);
    }
    if (threadIdx.x < 32) {
        a = warp_sum(a);
        if (threadIdx.x == 0) rs_s = ss ? 1.f / sqrtf(a / (float)d_norm + eps) : 1.f;
    }
    __syncthreads();
    if (f < F) {
        const float rs = rs_s;
        float4 h = make_float4(silu(rs * gt.x) * (rs * up.x), silu(rs * gt.y) * (rs * up.y), silu(rs * gt.z) * (rs * up.z),
                               silu(rs * gt.w) * (rs * up.w));
        store_split4(Hb, (size_t)row * F + f, lo_off, h);
    }
}

// qkv_epilogue_kernel for R primary rows of a bf16 cache: 1/rms, RoPE on Q and K, append K_1, V_1.
// grid (R, ceil((n_q + n_kv) * (dh / 8) / 256)): a thread takes four consecutive rotation pairs of a head.
__global__ void __launch_bounds__(256) qkv_rows_kernel(const float *P, int nsplit, size_t split_stride, float *Q, RowMap rm,
                                                       int n_q, int n_kv, int dh, const float2 *__restrict__ rope_tab,
                                                       const int32_t *seq_len, const int32_t *__restrict__ page_table,
                                                       int pt_stride, int num_pages, int page_size, __nv_bfloat16 *kpool,
                                                       __nv_bfloat16 *vpool, int *status, const float *ss, int ss_tiles,
                                                       int ss_ld, int d_norm, float eps) {
    pdl_launch_dependents();
    __shared__ float rs_s;
    const int item = blockIdx.x, half = dh / 2, per_head = half / 4;
    const int w = blockIdx.y * 256 + threadIdx.x, hh = w / per_head, i = (w % per_head) * 4;
    const bool act = hh < n_q + n_kv;
    pdl_wait();
    float a = 0.f;
    if (ss && threadIdx.x < 32)
        for (int t = threadIdx.x; t < ss_tiles; t += 32) a += __ldcg(ss + (size_t)t * ss_ld + item);
    const int seq = rm.seq(item), pos = ld_mut(seq_len + seq) + rm.off(item);
    const int q_dim = n_q * dh, kv_dim = n_kv * dh, ldp = q_dim + 2 * kv_dim;
    const size_t p1 = (size_t)item * ldp;
    const bool is_q = hh < n_q;
    float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), x1 = x0, v0 = x0, v1 = x0, c = x0, sn = x0;
    int page = 0;
    size_t o0 = 0;
    if (act) {
        const float4 t0 = *reinterpret_cast<const float4 *>(rope_tab + (size_t)pos * half + i);
        const float4 t1 = *reinterpret_cast<const float4 *>(rope_tab + (size_t)pos * half + i + 2);
        c = make_float4(t0.x, t0.z, t1.x, t1.z);
        sn = make_float4(t0.y, t0.w, t1.y, t1.w);
        o0 = is_q ? (size_t)hh * dh + i : (size_t)q_dim + (size_t)(hh - n_q) * dh + i;
        x0 = sum_splits4(P, split_stride, nsplit, p1 + o0);
        x1 = sum_splits4(P, split_stride, nsplit, p1 + o0 + half);
        if (!is_q) {
            v0 = sum_splits4(P, split_stride, nsplit, p1 + o0 + kv_dim);
            v1 = sum_splits4(P, split_stride, nsplit, p1 + o0 + kv_dim + half);
            page = page_table[(size_t)seq * pt_stride + pos / page_size];
        }
    }
    if (threadIdx.x < 32) {
        a = warp_sum(a);
        if (threadIdx.x == 0) rs_s = ss ? 1.f / sqrtf(a / (float)d_norm + eps) : 1.f;
    }
    __syncthreads();
    if (!act) return;
    const float rs = rs_s;
    x0 = make_float4(rs * x0.x, rs * x0.y, rs * x0.z, rs * x0.w);
    x1 = make_float4(rs * x1.x, rs * x1.y, rs * x1.z, rs * x1.w);
    const float4 r0 = make_float4(x0.x * c.x - x1.x * sn.x, x0.y * c.y - x1.y * sn.y, x0.z * c.z - x1.z * sn.z,
                                  x0.w * c.w - x1.w * sn.w);
    const float4 r1 = make_float4(x1.x * c.x + x0.x * sn.x, x1.y * c.y + x0.y * sn.y, x1.z * c.z + x0.z * sn.z,
                                  x1.w * c.w + x0.w * sn.w);
    if (is_q) {
        float *q1 = Q + (size_t)item * q_dim + o0;
        *reinterpret_cast<float4 *>(q1) = r0;
        *reinterpret_cast<float4 *>(q1 + half) = r1;
        return;
    }
    if (page < 0 || page >= num_pages) {
        if (i == 0) report(status, kStatusBadPage, page);
        return;
    }
    const size_t base = (((size_t)page * n_kv + (hh - n_q)) * page_size + pos % page_size) * dh + i;
    auto st4 = [](__nv_bfloat16 *dst, float4 v) {
        __nv_bfloat162 a2 = __floats2bfloat162_rn(v.x, v.y), b2 = __floats2bfloat162_rn(v.z, v.w);
        *reinterpret_cast<uint2 *>(dst) = make_uint2(*reinterpret_cast<uint32_t *>(&a2), *reinterpret_cast<uint32_t *>(&b2));
    };
    st4(kpool + base, r0);
    st4(kpool + base + half, r1);
    st4(vpool + base, make_float4(rs * v0.x, rs * v0.y, rs * v0.z, rs * v0.w));
    st4(vpool + base + half, make_float4(rs * v1.x, rs * v1.y, rs * v1.z, rs * v1.w));
}

// Eq. embeddings for the fused path: S^0 = RMSNorm(E[x]) and, for the first layer's Q|K|V GEMM,
// the input g_next * S^0 as two bf16 planes plus sum(S^0 ^2) per row (tile 0 carries the whole
// sum, the other tile slots are zeroed).  One block per row.
template <typename WT>
__global__ void __launch_bounds__(256) embed_fused_kernel(const int32_t *tokens, int n, int p0, RowMap rm,
                                                          const WT *__restrict__ E1, const WT *__restrict__ E2,
                                                          const float *__restrict__ g, float eps, int d, int V,
                                                          float *S, const float *__restrict__ g_next,
                                                          __nv_bfloat16 *Xb, size_t lo_off, float *ss_out, int ss_ld,
                                                          int ss_tiles, int *status) {
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
    float inv = 1.f / sqrtf(ss / (float)d + eps), sq = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float s0 = g[i] * load1(e + i) * inv;
        S[(size_t)r * d + i] = s0;
        store_split(Xb, (size_t)r * d + i, lo_off, g_next[i] * s0);
        sq += s0 * s0;
    }
    sq = block_sum(sq, scratch);
    for (int t = threadIdx.x; t < ss_tiles; t += blockDim.x) ss_out[(size_t)t * ss_ld + r] = t == 0 ? sq : 0.f;
}

// ---- MoE on tensor cores: rows sorted by expert ---------------------------------------------

// Per-expert row lists -> offsets and the sorted position of every (row, slot) entry.  Entries of
// one expert keep ascending (row, slot) order; experts follow each other in index order.
// One block, one thread per expert (E <= blockDim.x <= 1024); the offsets come from a two-level shuffle scan.
__global__ void __launch_bounds__(1024) moe_sort_kernel(const int32_t *idx, int R, int kmax, int E, int32_t *cnt,
                                                        int32_t *off, int32_t *pos, int32_t *union_count) {
    DBT_TL_DECL;
    pdl_enter();
    DBT_TL_WAITED;
    __shared__ int s_wsum[32];
    __shared__ int s_idx[4096];  // the selections, staged once (larger lists are read from global memory)
    const int n = R * kmax;
    // Long lists (prompt chunks, large batches): counts and positions through shared-memory atomics by all
    // threads.  The order of an expert's rows is then arbitrary, which no value depends on (every row's products
    // are its own, whatever its place in the tile).  Short lists keep the ascending order below.
    const bool parallel = n > 512;
    __shared__ int s_cnt[1024], s_fill[1024];
    const bool staged = !parallel && n <= 4096;
    if (staged)
        for (int i = threadIdx.x; i < n; i += blockDim.x) s_idx[i] = idx[i];
    if (parallel) {
        for (int i = threadIdx.x; i < 1024; i += blockDim.x) s_cnt[i] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int ex = idx[i];
            if (ex >= 0 && ex < E) atomicAdd(&s_cnt[ex], 1);
        }
    }
    __syncthreads();
    const int32_t *src = staged ? s_idx : idx;
    const int e = threadIdx.x, lane = e & 31, wp = e >> 5;
    int c = 0;
    if (parallel) {
        c = e < E ? s_cnt[e] : 0;
    } else if (e < E) {
        for (int i = 0; i < n; i++) c += src[i] == e;
    }
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_wsum[wp] = incl;
    const int uni = __syncthreads_count(c > 0);
    if (wp == 0) {
        int v = lane < (int)(blockDim.x >> 5) ? s_wsum[lane] : 0, w = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        s_wsum[lane] = w - v;  // experts before this warp's
    }
    __syncthreads();
    const int my_off = s_wsum[wp] + incl - c;
    if (e < E) {
        cnt[e] = c;
        off[e] = my_off;
        if (parallel) {
            s_fill[e] = my_off;
        } else {
            int k = 0;
            for (int i = 0; i < n && k < c; i++)
                if (src[i] == e) pos[i] = my_off + k++;
        }
    }
    if (parallel) {
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int ex = idx[i];
            if (ex >= 0 && ex < E) pos[i] = atomicAdd(&s_fill[ex], 1);
        }
    }
    if (e == E - 1) off[E] = my_off + c;
    if (e == 0 && union_count) *union_count = uni;
    DBT_TL_END("moe_sort");
}

// Copy each entry's activation row (both bf16 planes) to its sorted position.  ss != nullptr: the rows
// hold g * S, not yet divided by rms(S); the row's factor 1/rms goes to rs_sorted[position] for the
// SwiGLU kernel behind the per-expert gate|up GEMM.
__global__ void __launch_bounds__(256) moe_gather_kernel(const __nv_bfloat16 *Xb, size_t lo_in, const int32_t *idx,
                                                         const int32_t *pos, int kmax, int d, __nv_bfloat16 *Xs,
                                                         size_t lo_out, const float *ss, int ss_tiles, int ss_ld,
                                                         float eps, float *rs_sorted) {
    DBT_TL_DECL;
    // Wait first, then let the per-expert GEMM in: by the time one of its CTAs is resident the sort kernel's lists
    // are final, so it may read them (and request its first weight tiles) before its own dependency wait.
    pdl_wait();
    pdl_launch_dependents();
    DBT_TL_WAITED;
    int entry = blockIdx.x;
    if (idx[entry] < 0) return;
    if (ss && threadIdx.x < 32) {
        float a = 0.f;
        for (int t = threadIdx.x; t < ss_tiles; t += 32) a += __ldcg(ss + (size_t)t * ss_ld + entry / kmax);
        a = warp_sum(a);
        if (threadIdx.x == 0) rs_sorted[pos[entry]] = 1.f / sqrtf(a / (float)d + eps);
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(Xb + (size_t)(entry / kmax) * d);
    uint4 *dst = reinterpret_cast<uint4 *>(Xs + (size_t)pos[entry] * d);
    for (int i = threadIdx.x; i < d / 8; i += blockDim.x) {
        dst[i] = src[i];
        if (lo_out) dst[i + lo_out / 8] = src[i + lo_in / 8];
    }
    DBT_TL_END("moe_gath");
}

// H = SiLU(gate) * up on the sorted rows; Pe rows are [Fe gate | Fe up] (one split).  rs (nullable):
// the rows' 1/rms factors when the GEMM ran on inputs not yet divided by it.
__global__ void __launch_bounds__(256) moe_swiglu_kernel(const float *Pe, const int32_t *off_total, int Fe,
                                                         __nv_bfloat16 *Hs, size_t lo_off, const float *rs) {
    DBT_TL_DECL;
    pdl_enter();
    DBT_TL_WAITED;
    int p = blockIdx.x, f = blockIdx.y * blockDim.x + threadIdx.x;
    if (p >= *off_total || f >= Fe) return;
    const float sc = rs ? __ldcg(rs + p) : 1.f;
    float h = silu(sc * Pe[(size_t)p * 2 * Fe + f]) * (sc * Pe[(size_t)p * 2 * Fe + Fe + f]);
    store_split(Hs, (size_t)p * Fe + f, lo_off, h);
    DBT_TL_END("moe_swig");
}

// M_1 = sum_j w_1j Expert_j(m_1) + G(m_1);  M_2 = sum_j w_2j Expert_j(m_2) + G~(m_2) + c*M_1;
// S_i += M_i.  Ys: expert outputs at sorted positions; Psh: split-K partials of the shared
// expert's down projection (nullptr: no shared expert).  One block per primary row.
// gate_g != nullptr (Eq. matched_shared_expert): M_2 = sum_j w_2j Expert_j(m_2) + g_G * G(m_1), no c
// term; Psh then holds primary rows only.
// Xn != nullptr (grid (Bc, ceil(d / 256)), 256 threads): the block also leaves the next layer's GEMM
// input g_next * S (two bf16 planes, the 1/rms factor is applied after that GEMM) and its 256-column
// share of sum(S^2) for both rows, as resid_wide_kernel does.
template <bool MULTI>
__global__ void __launch_bounds__(256) moe_combine_sorted_kernel(const float *Ys, const float *Psh, int nsplit,
                                                                 size_t split_stride, const int32_t *idx,
                                                                 const int32_t *pos, const float *wts, int kmax, int Bc,
                                                                 int grouped, const float *__restrict__ coup_c,
                                                                 const float *__restrict__ gate_g, int d, float *S,
                                                                 const float *__restrict__ g_next, __nv_bfloat16 *Xn,
                                                                 size_t lo_off, float *ss_out, int ss_ld) {
    DBT_TL_DECL;
    pdl_enter();
    DBT_TL_WAITED;
    __shared__ float scratch[64];
    float q1 = 0.f, q2 = 0.f;
    int b = blockIdx.x;
    // the row's selections (weights, sorted positions) once, then all expert rows of a column in
    // flight together; terms are added in slot order
    constexpr int KM = 8;
    const bool first = MULTI ? blockIdx.z == 0 : true;
    const int r2 = MULTI ? ((int)blockIdx.z + 1) * Bc + b : Bc + b;
    for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < d; i += gridDim.y * blockDim.x) {
        float m1 = 0.f, m2 = 0.f;
        // Everything that does not depend on the routing is requested first: the residual rows and (up to 8
        // splits of) the shared expert's partials; they travel while the selections, then the expert rows, arrive.
        const float s1_in = first ? __ldcg(S + (size_t)b * d + i) : 0.f, s2_in = grouped ? __ldcg(S + (size_t)r2 * d + i) : 0.f;
        const size_t offs[2] = {(size_t)b * d + i, (size_t)(grouped && !gate_g ? r2 : b) * d + i};
        const bool early = Psh && nsplit <= 8;
        float pv[8][2];
#pragma unroll
        for (int sp = 0; sp < 8; sp++) {
            pv[sp][0] = early && sp < nsplit ? __ldcg(Psh + (size_t)sp * split_stride + offs[0]) : 0.f;
            pv[sp][1] = early && sp < nsplit ? __ldcg(Psh + (size_t)sp * split_stride + offs[1]) : 0.f;
        }
        for (int j0 = 0; j0 < kmax; j0 += KM) {
            // selections, weights and sorted positions of both rows in one round, the expert rows in the next
            int e1[KM], e2[KM], p1[KM], p2[KM];
            float y1[KM], w1[KM], y2[KM], w2[KM];
#pragma unroll
            for (int j = 0; j < KM; j++) {
                const bool in = j0 + j < kmax;
                const size_t o1 = (size_t)b * kmax + j0 + j, o2 = (size_t)r2 * kmax + j0 + j;
                e1[j] = in ? idx[o1] : -1;
                p1[j] = in ? pos[o1] : 0;
                w1[j] = in ? wts[o1] : 0.f;
                e2[j] = in && grouped ? idx[o2] : -1;
                p2[j] = in && grouped ? pos[o2] : 0;
                w2[j] = in && grouped ? wts[o2] : 0.f;
            }
#pragma unroll
            for (int j = 0; j < KM; j++) {
                if (e1[j] < 0) w1[j] = 0.f;
                if (e2[j] < 0) w2[j] = 0.f;
                y1[j] = e1[j] >= 0 ? __ldcg(Ys + (size_t)p1[j] * d + i) : 0.f;
                y2[j] = e2[j] >= 0 ? __ldcg(Ys + (size_t)p2[j] * d + i) : 0.f;
            }
#pragma unroll
            for (int j = 0; j < KM; j++) {
                if (j0 + j < kmax && w1[j] != 0.f) m1 = fmaf(w1[j], y1[j], m1);
                if (j0 + j < kmax && w2[j] != 0.f) m2 = fmaf(w2[j], y2[j], m2);
            }
        }
        if (Psh) {
            float sm[2] = {0.f, 0.f};
            if (early) {
#pragma unroll
                for (int sp = 0; sp < 8; sp++) {
                    sm[0] += pv[sp][0];
                    sm[1] += pv[sp][1];
                }
            } else {
                sum_splits_k<2, 8>(Psh, split_stride, nsplit, offs, sm);
            }
            m1 += sm[0];
            m2 += gate_g ? gate_g[i] * sm[0] : sm[1];
        }
        const float gn = Xn ? g_next[i] : 0.f;
        if (first) {
            const float v1 = s1_in + m1;
            S[(size_t)b * d + i] = v1;
            if (Xn) store_split(Xn, (size_t)b * d + i, lo_off, gn * v1);
            q1 += v1 * v1;
        }
        if (grouped) {
            if (!gate_g) m2 += coup_c[i] * m1;
            const float v2 = s2_in + m2;
            S[(size_t)r2 * d + i] = v2;
            if (Xn) store_split(Xn, (size_t)r2 * d + i, lo_off, gn * v2);
            q2 += v2 * v2;
        }
    }
    if (Xn) {  // (uniform per launch) the block's share of both rows' sum(S^2)
        q1 = warp_sum(q1);
        q2 = warp_sum(q2);
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
        if (lane == 0) {
            scratch[warp] = q1;
            scratch[32 + warp] = q2;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float a1 = 0.f, a2 = 0.f;
            for (int w2 = 0; w2 < nw; w2++) {
                a1 += scratch[w2];
                a2 += scratch[32 + w2];
            }
            if (first) ss_out[(size_t)blockIdx.y * ss_ld + b] = a1;
            if (grouped) ss_out[(size_t)blockIdx.y * ss_ld + r2] = a2;
        }
    }
    DBT_TL_END("moe_comb");
}

// moe_combine_sorted_kernel for R primary rows of a prompt chunk (no branch): S += sum_j w_j Expert_j(m) + G(m); the next
// layer's GEMM input g_next * S as two planes and the shares of sum(S^2).  grid (ceil(R / 4), d / 256), 64 threads
// per row, four consecutive columns per thread.  d % 4 == 0.
__global__ void __launch_bounds__(256) moe_combine_rows_kernel(const float *Ys, const float *Psh, int nsplit, size_t split_stride,
                                                               const int32_t *idx, const int32_t *pos, const float *wts,
                                                               int kmax, int R, int d, float *S,
                                                               const float *__restrict__ g_next, __nv_bfloat16 *Xn,
                                                               size_t lo_off, float *ss_out, int ss_ld) {
    pdl_launch_dependents();
    __shared__ float scratch[8];
    const int sub = threadIdx.x >> 6, row = blockIdx.x * 4 + sub, i = blockIdx.y * 256 + (threadIdx.x & 63) * 4;
    const bool act = row < R && i < d;
    float4 gn = make_float4(1.f, 1.f, 1.f, 1.f);
    if (act && Xn) gn = *reinterpret_cast<const float4 *>(g_next + i);
    pdl_wait();
    float q = 0.f;
    if (act) {
        const size_t o = (size_t)row * d + i;
        float4 s = ldcg4(S + o), m = make_float4(0.f, 0.f, 0.f, 0.f);
        constexpr int KM = 8;
        for (int j0 = 0; j0 < kmax; j0 += KM) {
            int e1[KM], p1[KM];
            float w1[KM];
            float4 y[KM];
#pragma unroll
            for (int j = 0; j < KM; j++) {
                const bool in = j0 + j < kmax;
                const size_t oj = (size_t)row * kmax + j0 + j;
                e1[j] = in ? idx[oj] : -1;
                p1[j] = in ? pos[oj] : 0;
                w1[j] = in ? wts[oj] : 0.f;
            }
#pragma unroll
            for (int j = 0; j < KM; j++) y[j] = e1[j] >= 0 ? ldcg4(Ys + (size_t)p1[j] * d + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < KM; j++)
                if (e1[j] >= 0 && w1[j] != 0.f) {
                    m.x = fmaf(w1[j], y[j].x, m.x);
                    m.y = fmaf(w1[j], y[j].y, m.y);
                    m.z = fmaf(w1[j], y[j].z, m.z);
                    m.w = fmaf(w1[j], y[j].w, m.w);
                }
        }
        if (Psh) {
            float4 sh = sum_splits4(Psh, split_stride, nsplit, o);
            m.x += sh.x, m.y += sh.y, m.z += sh.z, m.w += sh.w;
        }
        s.x += m.x, s.y += m.y, s.z += m.z, s.w += m.w;
        *reinterpret_cast<float4 *>(S + o) = s;
        if (Xn) store_split4(Xn, o, lo_off, make_float4(gn.x * s.x, gn.y * s.y, gn.z * s.z, gn.w * s.w));
        q = s.x * s.x + s.y * s.y + s.z * s.z + s.w * s.w;
    }
    if (Xn) {
        q = warp_sum(q);
        if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = q;
        __syncthreads();
        if ((threadIdx.x & 63) == 0 && row < R) ss_out[(size_t)blockIdx.y * ss_ld + row] = scratch[2 * sub] + scratch[2 * sub + 1];
    }
}

// Sum split partials into a plain fp32 matrix (used by the operator-level GEMM entry point).
__global__ void reduce_splits_kernel(const float *P, int nsplit, size_t split_stride, size_t n,
                                     float *Y) {
    pdl_enter();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) Y[i] = sum_splits(P, split_stride, nsplit, i);
}

__global__ void f32_to_bf16_kernel(const float *X, size_t n, __nv_bfloat16 *Y) {
    pdl_enter();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) Y[i] = __float2bfloat16_rn(X[i]);
}

}  // namespace dbt
