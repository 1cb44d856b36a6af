// Shared device helpers for the Decode-Branch kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

namespace dbt {

constexpr int kWarp = 32;

// Device status word values (see dbt_sync_status).
enum : int { kStatusOk = 0, kStatusBadToken = 1, kStatusBadPage = 2, kStatusWaitExpired = 3 };

__device__ __forceinline__ void report(int *status, int code, int detail) {
    if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// Programmatic dependent launch: a kernel lets its successor start early, and waits for its
// predecessor's results before reading or writing anything that predecessor touches.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ unsigned long long gtime() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Timeline instrumentation (compile with -DDBT_TIMELINE): block 0 of every instrumented kernel
// appends (name tag, entry, after the dependency wait, end, four optional marks) in nanoseconds of %globaltimer to a
// device array that dbt_debug_timeline copies out.  Stores only: a printf would itself delay the
// end of the kernel and with it the next one's start.
#ifdef DBT_TIMELINE
constexpr int kTlMax = 16384;
__device__ unsigned long long g_tl[kTlMax * 8];
__device__ unsigned int g_tl_n;
__device__ __forceinline__ unsigned long long tl_tag(const char *s) {
    unsigned long long t = 0;
    for (int i = 0; i < 8 && s[i]; i++) t |= (unsigned long long)(unsigned char)s[i] << (8 * i);
    return t;
}
#define DBT_TL_DECL unsigned long long tl0_ = gtime(), tl1_ = 0, tlx_[4] = {0, 0, 0, 0}
#define DBT_TL_WAITED tl1_ = gtime()
#define DBT_TL_MARK(k) tlx_[k] = gtime()
#define DBT_TL_END(name) DBT_TL_END_IF(blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0, name)
#define DBT_TL_END_IF(cond, name)                                                          \
    if (threadIdx.x == 0 && (cond)) {                                                      \
        unsigned int i_ = atomicAdd(&g_tl_n, 1u);                                          \
        if (i_ < (unsigned)kTlMax) {                                                       \
            g_tl[8 * i_] = tl_tag(name);                                                   \
            g_tl[8 * i_ + 1] = tl0_;                                                       \
            g_tl[8 * i_ + 2] = tl1_;                                                       \
            g_tl[8 * i_ + 3] = gtime();                                                    \
            for (int k_ = 0; k_ < 4; k_++) g_tl[8 * i_ + 4 + k_] = tlx_[k_];               \
        }                                                                                  \
    }
#else
#define DBT_TL_DECL
#define DBT_TL_WAITED
#define DBT_TL_MARK(k)
#define DBT_TL_END(name)
#define DBT_TL_END_IF(cond, name)
#endif
__device__ __forceinline__ void pdl_enter() {
    pdl_launch_dependents();
    pdl_wait();
}
// Under programmatic dependent launch a kernel is resident before its predecessors have
// finished, so "read-only for the lifetime of the kernel" does not hold for anything another
// kernel of the step writes (sequence lengths, tokens, activations, partials, the KV pool):
// such pointers carry no `const __restrict__` (which would permit non-coherent loads), and
// scalars are read with ld_mut.
template <typename T>
__device__ __forceinline__ T ld_mut(const T *p) {
    return __ldcg(p);
}

// ---- storage-type loads: 8 consecutive elements widened to fp32 -------------------------
__device__ __forceinline__ void load8(const float *p, float (&v)[8]) {
    float4 a = *reinterpret_cast<const float4 *>(p);
    float4 b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8]) {
    uint4 u = *reinterpret_cast<const uint4 *>(p);
    uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; i++) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ float load1(const float *p) { return *p; }
__device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store1(float *p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide sum with a fixed reduction tree (deterministic). `scratch` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float *scratch) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[w] = v;
    __syncthreads();
    float t = (lane < nw) ? scratch[lane] : 0.f;
    return warp_sum(t);
}
__device__ __forceinline__ float block_max(float v, float *scratch) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) scratch[w] = v;
    __syncthreads();
    float t = (lane < nw) ? scratch[lane] : -INFINITY;
    return warp_max(t);
}

__device__ __forceinline__ float silu(float x) { return x / (1.f + expf(-x)); }

// Row bookkeeping shared by every kernel.  A launch covers `Bc = B*cn` primary rows (B
// sequences, cn consecutive positions each: cn = 1 in decode, a prompt chunk in prefill)
// followed, in grouped mode, by Bc branch rows.  Row r belongs to sequence (r % Bc) / cn at
// position seq_len[seq] + (r % Bc) % cn.
struct RowMap {
    int B, cn;
    __device__ __forceinline__ int Bc() const { return B * cn; }
    __device__ __forceinline__ int seq(int r) const { return (r % (B * cn)) / cn; }
    __device__ __forceinline__ int off(int r) const { return (r % (B * cn)) % cn; }
};

}  // namespace dbt
