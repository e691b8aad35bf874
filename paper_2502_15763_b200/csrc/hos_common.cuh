// Shared device helpers of the hos kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "hos.h"

namespace hos {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int SORT_THREADS = 1024;          // one CTA per instance for the smem-resident kernels
constexpr int SORT_WARPS = SORT_THREADS / 32;
constexpr int RADIX_BITS = 8;
constexpr int RADIX = 1 << RADIX_BITS;
constexpr int MAX_CLIENTS = 256;
constexpr int MAX_CAP = 256;
constexpr int MAX_REQ = 24384;          // the request table, two id buffers and the radix counters fill one CTA's shared memory
constexpr size_t SMEM_LIMIT = 227 * 1024;

// Per-instance facts left in the workspace by the estimate+sort kernel.
struct InstInfo {
    unsigned long long sum_T;
    uint32_t max_T;
    int32_t status;
};

// ---------------------------------------------------------------------------------------
// Bounds-checked build (-DHOS_DEBUG_BOUNDS; libhos_debug.so).  Every data-dependent index into
// shared or global memory goes through HOS_IN(index, limit, site): in the ordinary build it is
// the constant `true`; in the checked build an index outside [0, limit) is counted, the first
// one is kept with its site number, and the access is skipped -- nothing faults or traps.  The
// counters are per translation unit (no relocatable device code); hos_debug_bounds_violations()
// adds them up.
// ---------------------------------------------------------------------------------------
#ifdef HOS_DEBUG_BOUNDS
static __device__ unsigned int g_bounds_count;
static __device__ long long g_bounds_first[3];           // site, index, limit of the first violation
__device__ __forceinline__ bool bounds_ok(long long idx, long long limit, int site) {
    if (idx >= 0 && idx < limit) return true;
    if (atomicAdd(&g_bounds_count, 1u) == 0u) {
        g_bounds_first[0] = site; g_bounds_first[1] = idx; g_bounds_first[2] = limit;
    }
    return false;
}
#define HOS_IN(idx, limit, site) (::hos::bounds_ok((long long)(idx), (long long)(limit), (site)))
// one per translation unit with kernels: adds this unit's count, keeps the first violation seen
#define HOS_DEFINE_BOUNDS_READER(name)                                                        \
    void name(unsigned long long* count, long long* first) {                                  \
        unsigned int c = 0;                                                                   \
        long long f[3] = {0, 0, 0};                                                           \
        cudaMemcpyFromSymbol(&c, g_bounds_count, sizeof(c));                                  \
        cudaMemcpyFromSymbol(f, g_bounds_first, sizeof(f));                                   \
        if (c && !*count) { first[0] = f[0]; first[1] = f[1]; first[2] = f[2]; }              \
        *count += c;                                                                          \
    }
#else
#define HOS_IN(idx, limit, site) (true)
#define HOS_DEFINE_BOUNDS_READER(name) \
    void name(unsigned long long*, long long*) {}
#endif

__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }
__device__ __forceinline__ int warp_id() { return threadIdx.x >> 5; }

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(FULL, v, d);
    return v;
}
__device__ __forceinline__ long long warp_max_i64(long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        long long w = __shfl_xor_sync(FULL, v, d);
        v = w > v ? w : v;
    }
    return v;
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        unsigned long long w = __shfl_xor_sync(FULL, v, d);
        v = w > v ? w : v;
    }
    return v;
}

// Block-wide reductions for blocks of up to 1024 threads; `scratch` holds 32 entries.
// Every thread gets the result.  Contains __syncthreads().
__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v,
                                                            unsigned long long* scratch) {
    v = warp_sum_u64(v);
    __syncthreads();
    if (lane_id() == 0) scratch[warp_id()] = v;
    __syncthreads();
    int nw = (blockDim.x + 31) >> 5;
    unsigned long long t = (lane_id() < nw) ? scratch[lane_id()] : 0ull;
    return warp_sum_u64(t);
}
__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long v,
                                                            unsigned long long* scratch) {
    v = warp_max_u64(v);
    __syncthreads();
    if (lane_id() == 0) scratch[warp_id()] = v;
    __syncthreads();
    int nw = (blockDim.x + 31) >> 5;
    unsigned long long t = (lane_id() < nw) ? scratch[lane_id()] : 0ull;
    return warp_max_u64(t);
}

__device__ __forceinline__ int bit_width_u32(uint32_t v) { return 32 - __clz(v); }

// One pass of a CTA over the request tables of an instance: f(i, p_i, o_i, e_i, a_i) for every
// request, four requests per thread and 16-byte loads when the rows allow it.  ei may be oi
// itself (no separate estimates); ai may be null (then a_i = 0).
template <typename F>
__device__ __forceinline__ void for_each_request(const uint32_t* __restrict__ pi, const uint32_t* __restrict__ oi,
                                                 const uint32_t* __restrict__ ei, const int32_t* __restrict__ ai,
                                                 int n, F&& f) {
    const uintptr_t bits = reinterpret_cast<uintptr_t>(pi) | reinterpret_cast<uintptr_t>(oi) |
                           reinterpret_cast<uintptr_t>(ei) | reinterpret_cast<uintptr_t>(ai);
    if ((n & 3) == 0 && (bits & 15) == 0) {
        for (int i4 = threadIdx.x; i4 < (n >> 2); i4 += blockDim.x) {
            const uint4 pv = __ldg(reinterpret_cast<const uint4*>(pi) + i4);
            const uint4 ov = __ldg(reinterpret_cast<const uint4*>(oi) + i4);
            const uint4 ev = ei != oi ? __ldg(reinterpret_cast<const uint4*>(ei) + i4) : ov;
            const int4 av = ai ? __ldg(reinterpret_cast<const int4*>(ai) + i4) : make_int4(0, 0, 0, 0);
            f(4 * i4 + 0, pv.x, ov.x, ev.x, av.x);
            f(4 * i4 + 1, pv.y, ov.y, ev.y, av.y);
            f(4 * i4 + 2, pv.z, ov.z, ev.z, av.z);
            f(4 * i4 + 3, pv.w, ov.w, ev.w, av.w);
        }
    } else {
        for (int i = threadIdx.x; i < n; i += blockDim.x) f(i, pi[i], oi[i], ei[i], ai ? ai[i] : 0);
    }
}

// Duration of a prefill stage over `tokens` prompt tokens: affine, or by level (Eq. 5-7).
__device__ __forceinline__ uint32_t prefill_us(const hos_cost_model& cm, uint32_t tokens) {
    if (cm.n_levels == 0) return cm.prefill_fixed_us + cm.prefill_per_token_us * tokens;
    uint32_t t = cm.level_time_us[cm.n_levels - 1];
    for (int l = (int)cm.n_levels - 2; l >= 0; --l)
        if (tokens <= cm.level_cap_tokens[l]) t = cm.level_time_us[l];
    return t;
}
// Most prompt tokens one prefill stage can take (and the longest admissible prompt).
__host__ __device__ __forceinline__ uint32_t stage_cap_tokens(const hos_cost_model& cm) {
    return cm.n_levels ? cm.level_cap_tokens[cm.n_levels - 1] : 0xFFFFFFFFu;
}

}  // namespace hos
