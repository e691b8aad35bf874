// CTA-wide stable LSD radix sort of item ids by a 32-bit key table held in shared memory.
//
// One CTA of SORT_THREADS threads owns one instance.  The ids 0..n-1 are sorted
// ascending by (key[id] ^ flip), `nbits` low bits significant, 8 bits per pass; equal keys
// keep id order (the first pass reads ids in natural order, every pass is stable).  Each
// warp owns a contiguous chunk of positions; a pass is (1) per-warp digit counts by shared
// memory atomics, (2) one exclusive scan over the [digit][warp] count matrix, (3) a stable
// scatter in which the rank of an item among the equal digits of its 32-wide row comes from
// one ballot per digit bit.  The count matrix has a row stride of 33 words so that the 32
// lanes of a warp, which all address their own warp's column, spread over the banks.
#pragma once

#include "hos_common.cuh"

namespace hos {

template <typename IdxT>
struct SortSmem {
    // layout inside dynamic shared memory, all 16-byte aligned
    uint32_t* key;      // [n]
    IdxT* buf0;         // [n]
    IdxT* buf1;         // [n]
    uint32_t* cnt;      // [CNT_WORDS], entry (digit, warp) at digit * CNT_STRIDE + warp
    uint32_t* wsum;     // [SORT_WARPS]
};

constexpr int CNT_STRIDE = SORT_WARPS + 1;
constexpr int CNT_PER_THREAD = (RADIX * CNT_STRIDE + SORT_THREADS - 1) / SORT_THREADS;
constexpr int CNT_WORDS = CNT_PER_THREAD * SORT_THREADS;     // padded; the padding stays zero

__host__ __device__ inline size_t align16(size_t x) { return (x + 15) & ~size_t(15); }

template <typename IdxT>
__host__ __device__ inline size_t sort_smem_bytes(int n) {
    return align16(size_t(n) * 4) + 2 * align16(size_t(n) * sizeof(IdxT)) +
           size_t(CNT_WORDS) * 4 + SORT_WARPS * 4;
}

template <typename IdxT>
__device__ inline SortSmem<IdxT> sort_smem_carve(unsigned char* base, int n) {
    SortSmem<IdxT> s;
    s.key = reinterpret_cast<uint32_t*>(base);
    base += align16(size_t(n) * 4);
    s.buf0 = reinterpret_cast<IdxT*>(base);
    base += align16(size_t(n) * sizeof(IdxT));
    s.buf1 = reinterpret_cast<IdxT*>(base);
    base += align16(size_t(n) * sizeof(IdxT));
    s.cnt = reinterpret_cast<uint32_t*>(base);
    base += size_t(CNT_WORDS) * 4;
    s.wsum = reinterpret_cast<uint32_t*>(base);
    return s;
}

// Exclusive scan of cnt[0 .. CNT_WORDS) in place.  All SORT_THREADS threads call it.
__device__ inline void scan_counts(uint32_t* cnt, uint32_t* wsum) {
    constexpr int PER = CNT_PER_THREAD;                      // consecutive entries per thread
    const int t = threadIdx.x;
    uint32_t v[PER];
    uint32_t run = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        uint32_t c = cnt[t * PER + k];
        v[k] = run;
        run += c;
    }
    // inclusive warp scan of the thread totals
    uint32_t inc = run;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t y = __shfl_up_sync(FULL, inc, d);
        if (lane_id() >= d) inc += y;
    }
    if (lane_id() == 31) wsum[warp_id()] = inc;
    __syncthreads();
    if (warp_id() == 0) {
        uint32_t w = wsum[lane_id()];
        uint32_t winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t y = __shfl_up_sync(FULL, winc, d);
            if (lane_id() >= d) winc += y;
        }
        wsum[lane_id()] = winc - w;                          // exclusive warp offsets
    }
    __syncthreads();
    uint32_t base = wsum[warp_id()] + inc - run;
#pragma unroll
    for (int k = 0; k < PER; ++k) cnt[t * PER + k] = base + v[k];
    __syncthreads();
}

// Returns the buffer (buf0 or buf1) that holds the sorted ids.  nbits == 0 leaves ids in
// natural order.  Ends with a __syncthreads().
template <typename IdxT>
__device__ inline IdxT* block_radix_sort_ids(const SortSmem<IdxT>& s, int n, int nbits,
                                             uint32_t flip) {
    const int lane = lane_id(), warp = warp_id();
    const int chunk = (((n + SORT_WARPS - 1) / SORT_WARPS) + 31) & ~31;   // positions per warp
    const int lo = warp * chunk;
    const int hi = min(n, lo + chunk);
    IdxT* src = s.buf1;
    IdxT* dst = s.buf0;
    bool natural = true;                                     // first pass reads id = position

    if (nbits <= 0) {
        for (int i = threadIdx.x; i < n; i += SORT_THREADS) dst[i] = (IdxT)i;
        __syncthreads();
        return dst;
    }
    for (int shift = 0; shift < nbits; shift += RADIX_BITS) {
        const int nb = min(RADIX_BITS, nbits - shift);       // significant bits of this digit
        const uint32_t dmask = (1u << nb) - 1u;
        for (int i = threadIdx.x; i < CNT_WORDS; i += SORT_THREADS) s.cnt[i] = 0;
        __syncthreads();
        // (1) per-warp digit counts
        for (int row = lo; row < hi; row += 32) {
            const int pos = row + lane;
            if (pos < hi) {
                const uint32_t id = natural ? (uint32_t)pos : (uint32_t)src[pos];
                const uint32_t dig = ((s.key[id] ^ flip) >> shift) & dmask;
                atomicAdd(&s.cnt[dig * CNT_STRIDE + warp], 1u);
            }
        }
        __syncthreads();
        // (2) offsets
        scan_counts(s.cnt, s.wsum);
        // (3) stable scatter, four rows at a time: the key loads and ballots of the four rows
        //     are independent of each other; only the counter updates run row after row
        constexpr int G = 4;
        for (int row = lo; row < hi; row += 32 * G) {
            uint32_t id[G], dig[G];
            unsigned m[G];
            bool valid[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const int pos = row + 32 * g + lane;
                valid[g] = pos < hi;
                id[g] = valid[g] ? (natural ? (uint32_t)pos : (uint32_t)src[pos]) : 0u;
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                dig[g] = valid[g] ? (((s.key[id[g]] ^ flip) >> shift) & dmask) : 0u;
                m[g] = __ballot_sync(FULL, valid[g]);        // lanes of this row with my digit
            }
            if (nb == RADIX_BITS) {                          // the usual digit: no loop, constant shifts
#pragma unroll
                for (int b = 0; b < RADIX_BITS; ++b) {
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const bool bit = (dig[g] >> b) & 1u;
                        const unsigned bal = __ballot_sync(FULL, bit);
                        m[g] &= bit ? bal : ~bal;
                    }
                }
            } else {
                for (int b = 0; b < nb; ++b) {
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const bool bit = (dig[g] >> b) & 1u;
                        const unsigned bal = __ballot_sync(FULL, bit);
                        m[g] &= bit ? bal : ~bal;
                    }
                }
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint32_t base = valid[g] ? s.cnt[dig[g] * CNT_STRIDE + warp] : 0u;
                __syncwarp();
                if (valid[g]) {
                    dst[base + __popc(m[g] & ((1u << lane) - 1u))] = (IdxT)id[g];
                    if (lane == (__ffs(m[g]) - 1)) s.cnt[dig[g] * CNT_STRIDE + warp] = base + __popc(m[g]);
                }
                __syncwarp();
            }
        }
        __syncthreads();
        IdxT* t = src; src = dst; dst = t;
        natural = false;
    }
    return src;
}

}  // namespace hos
