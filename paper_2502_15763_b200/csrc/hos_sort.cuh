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
                if (HOS_IN(id, n, 103) && HOS_IN(dig * CNT_STRIDE + warp, CNT_WORDS, 101)) atomicAdd(&s.cnt[dig * CNT_STRIDE + warp], 1u);
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
                    if (HOS_IN(base + __popc(m[g] & ((1u << lane) - 1u)), n, 102)) dst[base + __popc(m[g] & ((1u << lane) - 1u))] = (IdxT)id[g];
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


// ---------------------------------------------------------------------------------------
// Bucket sort of items by a 32-bit key, for keys that spread out (the usual case).
//
// The order wanted -- key ascending over its low `nbits` bits, then id ascending -- is a total
// order of distinct pairs, so it does not matter in which order the items of a bucket arrive:
// the top bits of the key choose a bucket (shared-memory histogram, scan, scatter by atomic slot
// counters); a bucket entry is the rest of the key above the id (and, below both, whatever
// the caller wants to carry along) in one 32-bit word, with the bucket number in a 16-bit table
// beside it; and an item's final position is its bucket's start plus the number of entries of
// that bucket below its own.  Ranks are taken in SLOT order: the 32 lanes of a warp look at
// neighbouring buckets, so their reads of a bucket's entries fall on the same or on
// neighbouring words (no bank conflicts, equal trip counts), and their results land on
// neighbouring positions, so the caller can write them straight to global memory.  With about
// two buckets per item this is a few compares per item instead of a ranking vote per key bit
// and pass.  The counters are 16 bits wide, two to a word (no count or offset reaches 2^16).
// In the scan every thread owns a run of consecutive counter words; a spare word after each such
// run keeps the threads of a warp on different banks (without it their runs, a power of two long,
// start on two banks in all: at 2^15 buckets the scan alone took a quarter of the sort).
// The keys themselves are not kept in shared memory: the caller passes over its data once to
// count and once to place (bucket_sort_count / bucket_sort_place).
//
// The sort declines (plan or scan return false, nothing written) when an entry does not fit 32
// bits or the buckets are so uneven that the compares would cost more than the radix passes
// (sum of squared bucket sizes above BUCKET_WORK_MAX per item); the caller then takes
// block_radix_sort_ids.  One CTA of SORT_THREADS threads.
// ---------------------------------------------------------------------------------------
constexpr int BUCKET_BITS_MAX = 15;
constexpr int BUCKET_WORK_MAX = 96;

// Most bucket bits whose counters fit beside the entry and bucket tables (host and device agree).
constexpr size_t BUCKET_PAD_BYTES = 4 * SORT_THREADS;      // one spare counter word per thread
__host__ __device__ inline int bucket_bits_cap(int n) {
    // 2 KB for static shared memory
    const size_t room = SMEM_LIMIT - 2048 - BUCKET_PAD_BYTES - align16(size_t(n) * 4) - align16(size_t(n) * 2);
    int bb = BUCKET_BITS_MAX;
    while (bb > 10 && (size_t(2) << bb) > room) --bb;
    int want = 11;                                                           // about two buckets per item
    while (want < BUCKET_BITS_MAX && (1 << want) < 2 * n) ++want;
    return bb < want ? bb : want;
}
__host__ __device__ inline size_t bucket_sort_smem_bytes(int n) {
    return align16(size_t(n) * 4) + align16(size_t(n) * 2) + (size_t(2) << bucket_bits_cap(n)) + BUCKET_PAD_BYTES;
}

struct BucketSort {
    int bbits, low_bits, id_bits, xbits, n_words, n;
    int pad_shift;              // counter word w lives at cntw[w + (w >> pad_shift)]
    uint32_t kmask, lmask;
    uint32_t* ent;              // [n]  (rest of key << id_bits | id) << xbits | extra, in slot order
    uint16_t* bkt;              // [n]  bucket of every slot
    uint32_t* cntw;             // [2^(bbits-1) + spares] two 16-bit counters per word
};

// Layout and bit budget for n items with `nbits` significant key bits and `xbits` extra bits per
// entry.  False when an entry does not fit.  Uniform over the CTA.
__device__ inline bool bucket_sort_plan(BucketSort& B, unsigned char* smem, int n, int nbits, int xbits) {
    B.bbits = max(1, min(nbits, bucket_bits_cap(n)));
    B.low_bits = max(0, nbits - B.bbits);
    B.id_bits = n > 1 ? bit_width_u32((uint32_t)(n - 1)) : 1;
    B.xbits = xbits;
    B.n = n;
    B.n_words = 1 << (B.bbits - 1);
    // a thread's run in the scan is n_words / SORT_THREADS words (a power of two); no spares for runs of one
    B.pad_shift = B.n_words > SORT_THREADS ? B.bbits - 1 - (31 - __clz(SORT_THREADS)) : 31;
    B.kmask = nbits >= 32 ? 0xFFFFFFFFu : ((1u << nbits) - 1u);
    B.lmask = B.low_bits >= 32 ? 0xFFFFFFFFu : ((1u << B.low_bits) - 1u);
    B.ent = reinterpret_cast<uint32_t*>(smem);
    B.bkt = reinterpret_cast<uint16_t*>(smem + align16(size_t(n) * 4));
    B.cntw = reinterpret_cast<uint32_t*>(smem + align16(size_t(n) * 4) + align16(size_t(n) * 2));
    return B.low_bits + B.id_bits + xbits <= 32;
}

// Where counter word w is kept, and bucket b's 16-bit counter.
__device__ __forceinline__ uint32_t bucket_word_at(const BucketSort& B, uint32_t w) { return w + (w >> B.pad_shift); }
__device__ __forceinline__ uint32_t bucket_half_at(const BucketSort& B, uint32_t b) {
    return (bucket_word_at(B, b >> 1) << 1) | (b & 1u);
}

// Zeroes the counters.  Ends with a __syncthreads().
__device__ inline void bucket_sort_clear(const BucketSort& B) {
    const int n_kept = (int)bucket_word_at(B, (uint32_t)B.n_words);
    for (int i = threadIdx.x; i < n_kept; i += SORT_THREADS) B.cntw[i] = 0;
    __syncthreads();
}

__device__ __forceinline__ void bucket_sort_count(const BucketSort& B, uint32_t key) {
    const uint32_t b = (key & B.kmask) >> B.low_bits;
    if (HOS_IN(b >> 1, B.n_words, 111)) atomicAdd(&B.cntw[bucket_word_at(B, b >> 1)], 1u << ((b & 1u) << 4));
}

// Exclusive scan of the bucket counts (after every bucket_sort_count).  Starts and ends with a
// __syncthreads().  False when the buckets are too uneven.
__device__ inline bool bucket_sort_scan(const BucketSort& B, int n) {
    __shared__ uint32_t s_wsum[SORT_WARPS];
    __shared__ unsigned long long s_work;
    const int t = threadIdx.x;
    if (t == 0) s_work = 0;
    __syncthreads();
    const int per = (B.n_words + SORT_THREADS - 1) / SORT_THREADS;   // consecutive words per thread
    const int w0 = min(B.n_words, t * per), w1 = min(B.n_words, w0 + per);
    uint32_t run = 0;
    unsigned long long work = 0;
    const int at0 = (int)bucket_word_at(B, (uint32_t)w0);   // a run never crosses a spare word
    for (int w = w0; w < w1; ++w) {
        const uint32_t c = B.cntw[at0 + (w - w0)], a = c & 0xFFFFu, b = c >> 16;
        run += a + b;
        work += (unsigned long long)(a * a + b * b);
    }
    uint32_t inc = run;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(FULL, inc, d);
        if (lane_id() >= d) inc += y;
    }
    work = warp_sum_u64(work);
    if (lane_id() == 31) s_wsum[warp_id()] = inc;
    if (lane_id() == 0 && work) atomicAdd(&s_work, work);
    __syncthreads();
    const uint32_t wv = s_wsum[lane_id()];
    uint32_t acc = __reduce_add_sync(FULL, lane_id() < warp_id() ? wv : 0u) + inc - run;
    for (int w = w0; w < w1; ++w) {
        const uint32_t c = B.cntw[at0 + (w - w0)], a = c & 0xFFFFu, b = c >> 16;
        B.cntw[at0 + (w - w0)] = acc | ((acc + a) << 16);
        acc += a + b;
    }
    __syncthreads();
    return s_work <= (unsigned long long)BUCKET_WORK_MAX * (unsigned long long)n;
}

// First slot of bucket b; valid between bucket_sort_scan and the first bucket_sort_place.
__device__ __forceinline__ uint32_t bucket_sort_start(const BucketSort& B, uint32_t b) {
    return reinterpret_cast<const uint16_t*>(B.cntw)[bucket_half_at(B, b)];
}

// Scatter: the counter of the item's bucket walks from the bucket's start to its end.
__device__ __forceinline__ void bucket_sort_place(const BucketSort& B, uint32_t key, uint32_t id, uint32_t extra) {
    const uint32_t fk = key & B.kmask;
    const uint32_t b = fk >> B.low_bits, sh = (b & 1u) << 4;
    if (!HOS_IN(b >> 1, B.n_words, 111)) return;
    const uint32_t slot = (atomicAdd(&B.cntw[bucket_word_at(B, b >> 1)], 1u << sh) >> sh) & 0xFFFFu;
    if (!HOS_IN(slot, B.n, 112)) return;
    B.ent[slot] = ((((fk & B.lmask) << B.id_bits) | id) << B.xbits) | extra;
    B.bkt[slot] = (uint16_t)b;
}

// Final position of the item in slot s (after every bucket_sort_place and a __syncthreads());
// its key, id and extra bits come back through the references.
__device__ __forceinline__ uint32_t bucket_sort_rank(const BucketSort& B, int s, uint32_t& key, uint32_t& id,
                                                     uint32_t& extra) {
    const uint16_t* cnt16 = reinterpret_cast<const uint16_t*>(B.cntw);
    const uint32_t mine = B.ent[s], b = B.bkt[s];
    const bool b_ok = HOS_IN(b, 1 << B.bbits, 113);
    uint32_t start = (b_ok && b) ? cnt16[bucket_half_at(B, b - 1)] : 0u, end = b_ok ? cnt16[bucket_half_at(B, b)] : 0u;
    if (!HOS_IN(end, B.n + 1, 114) || !HOS_IN(start, end + 1, 114)) start = end = 0;
    uint32_t r = start, j = start;
    for (; j + 1 < end; j += 2) r += (B.ent[j] < mine ? 1u : 0u) + (B.ent[j + 1] < mine ? 1u : 0u);
    if (j < end) r += B.ent[j] < mine ? 1u : 0u;
    const uint32_t body = B.xbits >= 32 ? 0u : mine >> B.xbits;
    extra = B.xbits >= 32 ? mine : (mine & ((1u << B.xbits) - 1u));
    id = body & ((1u << B.id_bits) - 1u);                       // id_bits <= 15 for any supported n
    key = (b << B.low_bits) | (B.id_bits >= 32 ? 0u : body >> B.id_bits);
    return r;
}

}  // namespace hos
