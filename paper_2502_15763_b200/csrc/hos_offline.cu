// Offline request scheduling kernels (Eq. 26-30 of arXiv 2502.15763):
//   k_estimate_sort  T_i and the per-instance order (T descending, index ascending)
//   k_lpt            longest-first list scheduling, one warp per instance
//   k_local_search   rounds of best move / pairwise swap off the critical client
//   k_lower_bound    Eq. 31-32 and the packing relaxations
#include "hos_common.cuh"
#include "hos_kernels.h"
#include "hos_sort.cuh"

namespace hos {

// ---------------------------------------------------------------------------------------
// Estimate + segmented sort.  One CTA per instance; the whole segment lives in shared
// memory: the T table, two id buffers and the radix counters.
// ---------------------------------------------------------------------------------------
template <typename IdxT>
__global__ void __launch_bounds__(SORT_THREADS, 1)
k_estimate_sort(const uint32_t* __restrict__ p, const uint32_t* __restrict__ o, int n_req,
                long long kv_budget, uint32_t e_p, uint32_t e_o,
                uint32_t* __restrict__ T_sorted, uint32_t* __restrict__ order,
                InstInfo* __restrict__ info, int32_t* __restrict__ status_out, int n_pad) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ unsigned long long red[32];
    SortSmem<IdxT> s = sort_smem_carve<IdxT>(smem_raw, n_req);
    const int inst = blockIdx.x;
    const uint32_t* pi = p + (size_t)inst * n_req;
    const uint32_t* oi = o + (size_t)inst * n_req;

    unsigned long long sum = 0, mx = 0, bad = 0;
    for (int i = threadIdx.x; i < n_req; i += SORT_THREADS) {
        const uint32_t pp = pi[i], oo = oi[i];
        const unsigned long long t = (unsigned long long)e_p * pp + (unsigned long long)e_o * oo;
        if (pp == 0 || oo == 0 || (long long)pp + (long long)oo > kv_budget || t > 0xFFFFFFFFull) bad = 1;
        s.key[i] = (uint32_t)t;
        sum += t;
        mx = t > mx ? t : mx;
    }
    sum = block_sum_u64(sum, red);
    mx = block_max_u64(mx, red);
    bad = block_max_u64(bad, red);
    __syncthreads();
    if (threadIdx.x == 0) {
        info[inst].sum_T = sum;
        info[inst].max_T = (uint32_t)mx;
        info[inst].status = bad ? HOS_ST_INVALID : 0;
        if (status_out) status_out[inst] = bad ? HOS_ST_INVALID : 0;
    }
    if (bad) return;                                  // uniform: every thread sees the same value

    const int nbits = bit_width_u32((uint32_t)mx);
    const uint32_t flip = nbits >= 32 ? 0xFFFFFFFFu : ((1u << nbits) - 1u);   // descending T
    const IdxT* sorted = block_radix_sort_ids<IdxT>(s, n_req, nbits, flip);

    uint32_t* Ts = T_sorted + (size_t)inst * n_pad;
    uint32_t* od = order + (size_t)inst * n_pad;
    for (int r = threadIdx.x; r < n_req; r += SORT_THREADS) {
        const uint32_t id = sorted[r];
        od[r] = id;
        Ts[r] = s.key[id];
    }
}

// ---------------------------------------------------------------------------------------
// LPT list scheduling.  One warp per instance: client j = slot * 32 + lane.  The chain of
// n_req dependent argmin steps runs on packed keys (load - base) << JB | j, so that one
// 32-bit warp min gives both the least load and, on ties, the lowest client.  The loads stay
// within max_T of their minimum (each item lands on the current minimum), which bounds the
// packed field between re-basings; instances that do not fit use 64-bit loads.
// ---------------------------------------------------------------------------------------
template <int KPL>
__global__ void __launch_bounds__(32)
k_lpt(const uint32_t* __restrict__ T_sorted, const uint32_t* __restrict__ order,
      const InstInfo* __restrict__ info, int n_req, int n_pad, int n_clients,
      int32_t* __restrict__ assign, long long* __restrict__ load_out,
      long long* __restrict__ makespan_out) {
    constexpr int JB = (KPL == 1) ? 5 : (KPL == 2) ? 6 : (KPL == 4) ? 7 : 8;
    const int inst = blockIdx.x;
    const int lane = threadIdx.x;
    const InstInfo inf = info[inst];
    int32_t* asg = assign + (size_t)inst * n_req;
    if (inf.status) {
        for (int i = lane; i < n_req; i += 32) asg[i] = -1;
        for (int j = lane; j < n_clients; j += 32) load_out[(size_t)inst * n_clients + j] = 0;
        if (lane == 0) makespan_out[inst] = 0;
        return;
    }
    const uint32_t* Ts = T_sorted + (size_t)inst * n_pad;
    const uint32_t* od = order + (size_t)inst * n_pad;

    long long load[KPL];
#pragma unroll
    for (int k = 0; k < KPL; ++k) load[k] = 0;

    // packed path is safe when (max_T * (2 + ceil(32 / M)) + 1) << JB fits 32 bits
    const unsigned long long span =
        (unsigned long long)inf.max_T * (2ull + (unsigned long long)((32 + n_clients - 1) / n_clients)) + 1ull;
    const bool packed = (span << JB) < 0xFFFFFFFFull;

    if (packed) {
        uint32_t key[KPL];
#pragma unroll
        for (int k = 0; k < KPL; ++k) {
            const int j = k * 32 + lane;
            key[k] = (j < n_clients) ? (uint32_t)j : 0xFFFFFFFFu;
        }
        unsigned long long rebased = 0;                 // sum of the bases subtracted so far
        uint32_t tv_next = (lane < n_req) ? Ts[lane] : 0u;
        uint32_t rq_next = (lane < n_req) ? od[lane] : 0u;
        for (int r0 = 0; r0 < n_req; r0 += 32) {
            const int r = r0 + lane;
            const uint32_t tsh = tv_next << JB;         // this chunk's items, already in key units
            const uint32_t rq = rq_next;
            const int rn = r + 32;                      // prefetch the next chunk behind the chain
            tv_next = (rn < n_req) ? Ts[rn] : 0u;
            rq_next = (rn < n_req) ? od[rn] : 0u;
            const int steps = min(32, n_req - r0);
            uint32_t mine = 0;
            for (int sidx = 0; sidx < steps; ++sidx) {
                uint32_t m = key[0];
#pragma unroll
                for (int k = 1; k < KPL; ++k) m = min(m, key[k]);
                const uint32_t g = __reduce_min_sync(FULL, m);
                const uint32_t j = g & ((1u << JB) - 1u);
                const uint32_t t = __shfl_sync(FULL, tsh, sidx);
                const bool own = lane == (int)(j & 31u);
#pragma unroll
                for (int k = 0; k < KPL; ++k) key[k] += (own && (int)(j >> 5) == k) ? t : 0u;
                mine = (lane == sidx) ? j : mine;
            }
            if (r < n_req) asg[rq] = (int32_t)mine;
            // re-base: subtract the current least relative load from every real key
            uint32_t m = key[0];
#pragma unroll
            for (int k = 1; k < KPL; ++k) m = min(m, key[k]);
            const uint32_t base = (__reduce_min_sync(FULL, m) >> JB) << JB;
            rebased += base >> JB;
#pragma unroll
            for (int k = 0; k < KPL; ++k)
                if (k * 32 + lane < n_clients) key[k] -= base;
        }
#pragma unroll
        for (int k = 0; k < KPL; ++k)
            if (k * 32 + lane < n_clients) load[k] = (long long)(rebased + (key[k] >> JB));
    } else {
        for (int r0 = 0; r0 < n_req; r0 += 32) {
            const int r = r0 + lane;
            const uint32_t tv = (r < n_req) ? Ts[r] : 0u;
            const uint32_t rq = (r < n_req) ? od[r] : 0u;
            const int steps = min(32, n_req - r0);
            uint32_t mine = 0;
            for (int sidx = 0; sidx < steps; ++sidx) {
                long long bl = 0x7FFFFFFFFFFFFFFFll;
                int bj = 0x7FFFFFFF;
#pragma unroll
                for (int k = 0; k < KPL; ++k) {
                    const int j = k * 32 + lane;
                    if (j < n_clients && load[k] < bl) { bl = load[k]; bj = j; }   // k ascending: lowest j first
                }
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    const long long ol = __shfl_xor_sync(FULL, bl, d);
                    const int oj = __shfl_xor_sync(FULL, bj, d);
                    if (ol < bl || (ol == bl && oj < bj)) { bl = ol; bj = oj; }
                }
                const uint32_t t = __shfl_sync(FULL, tv, sidx);
                const bool own = lane == (bj & 31);
#pragma unroll
                for (int k = 0; k < KPL; ++k) load[k] += (own && (bj >> 5) == k) ? (long long)t : 0ll;
                mine = (lane == sidx) ? (uint32_t)bj : mine;
            }
            if (r < n_req) asg[rq] = (int32_t)mine;
        }
    }
    long long mx = 0;
#pragma unroll
    for (int k = 0; k < KPL; ++k) {
        const int j = k * 32 + lane;
        if (j < n_clients) {
            load_out[(size_t)inst * n_clients + j] = load[k];
            mx = load[k] > mx ? load[k] : mx;
        }
    }
    mx = warp_max_i64(mx);
    if (lane == 0) makespan_out[inst] = mx;
}

// ---------------------------------------------------------------------------------------
// Local search.  One CTA per (instance, copy); the instance stays in shared memory for all
// rounds: T by rank, client by rank, request index by rank, the critical client's members.
//
// A round looks for the minimum of (v, i, k, u) over every move (u = -1, d = T_i) and swap
// (d = T_i - T_u > 0) off the critical client jmax, v = max(Lmax - d, load_k + d).  For a
// fixed (k, u), v falls while 2 d < Lmax - load_k and rises afterwards, so only two members
// of jmax can win: the one with the largest T below the turning point and the one with the
// smallest T at or above it (first index of its run of equal T).  Each thread owns the
// requests u of some ranks, finds those two members by binary search in the member list
// (sorted by T) and keeps its best tuple; a CTA-wide lexicographic min picks the step.
// ---------------------------------------------------------------------------------------
struct Cand {
    long long v;
    int i, k, u;       // request indices / client
    int ri, ru;        // ranks of i and u (ru = -1 for a move)
};

__device__ __forceinline__ bool cand_less(const Cand& a, const Cand& b) {
    if (a.v != b.v) return a.v < b.v;
    if (a.i != b.i) return a.i < b.i;
    if (a.k != b.k) return a.k < b.k;
    return a.u < b.u;
}

__device__ __forceinline__ Cand cand_shfl_xor(const Cand& c, int d) {
    Cand r;
    r.v = __shfl_xor_sync(FULL, c.v, d);
    r.i = __shfl_xor_sync(FULL, c.i, d);
    r.k = __shfl_xor_sync(FULL, c.k, d);
    r.u = __shfl_xor_sync(FULL, c.u, d);
    r.ri = __shfl_xor_sync(FULL, c.ri, d);
    r.ru = __shfl_xor_sync(FULL, c.ru, d);
    return r;
}

constexpr long long NO_V = 0x7FFFFFFFFFFFFFFFll;
constexpr int NO_I = 0x7FFFFFFF;

template <typename IdxT>
__global__ void __launch_bounds__(SORT_THREADS, 1)
k_local_search(const uint32_t* __restrict__ T_sorted, const uint32_t* __restrict__ order,
               const InstInfo* __restrict__ info, int n_req, int n_pad, int n_clients,
               int n_copies, int rounds, bool load_from_assign,
               int32_t* __restrict__ assign, long long* __restrict__ load_io,
               long long* __restrict__ makespan_out, int32_t* __restrict__ rounds_applied,
               hos_ls_move* __restrict__ ls_log, int32_t* __restrict__ status_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ long long s_load[MAX_CLIENTS];
    __shared__ Cand s_cand[32];
    __shared__ int s_wcnt[32];
    __shared__ int s_jmax, s_nm, s_kmin;
    __shared__ long long s_vb[32];
    __shared__ long long s_lmax;

    const int inst = blockIdx.x / n_copies;
    const size_t unit = blockIdx.x;                        // inst * n_copies + copy
    const int lane = lane_id(), warp = warp_id();
    const InstInfo inf = info[inst];
    int32_t* asg = assign + unit * n_req;
    long long* ld = load_io + unit * n_clients;
    hos_ls_move* log = ls_log ? ls_log + unit * rounds : nullptr;

    if (inf.status) {
        if (load_from_assign) {
            for (int j = threadIdx.x; j < n_clients; j += SORT_THREADS) ld[j] = 0;
            if (threadIdx.x == 0) makespan_out[unit] = 0;
        }
        if (threadIdx.x == 0) rounds_applied[unit] = 0;
        if (log)
            for (int r = threadIdx.x; r < rounds; r += SORT_THREADS) log[r] = hos_ls_move{-1, -1, -1, 0};
        return;
    }

    unsigned char* base = smem_raw;
    uint32_t* Ts = reinterpret_cast<uint32_t*>(base);   base += align16((size_t)n_req * 4);
    IdxT* ord = reinterpret_cast<IdxT*>(base);          base += align16((size_t)n_req * sizeof(IdxT));
    IdxT* mem = reinterpret_cast<IdxT*>(base);          base += align16((size_t)n_req * sizeof(IdxT));
    uint8_t* bins = reinterpret_cast<uint8_t*>(base);

    const uint32_t* gT = T_sorted + (size_t)inst * n_pad;
    const uint32_t* gO = order + (size_t)inst * n_pad;
    for (int j = threadIdx.x; j < n_clients; j += SORT_THREADS) s_load[j] = load_from_assign ? 0 : ld[j];
    __syncthreads();
    bool bad_assign = false;
    for (int r = threadIdx.x; r < n_req; r += SORT_THREADS) {
        const uint32_t t = gT[r], id = gO[r];
        const int c = asg[id];
        Ts[r] = t;
        ord[r] = (IdxT)id;
        if (c < 0 || c >= n_clients) { bad_assign = true; bins[r] = 0; }
        else {
            bins[r] = (uint8_t)c;
            if (load_from_assign) atomicAdd(reinterpret_cast<unsigned long long*>(&s_load[c]), (unsigned long long)t);
        }
    }
    if (__syncthreads_or(bad_assign)) {
        if (threadIdx.x == 0) {
            atomicOr(&status_out[inst], HOS_ST_INVALID);
            rounds_applied[unit] = 0;
            makespan_out[unit] = 0;
        }
        for (int j = threadIdx.x; j < n_clients; j += SORT_THREADS) ld[j] = 0;
        if (log)
            for (int r = threadIdx.x; r < rounds; r += SORT_THREADS) log[r] = hos_ls_move{-1, -1, -1, 0};
        return;
    }

    const int chunk = (((n_req + SORT_WARPS - 1) / SORT_WARPS) + 31) & ~31;
    const int lo = warp * chunk, hi = min(n_req, lo + chunk);
    int applied = 0;
    int done_at = rounds;

    for (int round = 0; round < rounds; ++round) {
        // (a) critical client: largest load, ties to the lowest client
        if (warp == 0) {
            long long bl = -1;
            int bj = NO_I;
            for (int j = lane; j < n_clients; j += 32)
                if (s_load[j] > bl) { bl = s_load[j]; bj = j; }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                const long long ol = __shfl_xor_sync(FULL, bl, d);
                const int oj = __shfl_xor_sync(FULL, bj, d);
                if (ol > bl || (ol == bl && oj < bj)) { bl = ol; bj = oj; }
            }
            if (lane == 0) { s_jmax = bj; s_lmax = bl; }
            // least loaded other client (any of them on ties: it only seeds the pruning bound)
            const int jm = __shfl_sync(FULL, bj, 0);
            long long ml = NO_V;
            int mj = -1;
            for (int j = lane; j < n_clients; j += 32)
                if (j != jm && s_load[j] < ml) { ml = s_load[j]; mj = j; }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                const long long ol = __shfl_xor_sync(FULL, ml, d);
                const int oj = __shfl_xor_sync(FULL, mj, d);
                if (ol < ml) { ml = ol; mj = oj; }
            }
            if (lane == 0) s_kmin = mj;
        }
        __syncthreads();
        const int jmax = s_jmax;
        const long long Lmax = s_lmax;

        // (b) members of jmax, in rank order (T descending, index ascending inside equal T)
        int cnt = 0;
        for (int row = lo; row < hi; row += 32) {
            const int r = row + lane;
            cnt += __popc(__ballot_sync(FULL, r < hi && bins[r] == jmax));
        }
        if (lane == 0) s_wcnt[warp] = cnt;
        __syncthreads();
        if (warp == 0) {
            const int c = s_wcnt[lane];
            int inc = c;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(FULL, inc, d);
                if (lane >= d) inc += y;
            }
            s_wcnt[lane] = inc - c;
            if (lane == 31) s_nm = inc;
        }
        __syncthreads();
        int off = s_wcnt[warp];
        for (int row = lo; row < hi; row += 32) {
            const int r = row + lane;
            const bool is = r < hi && bins[r] == jmax;
            const unsigned b = __ballot_sync(FULL, is);
            if (is) mem[off + __popc(b & ((1u << lane) - 1u))] = (IdxT)r;
            off += __popc(b);
        }
        __syncthreads();
        const int nm = s_nm;

        // (c) candidates: work item w < n_req is "swap with the request of rank w";
        //     w >= n_req is "move to client w - n_req".
        //     Any step onto client k ends with v >= ceil((Lmax + load_k) / 2).  A first sweep over
        //     the least loaded client alone gives an achievable v (`vbound`); the full sweep then
        //     skips every client whose floor is above it.  Ties in v survive the filter.
        auto evaluate = [&](int w, Cand& best, long long vbound) {
            int k, u, ru;
            long long Tu;
            if (w < n_req) { k = bins[w]; u = -2; ru = w; Tu = Ts[w]; }
            else { k = w - n_req; u = -1; ru = -1; Tu = 0; }
            if (k == jmax) return;
            const long long lk = s_load[k];
            const long long slack = Lmax - lk;
            if (slack <= 0 || ((Lmax + lk + 1) >> 1) > vbound) return;
            if (u == -2) u = (int)ord[w];
            const long long thr = Tu + ((slack + 1) >> 1);      // T_i >= thr  <=>  2 d >= slack
            // b = number of members with T >= thr (members are sorted by T descending)
            int a = 0, z = nm;
            while (a < z) {
                const int mid = (a + z) >> 1;
                if ((long long)Ts[mem[mid]] >= thr) a = mid + 1; else z = mid;
            }
            const int b = a;
            if (b > 0) {                                        // rising side: smallest T >= thr
                const long long Ti = Ts[mem[b - 1]];
                const long long d = Ti - Tu;
                if (d < slack) {
                    // first member of the run of equal T (smallest request index)
                    int a2 = 0, z2 = b - 1;
                    while (a2 < z2) {
                        const int mid = (a2 + z2) >> 1;
                        if ((long long)Ts[mem[mid]] > Ti) a2 = mid + 1; else z2 = mid;
                    }
                    Cand c;
                    c.v = lk + d; c.ri = (int)mem[a2]; c.i = (int)ord[c.ri]; c.k = k; c.u = u; c.ru = ru;
                    if (cand_less(c, best)) best = c;
                }
            }
            if (b < nm) {                                       // falling side: largest T < thr
                const long long Ti = Ts[mem[b]];
                const long long d = Ti - Tu;
                if (d > 0) {
                    Cand c;
                    c.v = Lmax - d; c.ri = (int)mem[b]; c.i = (int)ord[c.ri]; c.k = k; c.u = u; c.ru = ru;
                    if (cand_less(c, best)) best = c;
                }
            }
        };
        Cand best;
        best.v = NO_V; best.i = NO_I; best.k = NO_I; best.u = NO_I; best.ri = -1; best.ru = -1;
        const int kmin = s_kmin;
        if (kmin >= 0) {
            for (int w = threadIdx.x; w < n_req + n_clients; w += SORT_THREADS) {
                const int k = (w < n_req) ? (int)bins[w] : w - n_req;
                if (k == kmin) evaluate(w, best, NO_V);
            }
        }
        long long vb = best.v;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) vb = min(vb, __shfl_xor_sync(FULL, vb, d));
        if (lane == 0) s_vb[warp] = vb;
        __syncthreads();
        vb = s_vb[lane];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) vb = min(vb, __shfl_xor_sync(FULL, vb, d));
        const long long vbound = vb;
        best.v = NO_V; best.i = NO_I; best.k = NO_I; best.u = NO_I; best.ri = -1; best.ru = -1;
        for (int w = threadIdx.x; w < n_req + n_clients; w += SORT_THREADS) evaluate(w, best, vbound);
        // (d) CTA-wide lexicographic minimum
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const Cand oc = cand_shfl_xor(best, d);
            if (cand_less(oc, best)) best = oc;
        }
        if (lane == 0) s_cand[warp] = best;
        __syncthreads();
        if (warp == 0) {
            best = s_cand[lane];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                const Cand oc = cand_shfl_xor(best, d);
                if (cand_less(oc, best)) best = oc;
            }
            if (lane == 0) s_cand[0] = best;
        }
        __syncthreads();
        best = s_cand[0];
        const bool ok = best.v < Lmax;                          // NO_V when there was no candidate
        // (e) apply
        if (threadIdx.x == 0) {
            if (ok) {
                const long long d = (long long)Ts[best.ri] - (best.ru >= 0 ? (long long)Ts[best.ru] : 0ll);
                bins[best.ri] = (uint8_t)best.k;
                asg[best.i] = best.k;
                if (best.ru >= 0) { bins[best.ru] = (uint8_t)jmax; asg[best.u] = jmax; }
                s_load[jmax] -= d;
                s_load[best.k] += d;
                if (log) log[round] = hos_ls_move{best.i, best.u, best.k, best.v};
            } else if (log) {
                log[round] = hos_ls_move{-1, -1, -1, Lmax};
            }
        }
        __syncthreads();
        if (!ok) { done_at = round; break; }
        ++applied;
    }
    // a round without an improving step leaves the state as it is: all later rounds are the same
    if (log && done_at < rounds) {
        const hos_ls_move noop = hos_ls_move{-1, -1, -1, s_lmax};
        for (int r = done_at + 1 + threadIdx.x; r < rounds; r += SORT_THREADS) log[r] = noop;
    }
    long long mx = 0;
    for (int j = threadIdx.x; j < n_clients; j += SORT_THREADS) { ld[j] = s_load[j]; }
    if (warp == 0) {
        for (int j = lane; j < n_clients; j += 32) mx = s_load[j] > mx ? s_load[j] : mx;
        mx = warp_max_i64(mx);
        if (lane == 0) { makespan_out[unit] = mx; rounds_applied[unit] = applied; }
    }
}

// ---------------------------------------------------------------------------------------
// Lower bounds.  One CTA per instance; reads p, o once, and T_(M), T_(M+1) from the sorted
// table left by k_estimate_sort.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long floor_sum_below(unsigned long long n, unsigned long long q) {
    // sum over x in [0, n) of floor(x / q)
    const unsigned long long m = n / q, r = n % q;
    return q * (m * (m - 1ull + (m == 0ull)) / 2ull) + m * r;   // m = 0 -> 0
}

__global__ void __launch_bounds__(256)
k_lower_bound(const uint32_t* __restrict__ p, const uint32_t* __restrict__ o, int n_req, int n_pad,
              int n_clients, int cap, hos_cost_model cm, const uint32_t* __restrict__ T_sorted,
              const InstInfo* __restrict__ info, hos_lb* __restrict__ out) {
    __shared__ unsigned long long red[32];
    const int inst = blockIdx.x;
    const InstInfo inf = info[inst];
    if (inf.status) {
        if (threadIdx.x == 0) out[inst] = hos_lb{0, 0, 0, 0, 0, 0, 0, 0};
        return;
    }
    const uint32_t* pi = p + (size_t)inst * n_req;
    const uint32_t* oi = o + (size_t)inst * n_req;
    const unsigned long long ap = cm.prefill_fixed_us, bp = cm.prefill_per_token_us;
    const unsigned long long ad = cm.decode_fixed_us, bd = cm.decode_per_seq_us, q = cm.decode_kv_div;
    unsigned long long P = 0, O = 0, K = 0, chain = 0;
    for (int i = threadIdx.x; i < n_req; i += blockDim.x) {
        const unsigned long long pp = pi[i], oo = oi[i];
        P += pp;
        O += oo;
        K += oo * pp + oo * (oo - 1ull) / 2ull;
        const unsigned long long alone = ap + bp * pp + oo * (ad + bd) +
                                         floor_sum_below(pp + oo, q) - floor_sum_below(pp, q);
        chain = alone > chain ? alone : chain;
    }
    P = block_sum_u64(P, red);
    O = block_sum_u64(O, red);
    K = block_sum_u64(K, red);
    chain = block_max_u64(chain, red);
    if (threadIdx.x == 0) {
        const unsigned long long M = (unsigned long long)n_clients, C = (unsigned long long)cap;
        hos_lb r;
        const unsigned long long sumT = inf.sum_T, maxT = inf.max_T;
        unsigned long long pairT = 0;
        if (n_req > n_clients) {
            const uint32_t* Ts = T_sorted + (size_t)inst * n_pad;
            pairT = (unsigned long long)Ts[n_clients - 1] + (unsigned long long)Ts[n_clients];
        }
        unsigned long long lb = (sumT + M - 1ull) / M;
        lb = maxT > lb ? maxT : lb;
        lb = pairT > lb ? pairT : lb;
        const unsigned long long n_pre = ((unsigned long long)n_req + C - 1ull) / C;
        const unsigned long long n_dec = (O + C - 1ull) / C;
        const unsigned long long tp_star = ap * n_pre + bp * P;
        const unsigned long long td_q = q * ((ad - 1ull) * n_dec + bd * O) + K;
        const unsigned long long work = (q * tp_star + td_q + q * M - 1ull) / (q * M);
        r.lb_pack = (long long)lb; r.sum_T = (long long)sumT; r.max_T = (long long)maxT; r.pair_T = (long long)pairT;
        r.tp_star_us = (long long)((tp_star + M - 1ull) / M);
        r.td_star_us = (long long)((td_q + q * M - 1ull) / (q * M));
        r.chain_us = (long long)chain;
        r.lb_sim_us = (long long)(work > chain ? work : chain);
        out[inst] = r;
    }
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------
static size_t ls_smem_bytes(int n_req, size_t isz) {
    return align16((size_t)n_req * 4) + 2 * align16((size_t)n_req * isz) + align16((size_t)n_req);
}

size_t estimate_sort_smem(int n_req) {
    return n_req <= 65536 ? sort_smem_bytes<uint16_t>(n_req) : sort_smem_bytes<uint32_t>(n_req);
}
size_t local_search_smem(int n_req) { return ls_smem_bytes(n_req, n_req <= 65536 ? 2 : 4); }

cudaError_t launch_estimate_sort(const hos_batch& b, const hos_cost_model& cm, uint32_t* T_sorted,
                                 uint32_t* order, InstInfo* info, int32_t* status_out, int n_pad,
                                 cudaStream_t st) {
    const size_t smem = estimate_sort_smem(b.n_req);
    auto kern = b.n_req <= 65536 ? k_estimate_sort<uint16_t> : k_estimate_sort<uint32_t>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    launch_hook("k_estimate_sort", 0, st);
    kern<<<b.n_inst, SORT_THREADS, smem, st>>>(b.p, b.o, b.n_req, (long long)b.kv_budget,
                                               cm.est_per_prompt_token, cm.est_per_output_token,
                                               T_sorted, order, info, status_out, n_pad);
    launch_hook("k_estimate_sort", 1, st);
    return cudaGetLastError();
}

cudaError_t launch_lpt(const hos_batch& b, const uint32_t* T_sorted, const uint32_t* order,
                       const InstInfo* info, int n_pad, int32_t* assign, long long* load,
                       long long* makespan, cudaStream_t st) {
    const int M = b.n_clients;
#define HOS_LPT(KPL)                                                                               \
    k_lpt<KPL><<<b.n_inst, 32, 0, st>>>(T_sorted, order, info, b.n_req, n_pad, M, assign, load,    \
                                         makespan)
    launch_hook("k_lpt", 0, st);
    if (M <= 32) HOS_LPT(1);
    else if (M <= 64) HOS_LPT(2);
    else if (M <= 128) HOS_LPT(4);
    else HOS_LPT(8);
#undef HOS_LPT
    launch_hook("k_lpt", 1, st);
    return cudaGetLastError();
}

cudaError_t launch_local_search(const hos_batch& b, const uint32_t* T_sorted, const uint32_t* order,
                                const InstInfo* info, int n_pad, int n_copies, int rounds,
                                bool load_from_assign, int32_t* assign, long long* load,
                                long long* makespan, int32_t* rounds_applied, hos_ls_move* ls_log,
                                int32_t* status, cudaStream_t st) {
    const size_t smem = local_search_smem(b.n_req);
    auto kern = b.n_req <= 65536 ? k_local_search<uint16_t> : k_local_search<uint32_t>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    launch_hook("k_local_search", 0, st);
    kern<<<b.n_inst * n_copies, SORT_THREADS, smem, st>>>(T_sorted, order, info, b.n_req, n_pad,
                                                          b.n_clients, n_copies, rounds,
                                                          load_from_assign, assign, load, makespan,
                                                          rounds_applied, ls_log, status);
    launch_hook("k_local_search", 1, st);
    return cudaGetLastError();
}

cudaError_t launch_lower_bound(const hos_batch& b, const hos_cost_model& cm, const uint32_t* T_sorted,
                               const InstInfo* info, int n_pad, hos_lb* out, cudaStream_t st) {
    launch_hook("k_lower_bound", 0, st);
    k_lower_bound<<<b.n_inst, 256, 0, st>>>(b.p, b.o, b.n_req, n_pad, b.n_clients, b.batch_cap, cm,
                                            T_sorted, info, out);
    launch_hook("k_lower_bound", 1, st);
    return cudaGetLastError();
}

}  // namespace hos
