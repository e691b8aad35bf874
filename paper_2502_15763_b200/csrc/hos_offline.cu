// Offline request scheduling kernels (Eq. 26-30 of arXiv 2502.15763):
//   k_estimate_sort  T_i and the per-instance order (T descending, index ascending)
//   k_lpt            longest-first list scheduling, one warp per instance
//   k_ls_lists       the clients' member lists for the local search
//   k_local_search   rounds of best move / pairwise swap off the critical client
//   (the lower bounds of Eq. 31-32 ride in k_estimate_sort's load pass)
#include "hos_common.cuh"
#include "hos_kernels.h"
#include "hos_sort.cuh"

#include <type_traits>

namespace hos {

// ---------------------------------------------------------------------------------------
// Lower bounds (Eq. 31-32 and the packing relaxations): the sums over an instance's requests
// are taken in the load pass of the estimate + sort kernel, which reads p and o anyway, and
// one thread finishes them once the sorted table gives T_(M) and T_(M+1).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long floor_sum_below(uint32_t n, uint32_t q, int q_shift) {
    // sum over x in [0, n) of floor(x / q); n and q fit 32 bits, so one 32-bit division does
    // (a shift when q = 2^q_shift, q_shift >= 0)
    const uint32_t m = q_shift >= 0 ? n >> q_shift : n / q, r = n - m * q;
    return (unsigned long long)q * (((unsigned long long)m * (m - 1u + (m == 0u))) >> 1) +
           (unsigned long long)m * r;                           // m = 0 -> 0
}

struct LbSums {
    unsigned long long P, O, K, chain;      // sum p, sum o, sum of KV tokens attended, longest request alone
};

// a valid instance has p + o <= kv_budget < 2^31
__device__ __forceinline__ void lb_take(LbSums& a, const hos_cost_model& cm, int q_shift, uint32_t pp, uint32_t oo) {
    a.P += pp;
    a.O += oo;
    a.K += ((unsigned long long)oo * (2ull * pp + oo - 1ull)) >> 1;      // o p + o (o - 1) / 2
    // the request served alone: a maximum, so the exact value (two floor sums) is only taken when
    // an upper bound of it, sum of floor((p + s) / q) <= o (p + o) / q, beats the running maximum
    const unsigned long long fixed = (unsigned long long)prefill_us(cm, pp) +
                                     oo * ((unsigned long long)cm.decode_fixed_us + cm.decode_per_seq_us);
    const unsigned long long kv_hi = (unsigned long long)oo * (pp + oo);
    if (fixed + (q_shift >= 0 ? kv_hi >> q_shift : kv_hi / cm.decode_kv_div) > a.chain) {
        const unsigned long long alone = fixed + floor_sum_below(pp + oo, cm.decode_kv_div, q_shift) -
                                         floor_sum_below(pp, cm.decode_kv_div, q_shift);
        a.chain = alone > a.chain ? alone : a.chain;
    }
}

// One thread: the bounds of an instance from its sums.  pairT = T_(M) + T_(M+1), 0 when n_req <= M.
__device__ inline void lb_finish(const LbSums& a, const hos_cost_model& cm, int n_req, int n_clients, int cap,
                                 unsigned long long sumT, unsigned long long maxT, unsigned long long pairT,
                                 hos_lb* out, int32_t* status_word) {
    const unsigned long long ad = cm.decode_fixed_us, bd = cm.decode_per_seq_us, q = cm.decode_kv_div;
    const unsigned long long M = (unsigned long long)n_clients, C = (unsigned long long)cap;
    hos_lb r;
    unsigned long long lb = (sumT + M - 1ull) / M;
    lb = maxT > lb ? maxT : lb;
    lb = pairT > lb ? pairT : lb;
    const unsigned long long n_pre = ((unsigned long long)n_req + C - 1ull) / C;
    const unsigned long long n_dec = (a.O + C - 1ull) / C;
    // Scaled sums in 128 bits: coefficients and sums that are each inside their limits can still
    // carry these products past 64 bits, and a bound that does not fit is flagged, not wrapped.
    typedef unsigned __int128 u128;
    const u128 lim = (u128)0x7FFFFFFFFFFFFFFFull;
    u128 tp_wide, tp_paper_wide = 0;
    if (cm.n_levels == 0) {
        tp_wide = (u128)cm.prefill_fixed_us * n_pre + (u128)cm.prefill_per_token_us * a.P;
    } else {
        // at least n_pre stages of at least the smallest level's time; a stage of level l carries
        // at most N^cap_l tokens, so P tokens cost at least min_l floor(P / N^cap_l) T^p_l
        const u128 by_count = (u128)cm.level_time_us[0] * n_pre;
        u128 by_tokens = ~(u128)0;
        for (uint32_t l = 0; l < cm.n_levels; ++l) {
            const u128 v = (u128)(a.P / cm.level_cap_tokens[l]) * cm.level_time_us[l];
            by_tokens = v < by_tokens ? v : by_tokens;
        }
        tp_wide = by_count > by_tokens ? by_count : by_tokens;
        tp_paper_wide = (u128)(a.P / cm.level_cap_tokens[cm.n_levels - 1]) * cm.level_time_us[cm.n_levels - 1];
    }
    const u128 td_q = (u128)q * ((u128)(ad - 1ull) * n_dec + (u128)bd * a.O) + a.K;
    const u128 tot_q = (u128)q * tp_wide + td_q + (u128)(q * M - 1ull);
    if (tp_wide > lim || tp_paper_wide > lim || td_q > lim || tot_q > lim) {
        *out = hos_lb{0, 0, 0, 0, 0, 0, 0, 0, 0};
        if (status_word) *status_word |= HOS_ST_RANGE;
        return;
    }
    const unsigned long long tp_star = (unsigned long long)tp_wide;
    const unsigned long long td_q64 = (unsigned long long)td_q;
    const unsigned long long work = (unsigned long long)tot_q / (q * M);
    r.tp_paper_us = (long long)(unsigned long long)tp_paper_wide;
    r.lb_pack = (long long)lb; r.sum_T = (long long)sumT; r.max_T = (long long)maxT; r.pair_T = (long long)pairT;
    r.tp_star_us = (long long)((tp_star + M - 1ull) / M);
    r.td_star_us = (long long)((td_q64 + q * M - 1ull) / (q * M));
    r.chain_us = (long long)a.chain;
    r.lb_sim_us = (long long)(work > a.chain ? work : a.chain);
    *out = r;
}

// ---------------------------------------------------------------------------------------
// Estimate + segmented sort (+ the lower bounds' sums).  One CTA per instance; the T table lives
// in shared memory.  FAST: the bucket sort, one CTA per instance; when it declines an instance
// (keys too wide or too bunched) it leaves SORT_PENDING in the instance's workspace status and
// the second launch of this kernel, !FAST, a few persistent CTAs with the radix sort's larger
// shared memory, takes exactly those instances.
// ---------------------------------------------------------------------------------------
constexpr int SORT_PENDING = 0x100;        // internal bit of InstInfo::status

template <bool FAST>
__global__ void __launch_bounds__(SORT_THREADS, 1)
k_estimate_sort(const uint32_t* __restrict__ p, const uint32_t* __restrict__ o,
                const uint32_t* __restrict__ o_est, int n_inst, int n_req,
                long long kv_budget, uint32_t p_max, hos_cost_model cm, int q_shift, int n_clients, int cap,
                uint32_t* __restrict__ T_sorted, uint32_t* __restrict__ order,
                InstInfo* __restrict__ info, int32_t* __restrict__ status_out, hos_lb* __restrict__ lb_out,
                int n_pad) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ uint32_t s_pair[2];                        // T_(M), T_(M+1)
    const uint32_t e_p = cm.est_per_prompt_token, e_o = cm.est_per_output_token;
    for (int inst = blockIdx.x; inst < n_inst; inst += gridDim.x) {
        if (!FAST) {
            __syncthreads();                              // the instance before is finished with shared memory
            if (!(info[inst].status & SORT_PENDING)) continue;      // uniform: one word read by every thread
        }
        const uint32_t* pi = p + (size_t)inst * n_req;
        const uint32_t* oi = o + (size_t)inst * n_req;
        const uint32_t* ei = o_est ? o_est + (size_t)inst * n_req : oi;   // the lengths the scheduler knows
        uint32_t* key = reinterpret_cast<uint32_t*>(smem_raw);            // the radix path keeps T here

        // first pass: checks, sums, the largest T (and the lower bounds' sums).  kv_budget here is
        // the most KV one request may need: the fixed reservation, if there is one
        unsigned long long sum = 0, mx = 0, bad = 0;
        uint32_t mx32 = 0;                                // a T beyond 32 bits marks the instance bad: mx is not used then
        LbSums a = {0ull, 0ull, 0ull, 0ull};
        for_each_request(pi, oi, ei, nullptr, n_req, [&](int i, uint32_t pp, uint32_t oo, uint32_t oe, int) {
            const unsigned long long t = (unsigned long long)e_p * pp + (unsigned long long)e_o * oe;
            if (pp == 0 || oo == 0 || oe == 0 || pp > p_max || (long long)pp + (long long)oo > kv_budget ||
                t > 0xFFFFFFFFull)
                bad = 1;
            else if (lb_out) lb_take(a, cm, q_shift, pp, oo);
            if (!FAST) key[i] = (uint32_t)t;
            sum += t;
            mx32 = max(mx32, (uint32_t)t);
        });
        mx = mx32;
        // all of them in one go: per warp, then warp k finishes value k (four sums, two maxima).  The
        // scratch is a part of the sort's shared memory that nothing uses before the sort starts.
        {
            typedef unsigned long long red_row[SORT_WARPS];
            red_row* red = reinterpret_cast<red_row*>(
                FAST ? smem_raw : reinterpret_cast<unsigned char*>(sort_smem_carve<uint16_t>(smem_raw, n_req).cnt));
            unsigned long long v[6] = {sum, a.P, a.O, a.K, mx, a.chain};
#pragma unroll
            for (int k = 0; k < 6; ++k) {
                v[k] = k < 4 ? warp_sum_u64(v[k]) : warp_max_u64(v[k]);
                if (lane_id() == 0) red[k][warp_id()] = v[k];
            }
            bad = __syncthreads_or(bad != 0);
            if (warp_id() < 6) {
                const unsigned long long t = red[warp_id()][lane_id()];
                const unsigned long long r = warp_id() < 4 ? warp_sum_u64(t) : warp_max_u64(t);
                if (lane_id() == 0) red[warp_id()][0] = r;
            }
            __syncthreads();
            sum = red[0][0]; a.P = red[1][0]; a.O = red[2][0]; a.K = red[3][0]; mx = red[4][0]; a.chain = red[5][0];
            __syncthreads();                              // the scratch is the sort's again
        }
        if (bad) {                                        // uniform: every thread sees the same value
            if (threadIdx.x == 0) {
                info[inst].sum_T = sum; info[inst].max_T = (uint32_t)mx; info[inst].status = HOS_ST_INVALID;
                if (status_out) status_out[inst] = HOS_ST_INVALID;
                if (lb_out) lb_out[inst] = hos_lb{0, 0, 0, 0, 0, 0, 0, 0, 0};
            }
            continue;
        }
        const int nbits = bit_width_u32((uint32_t)mx);
        const uint32_t flip = nbits >= 32 ? 0xFFFFFFFFu : ((1u << nbits) - 1u);   // descending T
        uint32_t* Ts = T_sorted ? T_sorted + (size_t)inst * n_pad : nullptr;
        uint32_t* od = T_sorted ? order + (size_t)inst * n_pad : nullptr;
        if (threadIdx.x < 2) s_pair[threadIdx.x] = 0;
        if (FAST) {
            // two more passes over the tables (now in L2): count, then place; T is taken again
            BucketSort B;
            bool ok = bucket_sort_plan(B, smem_raw, n_req, nbits, 0);
            if (ok) {
                bucket_sort_clear(B);
                for_each_request(pi, oi, ei, nullptr, n_req, [&](int, uint32_t pp, uint32_t, uint32_t oe, int) {
                    bucket_sort_count(B, (e_p * pp + e_o * oe) ^ flip);
                });
                ok = bucket_sort_scan(B, n_req);
            }
            if (!ok) {
                if (threadIdx.x == 0) info[inst].status = SORT_PENDING;
                continue;
            }
            if (!T_sorted) {
                // Bounds only: no order is wanted, just T_(M) and T_(M+1).  The buckets that hold
                // those two ranks are known from the scan; their items alone are collected and
                // ranked among themselves.
                if (n_req > n_clients) {
                    __shared__ uint32_t s_ncand;
                    if (threadIdx.x == 0) s_ncand = 0;
                    __syncthreads();
                    const uint32_t M = (uint32_t)n_clients, nb = 1u << B.bbits;
                    for_each_request(pi, oi, ei, nullptr, n_req, [&](int i, uint32_t pp, uint32_t, uint32_t oe, int) {
                        const uint32_t fk = ((e_p * pp + e_o * oe) ^ flip) & B.kmask, b = fk >> B.low_bits;
                        const uint32_t start = bucket_sort_start(B, b), end = b + 1 < nb ? bucket_sort_start(B, b + 1) : (uint32_t)n_req;
                        if (start <= M && M - 1 < end) {             // the bucket holds rank M - 1 or M
                            const uint32_t at = atomicAdd(&s_ncand, 1u);
                            if (HOS_IN(at, n_req, 203)) { B.ent[at] = ((fk & B.lmask) << B.id_bits) | (uint32_t)i; B.bkt[at] = (uint16_t)b; }
                        }
                    });
                    __syncthreads();
                    const uint32_t nc = s_ncand;
                    for (uint32_t c = threadIdx.x; c < nc; c += SORT_THREADS) {
                        const uint32_t mine = B.ent[c], b = B.bkt[c];
                        uint32_t r = bucket_sort_start(B, b);
                        for (uint32_t j = 0; j < nc; ++j) r += (B.bkt[j] == b && B.ent[j] < mine) ? 1u : 0u;
                        if (r + 1 == M || r == M) s_pair[r + 1 - M] = ((b << B.low_bits) | (mine >> B.id_bits)) ^ flip;
                    }
                }
            } else {
            for_each_request(pi, oi, ei, nullptr, n_req, [&](int i, uint32_t pp, uint32_t, uint32_t oe, int) {
                bucket_sort_place(B, (e_p * pp + e_o * oe) ^ flip, (uint32_t)i, 0u);
            });
            __syncthreads();
            for (int s = threadIdx.x; s < n_req; s += SORT_THREADS) {
                uint32_t fk, id, extra;
                const uint32_t r = bucket_sort_rank(B, s, fk, id, extra);
                const uint32_t T = fk ^ flip;             // T < 2^nbits: the flip is its own inverse there
                if (!HOS_IN(r, n_req, 201) || !HOS_IN(id, n_req, 202)) continue;
                od[r] = id;
                Ts[r] = T;
                if (r + 1 == (uint32_t)n_clients || r == (uint32_t)n_clients) s_pair[r + 1 - n_clients] = T;
            }
            }
        } else {
            SortSmem<uint16_t> s = sort_smem_carve<uint16_t>(smem_raw, n_req);
            const uint16_t* sorted = block_radix_sort_ids<uint16_t>(s, n_req, nbits, flip);
            for (int r = threadIdx.x; r < n_req; r += SORT_THREADS) {
                const uint32_t id = sorted[r];
                if (T_sorted) { od[r] = id; Ts[r] = key[id]; }
                if (r + 1 == n_clients || r == n_clients) s_pair[r + 1 - n_clients] = key[id];
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int32_t st = 0;
            const unsigned long long pairT = n_req > n_clients ? (unsigned long long)s_pair[0] + s_pair[1] : 0ull;
            if (lb_out) lb_finish(a, cm, n_req, n_clients, cap, sum, mx, pairT, &lb_out[inst], &st);
            info[inst].sum_T = sum; info[inst].max_T = (uint32_t)mx; info[inst].status = 0;
            if (status_out) status_out[inst] = st;
        }
    }
}

// ---------------------------------------------------------------------------------------
// LPT list scheduling.  One warp per instance: client j = slot * 32 + lane.  The chain of
// n_req dependent argmin steps runs on packed keys (load - base) << JB | j, so that one
// 32-bit warp min gives both the least load and, on ties, the lowest client.  The loads stay
// within max_T of their minimum (each item lands on the current minimum), which bounds the
// packed field between re-basings; instances that do not fit use 64-bit loads.
// ---------------------------------------------------------------------------------------
constexpr int LPT_AHEAD = 4;                // chunks of 32 items that k_lpt fetches ahead of their use
template <int KPL>
__global__ void __launch_bounds__(32)
k_lpt(const uint32_t* __restrict__ T_sorted, const uint32_t* __restrict__ order,
      const InstInfo* __restrict__ info, int n_req, int n_pad, int n_clients,
      int32_t* __restrict__ assign, long long* __restrict__ load_out,
      long long* __restrict__ makespan_out, uint8_t* __restrict__ rank_client) {
    constexpr int JB = (KPL == 1) ? 5 : (KPL == 2) ? 6 : (KPL == 4) ? 7 : 8;
    __shared__ uint32_t s_perm[32];
    __shared__ uint32_t s_tv[32 * LPT_AHEAD], s_rq[32 * LPT_AHEAD];
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
    // nullable: the client of the r-th request in sorted order, for the local search's list build
    uint8_t* rc = rank_client ? rank_client + (size_t)inst * n_pad : nullptr;

    long long load[KPL];
#pragma unroll
    for (int k = 0; k < KPL; ++k) load[k] = 0;

    // packed path is safe when (max_T * (2 + ceil(32 / M)) + 1) << JB fits 32 bits
    const unsigned long long span =
        (unsigned long long)inf.max_T * (2ull + (unsigned long long)((32 + n_clients - 1) / n_clients)) + 1ull;
    const bool packed = (span << JB) < 0xFFFFFFFFull;

    if (packed) {
        // Wave form of the chain.  With the keys sorted, s_0 < s_1 < ..., the next items t_0 >= t_1 >= ...
        // go to s_0, s_1, ... one each for as long as s_a is still below every updated key
        // s_b + t_b, b < a: exactly what the one-by-one rule does, found for up to 32 items at once by
        // one sort of the keys (bitonic, across the warp) and one prefix minimum.  Keys carry their
        // client in the low bits, so they may sit in any lane.
        uint32_t key[KPL];
#pragma unroll
        for (int k = 0; k < KPL; ++k) {
            const int j = k * 32 + lane;
            key[k] = (j < n_clients) ? (uint32_t)j : 0xFFFFFFFFu;
        }
        unsigned long long rebased = 0;                 // sum of the bases subtracted so far
        bool half_sorted = false;                       // key[0] is all new, key[1] still ascending
        // The items arrive LPT_AHEAD chunks ahead of their use: four chunks wait in shared memory
        // while the next four are on their way in registers (a chunk is a few hundred cycles of
        // dependent work and few warps share an SM, so one chunk ahead would leave most of a
        // memory round trip in the open).
        uint32_t tv_next[LPT_AHEAD], rq_next[LPT_AHEAD];
#pragma unroll
        for (int j = 0; j < LPT_AHEAD; ++j) {
            const int rn = 32 * j + lane;
            tv_next[j] = (rn < n_req) ? Ts[rn] : 0u;
            rq_next[j] = (rn < n_req) ? od[rn] : 0u;
        }
        for (int R0 = 0; R0 < n_req; R0 += 32 * LPT_AHEAD) {
        __syncwarp();                                   // the chunks before are used up
#pragma unroll
        for (int j = 0; j < LPT_AHEAD; ++j) {
            s_tv[32 * j + lane] = tv_next[j];
            s_rq[32 * j + lane] = rq_next[j];
        }
        __syncwarp();
#pragma unroll
        for (int j = 0; j < LPT_AHEAD; ++j) {
            const int rn = R0 + 32 * (LPT_AHEAD + j) + lane;
            tv_next[j] = (rn < n_req) ? Ts[rn] : 0u;
            rq_next[j] = (rn < n_req) ? od[rn] : 0u;
        }
        for (int r0 = R0; r0 < min(n_req, R0 + 32 * LPT_AHEAD); r0 += 32) {
            const int r = r0 + lane;
            const uint32_t tsh = s_tv[r - R0] << JB;    // this chunk's items, already in key units
            const uint32_t rq = s_rq[r - R0];
            const int steps = min(32, n_req - r0);
            uint32_t mine = 0;
            int pos = 0;
            while (pos < steps) {
                // sort all 32 * KPL keys ascending: element e = k * 32 + lane.  After a wave that
                // placed 32 items on 64 clients, the lower half (key[0]) is new and the upper half
                // is still in order: the lower half is sorted alone and merged with the upper one
                // (reversed, which makes the whole bitonic): 6 dependent compare-exchange steps
                // instead of 21.
                if (KPL == 2 && half_sorted) {
                    // the new half by rank: 32 independent compares instead of 15 dependent steps
                    // (keys are distinct: they carry their client)
                    uint32_t x = key[0];
                    int rk[4] = {0, 0, 0, 0};           // four short chains of additions instead of one long
#pragma unroll
                    for (int b = 0; b < 32; ++b) rk[b & 3] += __shfl_sync(FULL, x, b) < x ? 1 : 0;
                    if (HOS_IN((rk[0] + rk[1]) + (rk[2] + rk[3]), 32, 212)) s_perm[(rk[0] + rk[1]) + (rk[2] + rk[3])] = x;
                    __syncwarp();
                    x = s_perm[lane];
                    __syncwarp();
                    const uint32_t y = __shfl_sync(FULL, key[KPL - 1], 31 - lane);
                    uint32_t lo2 = min(x, y), hi2 = max(x, y);
#pragma unroll
                    for (int stride = 16; stride > 0; stride >>= 1) {
                        const uint32_t ol = __shfl_xor_sync(FULL, lo2, stride);
                        const uint32_t oh = __shfl_xor_sync(FULL, hi2, stride);
                        const bool lower = (lane & stride) == 0;
                        lo2 = lower ? min(lo2, ol) : max(lo2, ol);
                        hi2 = lower ? min(hi2, oh) : max(hi2, oh);
                    }
                    key[0] = lo2;
                    key[KPL - 1] = hi2;
                } else {
#pragma unroll
                for (int size = 2; size <= 32 * KPL; size <<= 1) {
#pragma unroll
                    for (int stride = size >> 1; stride > 0; stride >>= 1) {
                        if (stride < 32) {
#pragma unroll
                            for (int k = 0; k < KPL; ++k) {
                                const uint32_t other = __shfl_xor_sync(FULL, key[k], stride);
                                const bool up = ((k * 32 + lane) & size) == 0;
                                const bool lower = (lane & stride) == 0;
                                key[k] = (lower == up) ? min(key[k], other) : max(key[k], other);
                            }
                        } else {
                            const int kk = stride >> 5;
#pragma unroll
                            for (int k = 0; k < KPL; ++k) {
                                if ((k & kk) == 0) {
                                    const uint32_t a = key[k], b = key[k | kk];
                                    const bool up = ((k * 32) & size) == 0;
                                    key[k] = up ? min(a, b) : max(a, b);
                                    key[k | kk] = up ? max(a, b) : min(a, b);
                                }
                            }
                        }
                    }
                }
                }
                // lane a now holds the a-th smallest key in key[0]; item pos + a is its candidate
                if (pos == 0 && steps == 32) {
                    // a whole chunk at once when even the largest of the 32 keys is below every updated
                    // key (then it is below the updated keys of the lanes before it, and so are the
                    // smaller ones): one warp minimum instead of the prefix minimum
                    const uint32_t s_a = key[0];
                    const uint32_t u_a = s_a + tsh;
                    const uint32_t u_min = __reduce_min_sync(FULL, u_a);
                    const uint32_t s_top = __shfl_sync(FULL, s_a, 31);
                    if (s_top != 0xFFFFFFFFu && s_top < u_min) {
                        key[0] = u_a;
                        mine = s_a & ((1u << JB) - 1u);
                        pos = 32;
                        half_sorted = true;
                        continue;
                    }
                }
                const int src = pos + lane;
                const bool have = src < steps;
                const uint32_t t = __shfl_sync(FULL, tsh, src & 31);
                const uint32_t s_a = key[0];
                const uint32_t u_a = s_a + (have ? t : 0u);
                uint32_t inc = u_a;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t y = __shfl_up_sync(FULL, inc, d);
                    if (lane >= d) inc = min(inc, y);
                }
                uint32_t before = __shfl_up_sync(FULL, inc, 1);     // min of the updated keys of lower lanes
                if (lane == 0) before = 0xFFFFFFFFu;
                const bool ok = have && s_a != 0xFFFFFFFFu && (lane == 0 || s_a < before);
                const unsigned okm = __ballot_sync(FULL, ok);
                const int W = (okm == FULL) ? 32 : (__ffs(~okm) - 1);  // >= 1: lane 0 always qualifies
                if (lane < W) key[0] = u_a;
                const uint32_t jv = __shfl_sync(FULL, s_a & ((1u << JB) - 1u), (lane - pos) & 31);
                if (lane >= pos && lane < pos + W) mine = jv;
                pos += W;
                half_sorted = W == 32;
            }
            if (r < n_req && HOS_IN(rq, n_req, 211) && HOS_IN(mine, n_clients, 213)) {
                asg[rq] = (int32_t)mine;
                if (rc) rc[r] = (uint8_t)mine;
            }
            // re-base: subtract the current least relative load from every real key
            uint32_t m = key[0];
#pragma unroll
            for (int k = 1; k < KPL; ++k) m = min(m, key[k]);
            const uint32_t base = (__reduce_min_sync(FULL, m) >> JB) << JB;
            rebased += base >> JB;
#pragma unroll
            for (int k = 0; k < KPL; ++k)
                if (key[k] != 0xFFFFFFFFu) key[k] -= base;
        }
        }
        long long mx = 0;
#pragma unroll
        for (int k = 0; k < KPL; ++k) {
            if (key[k] != 0xFFFFFFFFu && HOS_IN(key[k] & ((1u << JB) - 1u), n_clients, 213)) {
                const long long l = (long long)(rebased + (key[k] >> JB));
                load_out[(size_t)inst * n_clients + (key[k] & ((1u << JB) - 1u))] = l;
                mx = l > mx ? l : mx;
            }
        }
        mx = warp_max_i64(mx);
        if (lane == 0) makespan_out[inst] = mx;
        return;
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
            if (r < n_req && HOS_IN(rq, n_req, 211) && HOS_IN(mine, n_clients, 213)) {
                asg[rq] = (int32_t)mine;
                if (rc) rc[r] = (uint8_t)mine;
            }
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
// Local search.  One small CTA per (instance, copy), many CTAs per SM: a round is a chain of
// short dependent phases, so throughput comes from running many instances side by side, not
// from a wide CTA.  The state of an instance is the clients' member lists in global memory
// (CSR: for every client its requests with T descending, index ascending inside equal T, as
// two arrays: T and request index); a round touches a few KB of them, which stay in L1/L2.
// Shared memory holds the loads, the list offsets and a copy of the critical client's list.
//
// A round looks for the minimum of (v, i, k, u) over every move (u = -1, d = T_i) and swap
// (d = T_i - T_u > 0) off the critical client jmax, v = max(Lmax - d, load_k + d).  For a
// fixed (k, u), v falls while 2 d < Lmax - load_k and rises afterwards, so only two members
// of jmax can win: the one with the largest T below the turning point and the one with the
// smallest T at or above it (first index of its run of equal T); both come from one binary
// search in jmax's member list.  Any step onto client k ends with
// v >= ceil((Lmax + load_k) / 2): the least loaded client is evaluated first, its best v
// bounds the optimum, and only clients whose floor does not exceed that bound are looked at
// (ties in v survive the filter).  Work items are taken from the member lists, so every lane
// has an item.  A swap keeps both list lengths: one warp per list shifts the entries between
// the old and the new position; a move rebuilds the lists from the assignment.
// ---------------------------------------------------------------------------------------
// A candidate step, ordered by (v, i, k, u) through three words that compare the same way:
// inv = ~(Lmax - v) (every useful candidate has 0 < Lmax - v <= T_i < 2^32), ik = i << 8 | k,
// u1 = u + 1 (0 for a move).  n_req < 2^15 and n_clients <= 2^8 keep ik inside 23 bits.
struct Cand {
    uint32_t inv, ik, u1;
    int pi, pu;        // positions of i in jmax's list and of u in k's list (pu = -1 for a move)
};
constexpr uint32_t NO_CAND = 0xFFFFFFFFu;

__device__ __forceinline__ bool cand_less(const Cand& a, const Cand& b) {
    if (a.inv != b.inv) return a.inv < b.inv;
    if (a.ik != b.ik) return a.ik < b.ik;
    return a.u1 < b.u1;
}

// Warp-wide minimum by three integer reductions; every lane gets the winner.
__device__ __forceinline__ Cand cand_warp_min(const Cand& c) {
    const uint32_t m0 = __reduce_min_sync(FULL, c.inv);
    const uint32_t m1 = __reduce_min_sync(FULL, c.inv == m0 ? c.ik : 0xFFFFFFFFu);
    const uint32_t m2 = __reduce_min_sync(FULL, (c.inv == m0 && c.ik == m1) ? c.u1 : 0xFFFFFFFFu);
    const unsigned who = __ballot_sync(FULL, c.inv == m0 && c.ik == m1 && c.u1 == m2);
    const int src = __ffs(who) - 1;
    Cand r;
    r.inv = m0; r.ik = m1; r.u1 = m2;
    r.pi = __shfl_sync(FULL, c.pi, src);
    r.pu = __shfl_sync(FULL, c.pu, src);
    return r;
}

constexpr long long NO_V = 0x7FFFFFFFFFFFFFFFll;
constexpr int NO_I = 0x7FFFFFFF;

constexpr int LS_THREADS = 128;
constexpr int LS_WARPS = LS_THREADS / 32;
constexpr int LS_STAGE = 512;             // longest critical list that is copied to shared memory
constexpr int LS_BATCH_MAX = 4;           // work items a thread has in flight: 2, 3 or 4, chosen per launch so
                                          // that a list of the usual length just fits one batch of the CTA

// Exclusive scan of a[0 .. len) in place by the whole CTA of NT threads; `wsum` holds NT / 32 words.
template <int NT>
__device__ inline void block_scan_u32(uint32_t* a, int len, uint32_t* wsum) {
    const int per = (len + NT - 1) / NT;
    const int lo = min(len, (int)threadIdx.x * per), hi = min(len, lo + per);
    uint32_t run = 0;
    for (int x = lo; x < hi; ++x) run += a[x];
    uint32_t inc = run;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(FULL, inc, d);
        if (lane_id() >= d) inc += y;
    }
    if (lane_id() == 31) wsum[warp_id()] = inc;
    __syncthreads();
    uint32_t before = 0;                                     // total of the warps before mine
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) before += w < warp_id() ? wsum[w] : 0u;
    uint32_t acc = before + inc - run;
    for (int x = lo; x < hi; ++x) { const uint32_t c = a[x]; a[x] = acc; acc += c; }
    __syncthreads();
}

// Member lists of all clients from the assignment: a stable split of the ranks 0..n-1 by
// client, as the members' request index (clI) and T (clT).  cnt holds n_clients * (NT / 32 + 1)
// words (NT = threads of the CTA; the odd row stride keeps the lanes of a warp on different banks).  off[k] = start of client k's list, off[M] = n.  rcl[r] is the client of rank r: with
// GATHER it is filled here from the assignment (asg[order[r]]), otherwise it was left by the
// packing kernel.  With CHECK, an assignment outside [0, M) makes every thread return true
// (lists not built), and `load`, if given, receives the clients' summed T.  Each warp takes
// LS_ROWS rows of 32 ranks at a time, so that their reads are in flight together.
constexpr int LS_ROWS = 4;
template <typename IdxT, bool CHECK, bool GATHER, int NT>
__device__ __noinline__ bool build_member_lists(const int32_t* asg, uint8_t* rcl, const uint32_t* __restrict__ gO,
                                          const uint32_t* __restrict__ gT, IdxT* clI, uint32_t* clT,
                                          int n, int n_clients, uint32_t* cnt, uint32_t* wsum, int* off,
                                          long long* load) {
    const int lane = lane_id(), warp = warp_id();
    const int chunk = (((n + (NT / 32) - 1) / (NT / 32)) + 31) & ~31;
    const int lo = warp * chunk, hi = min(n, lo + chunk);
    for (int x = threadIdx.x; x < n_clients * (NT / 32 + 1); x += NT) cnt[x] = 0;
    __syncthreads();
    bool bad = false;
    if (!GATHER) {
        // counts only: four ranks per lane and read
        for (int r4 = lo + 4 * lane; r4 < hi; r4 += 128) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(rcl + r4);   // rows start at multiples of 4
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (r4 + e < hi) atomicAdd(&cnt[((w >> (8 * e)) & 0xFFu) * (NT / 32 + 1) + warp], 1u);
        }
    } else {
        for (int row = lo; row < hi; row += 32 * LS_ROWS) {
            int c[LS_ROWS];
            uint32_t t[LS_ROWS], id[LS_ROWS];
#pragma unroll
            for (int e = 0; e < LS_ROWS; ++e) {
                const int r = row + e * 32 + lane;
                id[e] = r < hi ? __ldg(&gO[r]) : 0u;
                t[e] = (CHECK && load && r < hi) ? __ldg(&gT[r]) : 0u;
            }
#pragma unroll
            for (int e = 0; e < LS_ROWS; ++e) c[e] = row + e * 32 + lane < hi ? asg[id[e]] : 0;
#pragma unroll
            for (int e = 0; e < LS_ROWS; ++e) {
                const int r = row + e * 32 + lane;
                if (r < hi) {
                    if (CHECK && (c[e] < 0 || c[e] >= n_clients)) bad = true;
                    else {
                        rcl[r] = (uint8_t)c[e];
                        atomicAdd(&cnt[(uint32_t)c[e] * (NT / 32 + 1) + warp], 1u);
                        if (CHECK && load)
                            atomicAdd(reinterpret_cast<unsigned long long*>(&load[c[e]]), (unsigned long long)t[e]);
                    }
                }
            }
        }
    }
    if (CHECK) { if (__syncthreads_or(bad)) return true; }
    else __syncthreads();
    block_scan_u32<NT>(cnt, n_clients * (NT / 32 + 1), wsum);
    for (int k = threadIdx.x; k <= n_clients; k += NT)
        off[k] = k < n_clients ? (int)cnt[k * (NT / 32 + 1)] : n;
    __syncthreads();
    // placement, LS_ROWS rows at a time; the next rows' reads are in flight meanwhile
    const int nb = bit_width_u32((uint32_t)(n_clients - 1));
    uint32_t nid[LS_ROWS], ntr[LS_ROWS], ndig[LS_ROWS];
    auto fetch_rows = [&](int row) {
#pragma unroll
        for (int e = 0; e < LS_ROWS; ++e) {
            const int r = row + e * 32 + lane;
            const bool valid = r < hi;
            nid[e] = valid ? __ldg(&gO[r]) : 0u;
            ntr[e] = valid ? __ldg(&gT[r]) : 0u;
            ndig[e] = valid ? (uint32_t)rcl[r] : 0u;              // (with GATHER: written above by this same thread)
        }
    };
    if (lo < hi) fetch_rows(lo);
    for (int row = lo; row < hi; row += 32 * LS_ROWS) {
        uint32_t id[LS_ROWS], tr[LS_ROWS], dig[LS_ROWS];
        unsigned m[LS_ROWS];
#pragma unroll
        for (int e = 0; e < LS_ROWS; ++e) {
            id[e] = nid[e]; tr[e] = ntr[e]; dig[e] = ndig[e];
            m[e] = __ballot_sync(FULL, row + e * 32 + lane < hi);
        }
        if (row + 32 * LS_ROWS < hi) fetch_rows(row + 32 * LS_ROWS);
        for (int b = 0; b < nb; ++b) {                           // lanes of each row on my client
#pragma unroll
            for (int e = 0; e < LS_ROWS; ++e) {
                const bool bit = (dig[e] >> b) & 1u;
                const unsigned bal = __ballot_sync(FULL, bit);
                m[e] &= bit ? bal : ~bal;
            }
        }
#pragma unroll
        for (int e = 0; e < LS_ROWS; ++e) {
            const bool valid = row + e * 32 + lane < hi;
            const uint32_t base = valid ? cnt[dig[e] * (NT / 32 + 1) + warp] : 0u;
            __syncwarp();
            if (valid) {
                const uint32_t at = base + __popc(m[e] & ((1u << lane) - 1u));
                if (!HOS_IN(at, n, 222)) continue;
                clI[at] = (IdxT)id[e];
                clT[at] = tr[e];
                if (lane == (__ffs(m[e]) - 1)) cnt[dig[e] * (NT / 32 + 1) + warp] = base + __popc(m[e]);
            }
            __syncwarp();
        }
    }
    __syncthreads();
    return false;
}

// One warp: in the list (segT, segI)[0 .. len), ordered by (T descending, index ascending),
// drop the entry at position `gone` and insert (valT, valI) at its place in the order.
template <typename IdxT>
__device__ __noinline__ void warp_patch_list(uint32_t* segT, IdxT* segI, int len, int gone, uint32_t valT,
                                       uint32_t valI) {
    const int lane = lane_id();
    int a = 0, z = len;                                      // entries that come before the new one
    while (a < z) {
        const int mid = (a + z) >> 1;
        const uint32_t t = segT[mid];
        const bool before = t > valT || (t == valT && (uint32_t)segI[mid] < valI);
        if (before) a = mid + 1; else z = mid;
    }
    if (!HOS_IN(gone, len, 232) || !HOS_IN(a, len + 1, 231)) return;
    const uint32_t tg = segT[gone];
    const bool gone_before = tg > valT || (tg == valT && (uint32_t)segI[gone] < valI);
    const int at = a - (gone_before ? 1 : 0);                // position among the remaining entries
    if (at > gone) {                                         // entries (gone, at] move down by one
        for (int x0 = gone + 1; x0 <= at; x0 += 32) {
            const int x = x0 + lane;
            const bool ok = x <= at;
            const uint32_t t = ok ? segT[x] : 0u;
            const IdxT i = ok ? segI[x] : (IdxT)0;
            __syncwarp();
            if (ok) { segT[x - 1] = t; segI[x - 1] = i; }
        }
    } else if (at < gone) {                                  // entries [at, gone) move up by one
        for (int x1 = gone - 1; x1 >= at; x1 -= 32) {
            const int x = x1 - lane;
            const bool ok = x >= at;
            const uint32_t t = ok ? segT[x] : 0u;
            const IdxT i = ok ? segI[x] : (IdxT)0;
            __syncwarp();
            if (ok) { segT[x + 1] = t; segI[x + 1] = i; }
        }
    }
    __syncwarp();
    if (lane == 0) { segT[at] = valT; segI[at] = (IdxT)valI; }
}

// The same lists from the clients by rank that the packing kernel left (rcl), with coalesced
// list writes.  Counts per (client, warp) and their scan give every warp the place of its members
// in each client's list, as in build_member_lists.  Then a warp takes its ranks LSB_SUB at a time:
// it counts them per client, lays them out by client in a staging area of its own (a client's
// members of these ranks are consecutive in that client's list), and writes the staging area out
// in order, so that neighbouring lanes write neighbouring list entries instead of one list each.
// `stage` holds, per warp, LSB_SUB entries of T, index and client and two words per client.
constexpr int LSB_SUB = 512;
template <typename IdxT>
__host__ __device__ constexpr size_t lists_stage_bytes_per_warp(int n_clients) {
    return (size_t)LSB_SUB * (4 + sizeof(IdxT) + 1) + (size_t)((n_clients + 3) & ~3) * 8;
}
template <typename IdxT, int NT>
__device__ inline void place_lists_staged(const uint8_t* __restrict__ rcl, const uint32_t* __restrict__ gO,
                                          const uint32_t* __restrict__ gT, IdxT* clI, uint32_t* clT, int n,
                                          int n_clients, uint32_t* cnt, uint32_t* wsum, int* off,
                                          unsigned char* stage) {
    constexpr int NW = NT / 32, STRIDE = NW + 1;
    const int lane = lane_id(), warp = warp_id();
    const int chunk = (((n + NW - 1) / NW) + 31) & ~31;
    const int lo = warp * chunk, hi = min(n, lo + chunk);
    const int nb = bit_width_u32((uint32_t)(n_clients - 1));
    const int mpad = (n_clients + 3) & ~3;
    unsigned char* mine = stage + (size_t)warp * lists_stage_bytes_per_warp<IdxT>(n_clients);
    uint32_t* stT = reinterpret_cast<uint32_t*>(mine);
    uint32_t* lcur = stT + LSB_SUB;                          // per client: next free staging slot
    uint32_t* lbeg = lcur + mpad;                            // per client: its first staging slot
    IdxT* stI = reinterpret_cast<IdxT*>(lbeg + mpad);
    uint8_t* stC = reinterpret_cast<uint8_t*>(stI + LSB_SUB);

    for (int x = threadIdx.x; x < n_clients * STRIDE; x += NT) cnt[x] = 0;
    __syncthreads();
    for (int r4 = lo + 4 * lane; r4 < hi; r4 += 128) {       // four ranks per lane and read
        const uint32_t w = *reinterpret_cast<const uint32_t*>(rcl + r4);
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (r4 + e < hi) atomicAdd(&cnt[((w >> (8 * e)) & 0xFFu) * STRIDE + warp], 1u);
    }
    __syncthreads();
    block_scan_u32<NT>(cnt, n_clients * STRIDE, wsum);
    for (int k = threadIdx.x; k <= n_clients; k += NT) off[k] = k < n_clients ? (int)cnt[k * STRIDE] : n;
    __syncthreads();

    const int per = (n_clients + 31) / 32;                  // clients per lane in the scan below
    for (int sub = lo; sub < hi; sub += LSB_SUB) {
        const int end = min(hi, sub + LSB_SUB);
        for (int c = lane; c < n_clients; c += 32) lcur[c] = 0;
        __syncwarp();
        for (int r4 = sub + 4 * lane; r4 < end; r4 += 128) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(rcl + r4);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (r4 + e < end) atomicAdd(&lcur[(w >> (8 * e)) & 0xFFu], 1u);
        }
        __syncwarp();
        {   // exclusive scan of the counts over the clients: first staging slot of every client
            uint32_t run = 0;
            for (int k = 0; k < per; ++k) { const int c = lane * per + k; if (c < n_clients) run += lcur[c]; }
            uint32_t inc = run;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t y = __shfl_up_sync(FULL, inc, d);
                if (lane >= d) inc += y;
            }
            uint32_t acc = inc - run;
            for (int k = 0; k < per; ++k) {
                const int c = lane * per + k;
                if (c < n_clients) { const uint32_t v = lcur[c]; lbeg[c] = acc; lcur[c] = acc; acc += v; }
            }
        }
        __syncwarp();
        for (int row = sub; row < end; row += 32 * LS_ROWS) {
            uint32_t id[LS_ROWS], tr[LS_ROWS], dig[LS_ROWS];
            unsigned m[LS_ROWS];
#pragma unroll
            for (int e = 0; e < LS_ROWS; ++e) {
                const int r = row + e * 32 + lane;
                const bool valid = r < end;
                id[e] = valid ? __ldg(&gO[r]) : 0u;
                tr[e] = valid ? __ldg(&gT[r]) : 0u;
                dig[e] = valid ? (uint32_t)rcl[r] : 0u;
                m[e] = __ballot_sync(FULL, valid);
            }
            for (int b = 0; b < nb; ++b) {                   // lanes of each row on my client
#pragma unroll
                for (int e = 0; e < LS_ROWS; ++e) {
                    const bool bit = (dig[e] >> b) & 1u;
                    const unsigned bal = __ballot_sync(FULL, bit);
                    m[e] &= bit ? bal : ~bal;
                }
            }
#pragma unroll
            for (int e = 0; e < LS_ROWS; ++e) {
                const bool valid = row + e * 32 + lane < end;
                const uint32_t base = valid ? lcur[dig[e]] : 0u;
                __syncwarp();
                if (valid) {
                    const uint32_t at = base + __popc(m[e] & ((1u << lane) - 1u));
                    if (!HOS_IN(at, LSB_SUB, 224)) continue;
                    stT[at] = tr[e];
                    stI[at] = (IdxT)id[e];
                    stC[at] = (uint8_t)dig[e];
                    if (lane == (__ffs(m[e]) - 1)) lcur[dig[e]] = base + __popc(m[e]);
                }
                __syncwarp();
            }
        }
        for (int x = lane; x < end - sub; x += 32) {         // staging slot x -> its place in the client's list
            const uint32_t c = stC[x];
            if (!HOS_IN(c, n_clients, 223)) continue;
            const uint32_t g = cnt[c * STRIDE + warp] + ((uint32_t)x - lbeg[c]);
            if (!HOS_IN(g, n, 225)) continue;
            clT[g] = stT[x];
            clI[g] = stI[x];
        }
        __syncwarp();
        for (int c = lane; c < n_clients; c += 32) cnt[c * STRIDE + warp] += lcur[c] - lbeg[c];
        __syncwarp();
    }
    __syncthreads();
}

// Member lists before the first round: one CTA per (instance, copy).  Leaves the lists (ws_T,
// ws_I), their offsets (ws_off, n_clients + 1 per unit) and, for a caller's assignment, the
// clients' loads; ws_bad[unit] != 0 marks an assignment outside [0, n_clients).
constexpr int LSB_THREADS = 256;
template <typename IdxT>
__global__ void __launch_bounds__(LSB_THREADS)
k_ls_lists(const uint32_t* __restrict__ T_sorted, const uint32_t* __restrict__ order,
           const InstInfo* __restrict__ info, int n_req, int n_pad, int n_clients, int n_copies,
           bool load_from_assign, const int32_t* __restrict__ assign, long long* __restrict__ load_io,
           uint32_t* __restrict__ ws_T, IdxT* __restrict__ ws_I, uint8_t* __restrict__ ws_C,
           int32_t* __restrict__ ws_off, int32_t* __restrict__ ws_bad) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ long long s_load[MAX_CLIENTS];
    __shared__ int s_off[MAX_CLIENTS + 1];
    __shared__ uint32_t s_wsum[LSB_THREADS / 32];
    const int inst = blockIdx.x / n_copies;
    const size_t unit = blockIdx.x;
    if (info[inst].status) return;                          // the search kernel zeroes this unit's results
    uint32_t* cnt = reinterpret_cast<uint32_t*>(smem_raw);
    const uint32_t* gT = T_sorted + (size_t)inst * n_pad;
    const uint32_t* gO = order + (size_t)inst * n_pad;
    const int32_t* asg = assign + unit * n_req;
    for (int j = threadIdx.x; j < n_clients; j += LSB_THREADS) s_load[j] = 0;
    __syncthreads();
    // a caller's assignment is gathered and checked; the packing kernel's comes with the clients by rank
    bool failed = false;
    if (load_from_assign)
        failed = build_member_lists<IdxT, true, true, LSB_THREADS>(asg, ws_C + unit * n_pad, gO, gT,
                                                                   ws_I + unit * n_pad, ws_T + unit * n_pad, n_req,
                                                                   n_clients, cnt, s_wsum, s_off, s_load);
    else
        place_lists_staged<IdxT, LSB_THREADS>(ws_C + unit * n_pad, gO, gT, ws_I + unit * n_pad, ws_T + unit * n_pad,
                                              n_req, n_clients, cnt, s_wsum, s_off,
                                              smem_raw + (((size_t)n_clients * (LSB_THREADS / 32 + 1) * 4 + 15) & ~(size_t)15));
    if (threadIdx.x == 0) ws_bad[unit] = failed ? 1 : 0;
    if (failed) return;
    for (int k = threadIdx.x; k <= n_clients; k += LSB_THREADS) ws_off[unit * (n_clients + 1) + k] = s_off[k];
    if (load_from_assign)
        for (int j = threadIdx.x; j < n_clients; j += LSB_THREADS) load_io[unit * n_clients + j] = s_load[j];
}

// The clients one round looks at (see (b) in the kernel), double-buffered: the next round's list
// is made while the current step is applied.
struct LsListing {
    int as[MAX_CLIENTS + 1];            // first work item of every listed client, then the total
    int cb[MAX_CLIENTS];                // start of its member list
    uint32_t cs[MAX_CLIENTS];           // Lmax - load (when that fits 32 bits)
    uint8_t ak[MAX_CLIENTS];            // the client
    long long min_unlisted;             // least floor among the clients left out
    int na, nitems;
};

// b[u] += members with T >= thr[u], for NB searches side by side.  A = s_T + 1 holds the
// members' T (descending), then zeros up to 2^STEPS entries, and s_T[0] is all ones.
template <int STEPS, int NB>
__device__ __forceinline__ void count_ge_batch(const uint32_t* s_T, const uint32_t (&thr)[NB],
                                               int (&b)[NB], int top) {
    if (STEPS > 0) {
#pragma unroll
        for (int st = STEPS - 1; st >= 0; --st) {
#pragma unroll
            for (int u = 0; u < NB; ++u)
                if (s_T[b[u] + (1 << st)] >= thr[u]) b[u] += 1 << st;
        }
    } else {
        for (int step = top; step > 0; step >>= 1) {
#pragma unroll
            for (int u = 0; u < NB; ++u)
                if (s_T[b[u] + step] >= thr[u]) b[u] += step;
        }
    }
}

// Named barrier 1 pairs warp 0 (which finds the next critical client) with warp 1 (which copies
// that client's list) while the other warps patch the lists.
__device__ __forceinline__ void pair_arrive() { asm volatile("bar.arrive 1, 64;" ::: "memory"); }
__device__ __forceinline__ void pair_wait() { asm volatile("bar.sync 1, 64;" ::: "memory"); }
// Named barrier 2 lets warps 2 and 3, once their lists are patched, help with that copy.
__device__ __forceinline__ void trio_arrive() { asm volatile("bar.arrive 2, 96;" ::: "memory"); }
__device__ __forceinline__ void trio_wait() { asm volatile("bar.sync 2, 96;" ::: "memory"); }

template <typename IdxT, int LS_BATCH>
__global__ void __launch_bounds__(LS_THREADS, 7)
k_local_search(const uint32_t* __restrict__ T_sorted, const uint32_t* __restrict__ order,
               const InstInfo* __restrict__ info, int n_req, int n_pad, int n_clients,
               int n_copies, int rounds, bool load_from_assign,
               int32_t* __restrict__ assign, long long* __restrict__ load_io,
               long long* __restrict__ makespan_out, int32_t* __restrict__ rounds_applied,
               hos_ls_move* __restrict__ ls_log, int32_t* __restrict__ status_out,
               uint32_t* __restrict__ ws_T, IdxT* __restrict__ ws_I, uint8_t* __restrict__ ws_C,
               const int32_t* __restrict__ ws_off, const int32_t* __restrict__ ws_bad) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ long long s_load[MAX_CLIENTS];
    __shared__ int s_off[MAX_CLIENTS + 1];
    __shared__ Cand s_cand[LS_WARPS];
    __shared__ uint32_t s_wsum[LS_WARPS];
    __shared__ LsListing s_ls[2];
    __shared__ uint8_t s_listed[MAX_CLIENTS];
    __shared__ uint32_t s_T[LS_STAGE + 1];                  // [0] = all ones, [1 .. nm] = jmax's T, then zeros
    __shared__ IdxT s_I[LS_STAGE];                          // jmax's request indices
    __shared__ int s_jmax, s_kmin;
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
            for (int j = threadIdx.x; j < n_clients; j += LS_THREADS) ld[j] = 0;
            if (threadIdx.x == 0) makespan_out[unit] = 0;
        }
        if (threadIdx.x == 0) rounds_applied[unit] = 0;
        if (log)
            for (int r = threadIdx.x; r < rounds; r += LS_THREADS) log[r] = hos_ls_move{-1, -1, -1, 0};
        return;
    }

    uint32_t* clT = ws_T + unit * n_pad;                   // T of the members, CSR order
    IdxT* clI = ws_I + unit * n_pad;                       // request index of the members, CSR order
    uint8_t* rcl = ws_C + unit * n_pad;                    // client of every rank in sorted order
    uint32_t* cnt = reinterpret_cast<uint32_t*>(smem_raw);

    const uint32_t* gT = T_sorted + (size_t)inst * n_pad;
    const uint32_t* gO = order + (size_t)inst * n_pad;
    // lists, offsets and (for a caller's assignment) loads were left by k_ls_lists
    const bool lists_failed = ws_bad[unit] != 0;
    if (!lists_failed) {
        for (int j = threadIdx.x; j < n_clients; j += LS_THREADS) s_load[j] = ld[j];
        for (int k = threadIdx.x; k <= n_clients; k += LS_THREADS) s_off[k] = ws_off[unit * (n_clients + 1) + k];
    }
    __syncthreads();
    if (lists_failed) {
        if (threadIdx.x == 0) {
            atomicOr(&status_out[inst], HOS_ST_INVALID);
            rounds_applied[unit] = 0;
            makespan_out[unit] = 0;
        }
        for (int j = threadIdx.x; j < n_clients; j += LS_THREADS) ld[j] = 0;
        if (log)
            for (int r = threadIdx.x; r < rounds; r += LS_THREADS) log[r] = hos_ls_move{-1, -1, -1, 0};
        return;
    }

    int applied = 0;
    int done_at = rounds;
    long long margin = 64;                  // how far above the least loaded client's floor to look first

    // critical client (largest load, ties to the lowest client) and least loaded client (ties to the
    // highest, so that it differs from the critical one unless all loads are equal); one warp
    auto find_extremes = [&]() {
        long long bl = -1, ml = NO_V;
        int bj = NO_I, mj = -1;
        for (int j = lane; j < n_clients; j += 32) {
            const long long l = s_load[j];
            if (l > bl) { bl = l; bj = j; }
            if (l <= ml) { ml = l; mj = j; }
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const long long ol = __shfl_xor_sync(FULL, bl, d);
            const int oj = __shfl_xor_sync(FULL, bj, d);
            if (ol > bl || (ol == bl && oj < bj)) { bl = ol; bj = oj; }
            const long long pl = __shfl_xor_sync(FULL, ml, d);
            const int pj = __shfl_xor_sync(FULL, mj, d);
            if (pl < ml || (pl == ml && pj > mj)) { ml = pl; mj = pj; }
        }
        if (lane == 0) { s_jmax = bj; s_lmax = bl; s_kmin = mj; }
    };
    // One warp: the clients a round looks at, with the running count of their work items (see (b)).
    // Without skip_listed it also leaves the least floor of the clients it left out.
    auto list_clients = [&](LsListing& L, int jmax, long long Lmax, long long vlimit, bool skip_listed) {
        int n_alive = 0, n_items = 0;
        long long min_out = NO_V;
        for (int k0 = 0; k0 < n_clients; k0 += 32) {
            const int k = k0 + lane;
            bool alive = false;
            int sz = 0;
            if (k < n_clients && k != jmax) {
                const long long lk = s_load[k];
                const long long fl = (Lmax + lk + 1) >> 1;
                alive = lk < Lmax && fl <= vlimit && !(skip_listed && s_listed[k]);
                if (lk < Lmax && fl > vlimit) min_out = fl < min_out ? fl : min_out;
                sz = alive ? s_off[k + 1] - s_off[k] + 1 : 0;
                if (!skip_listed) s_listed[k] = alive;
                else if (alive) s_listed[k] = 1;
            }
            const unsigned am = __ballot_sync(FULL, alive);
            int inc = sz;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(FULL, inc, d);
                if (lane >= d) inc += y;
            }
            if (alive) {
                const int pos = n_alive + __popc(am & ((1u << lane) - 1u));
                L.ak[pos] = (uint8_t)k;
                L.as[pos] = n_items + inc - sz;
                L.cb[pos] = s_off[k];
                L.cs[pos] = (uint32_t)(Lmax - s_load[k]);
            }
            n_alive += __popc(am);
            n_items += __shfl_sync(FULL, inc, 31);
        }
        if (!skip_listed) {
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                const long long y = __shfl_xor_sync(FULL, min_out, d);
                min_out = y < min_out ? y : min_out;
            }
        }
        if (lane == 0) {
            L.na = n_alive; L.nitems = n_items; L.as[n_alive] = n_items;
            if (!skip_listed) L.min_unlisted = min_out;
        }
    };
    // Copy of a critical client's list to shared memory by `nthr` threads (this one is number `t`):
    // the T entries by asynchronous 4-byte copies (all in flight at once, no registers) with the
    // guard values written by hand, and the 2-byte request indices.  Each part ends when this
    // thread's share of it has landed.
    auto copy_list_T = [&](int base, int nmem, int t, int nthr) {
        const int top2 = 2 << (31 - __clz(nmem));
        for (int x = t; x <= top2; x += nthr) {
            if (x >= 1 && x <= nmem) {
                const unsigned sa = (unsigned)__cvta_generic_to_shared(&s_T[x]);
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" :: "r"(sa), "l"(clT + base + x - 1) : "memory");
            } else {
                s_T[x] = x == 0 ? 0xFFFFFFFFu : 0u;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    };
    auto copy_list_I = [&](int base, int nmem, int t, int nthr) {
#pragma unroll 4
        for (int x = t; x < nmem; x += nthr) s_I[x] = clI[base + x];
    };
    auto copy_list = [&](int base, int nmem, int t, int nthr) {
        copy_list_I(base, nmem, t, nthr);
        copy_list_T(base, nmem, t, nthr);
    };
    auto is_fast = [&](int nmem, long long Lmax) { return nmem >= 1 && nmem < LS_STAGE && Lmax <= 0x7FFFFFFFll; };
    auto floor_of_min = [&](int jmax, long long Lmax) {
        const int km = s_kmin;
        return (km != jmax && s_load[km] < Lmax) ? ((Lmax + s_load[km] + 1) >> 1) : Lmax;
    };
    if (warp == 0) find_extremes();
    __syncthreads();

    bool have_list = false;                 // this round's listing was made during the last apply
    bool have_copy = false;                 // and so was the copy of the critical list
    int buf = 0;
    for (int round = 0; round < rounds; ++round) {
        LsListing& L = s_ls[buf];
        const int jmax = s_jmax;
        const long long Lmax = s_lmax;
        // all loads equal: the least loaded client is as loaded as the critical one; nothing can improve
        const long long floor_min = floor_of_min(jmax, Lmax);
        const int base_j = s_off[jmax];
        const int nm = s_off[jmax + 1] - base_j;            // jmax's members, T descending
        // short critical list and loads below 2^31: the list is copied to shared memory and the
        // evaluation runs in 32-bit arithmetic; otherwise the general form reads it in place
        const bool fast = is_fast(nm, Lmax);
        const int top = fast ? 1 << (31 - __clz(nm)) : 0;  // largest power of two <= nm

        // (a) one work item: partner (Tu, u1 = u + 1, position pu; the move has Tu = 0, u1 = 0,
        //     pu = -1) on client k, against jmax's list (memT, memI)
        auto evaluate = [&](const uint32_t* memT, const IdxT* memI, int k, uint32_t Tu32, uint32_t u1, int pu,
                            Cand& best) {
            const long long slack = Lmax - s_load[k];
            const long long Tu = Tu32;
            const long long thr64 = Tu + ((slack + 1) >> 1);    // T_i >= thr  <=>  2 d >= slack
            const uint32_t thr = (uint32_t)thr64;
            int a = 0, z = thr64 > 0xFFFFFFFFll ? 0 : nm;       // b = members with T >= thr (none if it
            while (a < z) {                                     // is beyond every T)
                const int mid = (a + z) >> 1;
                if (memT[mid] >= thr) a = mid + 1; else z = mid;
            }
            const int b = a;
            if (b > 0) {                                        // rising side: smallest T >= thr
                const uint32_t Ti = memT[b - 1];
                const long long d = (long long)Ti - Tu;
                if (d < slack) {
                    int a2 = b - 1;                             // first member of the run of equal T
                    if (b >= 2 && memT[b - 2] == Ti) {
                        int z2 = b - 2;
                        a2 = 0;
                        while (a2 < z2) {
                            const int mid = (a2 + z2) >> 1;
                            if (memT[mid] > Ti) a2 = mid + 1; else z2 = mid;
                        }
                    }
                    Cand c;                                     // v = lk + d, Lmax - v = slack - d
                    c.inv = ~(uint32_t)(slack - d); c.pi = a2; c.ik = ((uint32_t)memI[a2] << 8) | (uint32_t)k;
                    c.u1 = u1; c.pu = pu;
                    if (cand_less(c, best)) best = c;
                }
            }
            if (b < nm) {                                       // falling side: largest T < thr
                const long long d = (long long)memT[b] - Tu;
                if (d > 0) {
                    Cand c;                                     // v = Lmax - d
                    c.inv = ~(uint32_t)d; c.pi = b; c.ik = ((uint32_t)memI[b] << 8) | (uint32_t)k;
                    c.u1 = u1; c.pu = pu;
                    if (cand_less(c, best)) best = c;
                }
            }
        };
        // (b) The clients to look at are listed with the running count of their work items (list
        //     length + 1 move).  Any step onto client k ends with v >= floor_k = ceil((Lmax + load_k) / 2),
        //     so a client whose floor is above an achieved v cannot win or tie.  First pass: the
        //     clients whose floor is within `margin` of the least loaded client's; after the
        //     reduction, if a client left out has a floor that does not exceed the best v found, those
        //     are evaluated in a second pass (vlimit = that v), which makes the result exact whatever
        //     the margin was.
        auto evaluate_listed = [&](Cand& best) {
            const int n_items = L.nitems;
            const uint32_t* memT = clT + base_j;
            const IdxT* memI = clI + base_j;
            int ci = 0;
            for (int x = threadIdx.x; x < n_items; x += LS_THREADS) {
                while (x >= L.as[ci + 1]) ++ci;                 // as[n_alive] = n_items ends the walk
                const int k = L.ak[ci], idx = x - L.as[ci], at = L.cb[ci] + idx;
                if (x + 1 < L.as[ci + 1]) evaluate(memT, memI, k, clT[at], (uint32_t)clI[at] + 1u, idx, best);
                else evaluate(memT, memI, k, 0u, 0u, -1, best);
            }
        };
        // The same over the shared-memory copy.  A = s_T + 1 holds the members' T, then zeros up to
        // 2 * top entries, and A[-1] is all ones: the number of members with T >= thr comes from
        // a fixed sequence of probes without bounds tests, and both neighbours of the turning point
        // can be read unconditionally (the guard values never make a valid step).  A thread takes
        // LS_BATCH items at a time: their partners' T are fetched together, one batch ahead of their
        // use, and the searches of a batch advance side by side, so that neither the list reads nor
        // the probe chains are waited for one by one.  The partner's request index is read only
        // when (v, i, k) ties, or at the end for the thread's best step.
        auto count_ge = [&](uint32_t thr) {
            int cnt_ge = 0;
            for (int step = top; step > 0; step >>= 1)
                if (s_T[cnt_ge + step] >= thr) cnt_ge += step;   // A[cnt_ge + step - 1]
            return cnt_ge;
        };
        auto evaluate_listed_fast = [&](Cand& best, auto steps_c) {
            constexpr int STEPS = decltype(steps_c)::value;
            const int na = L.na;
            int best_at = -1;                                   // where the best partner's index is, if not read yet
            auto consider = [&](uint32_t inv, int pi, uint32_t k, bool move, int at, int idx) {
                if (!HOS_IN(pi, LS_STAGE, 242)) return;
                const uint32_t ik = ((uint32_t)s_I[pi] << 8) | k;
                if (inv < best.inv || (inv == best.inv && ik < best.ik)) {
                    best.inv = inv; best.ik = ik; best.pi = pi; best.pu = move ? -1 : idx;
                    best.u1 = 0u; best_at = move ? -1 : at;
                } else if (inv == best.inv && ik == best.ik) {
                    if (best_at >= 0) { best.u1 = (uint32_t)clI[best_at] + 1u; best_at = -1; }
                    const uint32_t u1 = move ? 0u : (uint32_t)clI[at] + 1u;
                    if (u1 < best.u1) { best.pi = pi; best.pu = move ? -1 : idx; best.u1 = u1; }
                }
            };
            // The listed clients one after the other, so that client, list start and slack are the
            // same for the whole CTA; item idx of a client is its idx-th member, idx = len is the move.
            // Nothing worse than the best step any lane of this warp has found so far can be the CTA's
            // minimum, so that (one warp minimum per batch) is what a candidate is held against first:
            // against its own best alone nearly every item would send some lane of the warp down the
            // bookkeeping path.  Equal values pass: the order among them is decided by (i, k, u).
            uint32_t wbest = NO_CAND;
            uint32_t nTu[LS_BATCH];                             // next batch: partner T (0 for the move)
            auto fetch = [&](int cb, int len, int i0) {
#pragma unroll
                for (int u = 0; u < LS_BATCH; ++u) {
                    const int idx = i0 + u * LS_THREADS + (int)threadIdx.x;
                    nTu[u] = idx < len ? clT[cb + idx] : 0u;
                }
            };
            if (na > 0) fetch(L.cb[0], L.as[1] - L.as[0] - 1, 0);
            for (int ci = 0; ci < na; ++ci) {
                const int cb = L.cb[ci], len = L.as[ci + 1] - L.as[ci] - 1;
                const uint32_t slack = L.cs[ci], half = (slack + 1u) >> 1, k = L.ak[ci];
                for (int i0 = 0; i0 <= len; i0 += LS_BATCH * LS_THREADS) {
                    uint32_t Tu[LS_BATCH], thr[LS_BATCH];
                    int b[LS_BATCH];
#pragma unroll
                    for (int u = 0; u < LS_BATCH; ++u) { Tu[u] = nTu[u]; thr[u] = Tu[u] + half; b[u] = 0; }
                    // the next batch's reads are in flight during this batch's searches
                    if (i0 + LS_BATCH * LS_THREADS <= len) fetch(cb, len, i0 + LS_BATCH * LS_THREADS);
                    else if (ci + 1 < na) fetch(L.cb[ci + 1], L.as[ci + 2] - L.as[ci + 1] - 1, 0);
                    count_ge_batch<STEPS, LS_BATCH>(s_T, thr, b, top);
#pragma unroll
                    for (int u = 0; u < LS_BATCH; ++u) {
                        const int idx = i0 + u * LS_THREADS + (int)threadIdx.x;
                        if (idx > len) continue;
                        if (!HOS_IN(b[u] + 1, LS_STAGE + 1, 241) || !HOS_IN(cb + idx, n_req + 1, 246)) continue;
                        const uint32_t Ti = s_T[b[u]];          // A[b - 1]: smallest T >= thr (rising side)
                        const uint32_t d = Ti - Tu[u];
                        const uint32_t inv_r = d < slack ? ~(slack - d) : NO_CAND;
                        const int d2 = (int)(s_T[b[u] + 1] - Tu[u]);   // A[b]: largest T < thr (falling side)
                        const uint32_t inv_f = d2 > 0 ? ~(uint32_t)d2 : NO_CAND;
                        if (min(inv_r, inv_f) > wbest) continue;        // NO_CAND is the largest value
                        const bool move = idx == len;
                        if (inv_r != NO_CAND && inv_r <= best.inv) {
                            // first member of the run of equal T: b - 1 itself unless its predecessor ties
                            const int pi = s_T[b[u] - 1] != Ti ? b[u] - 1 : count_ge(Ti + 1u);
                            consider(inv_r, pi, k, move, cb + idx, idx);
                        }
                        if (inv_f != NO_CAND && inv_f <= best.inv) consider(inv_f, b[u], k, move, cb + idx, idx);
                    }
                    wbest = __reduce_min_sync(FULL, best.inv);
                }
            }
            if (best_at >= 0) best.u1 = (uint32_t)clI[best_at] + 1u;
        };
        Cand best;
        best.inv = NO_CAND; best.ik = NO_CAND; best.u1 = NO_CAND; best.pi = -1; best.pu = -1;
        if (!have_list || (fast && !have_copy)) {
            if (warp == 0) { if (!have_list) list_clients(L, jmax, Lmax, floor_min + margin, false); }
            else if (fast && !have_copy) copy_list(base_j, nm, (int)threadIdx.x - 32, LS_THREADS - 32);
            __syncthreads();
        }
        long long best_v = Lmax;
        for (int pass = 0; pass < 2; ++pass) {
            if (!fast) evaluate_listed(best);
            else evaluate_listed_fast(best, std::integral_constant<int, 0>());
            // CTA-wide lexicographic minimum: per warp, then every warp reduces the warps' records
            best = cand_warp_min(best);
            if (lane == 0) s_cand[warp] = best;
            __syncthreads();
            {
                Cand mine;
                mine.inv = NO_CAND; mine.ik = NO_CAND; mine.u1 = NO_CAND; mine.pi = -1; mine.pu = -1;
                if (lane < LS_WARPS) mine = s_cand[lane];
                best = cand_warp_min(mine);
            }
            best_v = best.inv != NO_CAND ? Lmax - (long long)(~best.inv) : Lmax;
            // is a client that was left out still able to reach best_v?  (uniform)
            if (pass == 1 || L.min_unlisted > best_v) break;
            __syncthreads();                                    // everyone has read the listing
            if (warp == 0) list_clients(L, jmax, Lmax, best_v, true);
            __syncthreads();
        }
        const bool ok = best.inv != NO_CAND;                    // a candidate always has v < Lmax
        if (!ok) {
            if (threadIdx.x == 0 && log) log[round] = hos_ls_move{-1, -1, -1, Lmax};
            done_at = round;
            break;
        }
        margin = (best_v - floor_min) + 2;                      // uniform: every thread holds the same best
        const int best_k = (int)(best.ik & 0xFFu);
        const int best_i = (int)(best.ik >> 8);
        const int best_u = (int)best.u1 - 1;
        const bool swap = best.pu >= 0;
        // (c) apply.  Warp 0 updates the two loads, finds the next round's extremes and lists its
        //     clients; warp 1 writes the assignment and the log and, once warp 0 has the next critical
        //     client, copies its list unless that is one of the two being patched; warps 2 and 3 patch
        //     one member list each.  (A move rebuilds the lists, so nothing is prepared ahead.)
        const int base_k = s_off[best_k];
        if (!HOS_IN(base_j + best.pi, n_req, 247) || !HOS_IN(base_k + (swap ? best.pu : 0), n_req + 1, 247)) break;   // uniform
        const uint32_t Ti_w = clT[base_j + best.pi];            // read by every warp before any list changes
        const uint32_t Tu_w = swap ? clT[base_k + best.pu] : 0u;
        __syncthreads();
        if (warp == 0) {
            const long long dT = (long long)Ti_w - (long long)Tu_w;
            if (lane == 0) { s_load[jmax] -= dT; s_load[best_k] += dT; }
            __syncwarp();
            find_extremes();
            __syncwarp();
            __threadfence_block();                              // the extremes are written before warp 1 is let go
            pair_arrive();
            if (swap) trio_arrive();
            if (swap) {
                const int nj = s_jmax;
                const long long nL = s_lmax;
                list_clients(s_ls[buf ^ 1], nj, nL, floor_of_min(nj, nL) + margin, false);
            }
        } else if (warp == 1) {
            if (lane == 0 && HOS_IN(best_i, n_req, 243) && HOS_IN(best_k, n_clients, 244) && HOS_IN(best_u + 1, n_req + 1, 243)) {
                asg[best_i] = best_k;
                if (best_u >= 0) asg[best_u] = jmax;
                if (log) log[round] = hos_ls_move{best_i, best_u, best_k, best_v};
            }
            __syncwarp();
            pair_wait();
            const int nj = s_jmax;
            if (swap && nj != jmax && nj != best_k) {
                const int nb = s_off[nj], nn = s_off[nj + 1] - nb;
                if (is_fast(nn, s_lmax)) copy_list_T(nb, nn, lane, 32);   // warps 2 and 3 bring the indices
            }
        } else if (swap) {
            if (warp == 2) warp_patch_list<IdxT>(clT + base_j, clI + base_j, nm, best.pi, Tu_w, (uint32_t)best_u);
            else if (warp == 3)
                warp_patch_list<IdxT>(clT + base_k, clI + base_k, s_off[best_k + 1] - base_k, best.pu, Ti_w,
                                      (uint32_t)best_i);
            trio_wait();                                        // warp 0 has found the next critical client
            const int nj = s_jmax;
            if (nj != jmax && nj != best_k) {
                const int nb = s_off[nj], nn = s_off[nj + 1] - nb;
                if (is_fast(nn, s_lmax)) copy_list_I(nb, nn, (int)threadIdx.x - 64, 64);
            }
        }
        __syncthreads();
        if (!swap)
            build_member_lists<IdxT, false, true, LS_THREADS>(asg, rcl, gO, gT, clI, clT, n_req, n_clients, cnt, s_wsum,
                                                              s_off, nullptr);
        have_list = swap;
        have_copy = swap && s_jmax != jmax && s_jmax != best_k;
        buf ^= 1;
        ++applied;
    }
    // a round without an improving step leaves the state as it is: all later rounds are the same
    if (log && done_at < rounds) {
        const hos_ls_move noop = hos_ls_move{-1, -1, -1, s_lmax};
        for (int r = done_at + 1 + threadIdx.x; r < rounds; r += LS_THREADS) log[r] = noop;
    }
    for (int j = threadIdx.x; j < n_clients; j += LS_THREADS) { ld[j] = s_load[j]; }
    if (warp == 0) {
        long long mx = 0;
        for (int j = lane; j < n_clients; j += 32) mx = s_load[j] > mx ? s_load[j] : mx;
        mx = warp_max_i64(mx);
        if (lane == 0) { makespan_out[unit] = mx; rounds_applied[unit] = applied; }
    }
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------

size_t estimate_sort_smem(int n_req) { return sort_smem_bytes<uint16_t>(n_req); }
size_t local_search_smem(int /*n_req*/, int n_clients) { return (size_t)n_clients * (LS_WARPS + 1) * 4; }
size_t local_search_index_bytes(int n_req) { return n_req <= 65536 ? 2 : 4; }

cudaError_t launch_estimate_sort(const hos_batch& b, const hos_cost_model& cm, uint32_t* T_sorted,
                                 uint32_t* order, InstInfo* info, int32_t* status_out, hos_lb* lb_out, int n_pad,
                                 cudaStream_t st) {
    // T_sorted == nullptr: the bounds only (no order is written; T_(M), T_(M+1) come from a selection)
    cudaError_t e = allow_max_dynamic_smem(reinterpret_cast<const void*>(k_estimate_sort<true>));
    if (e != cudaSuccess) return e;
    if ((e = allow_max_dynamic_smem(reinterpret_cast<const void*>(k_estimate_sort<false>))) != cudaSuccess) return e;
    int q_shift = -1;                                    // power-of-two KV divisor -> shift
    if ((cm.decode_kv_div & (cm.decode_kv_div - 1)) == 0)
        for (q_shift = 0; (1u << q_shift) != cm.decode_kv_div; ++q_shift) {}
    const long long most = b.kv_reserve_tokens ? (long long)b.kv_reserve_tokens : (long long)b.kv_budget;
    launch_hook("k_estimate_sort", 0, st);
    k_estimate_sort<true><<<b.n_inst, SORT_THREADS, bucket_sort_smem_bytes(b.n_req), st>>>(
        b.p, b.o, b.o_est, b.n_inst, b.n_req, most, stage_cap_tokens(cm), cm, q_shift, b.n_clients, b.batch_cap,
        T_sorted, order, info, status_out, lb_out, n_pad);
    launch_hook("k_estimate_sort", 1, st);
    // the instances the bucket sort declined (none, as a rule): one CTA per SM at most, each
    // walking the batch for pending instances
    int n_sm = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    launch_hook("k_estimate_sort_radix", 0, st);
    k_estimate_sort<false><<<b.n_inst < n_sm ? b.n_inst : n_sm, SORT_THREADS, estimate_sort_smem(b.n_req), st>>>(
        b.p, b.o, b.o_est, b.n_inst, b.n_req, most, stage_cap_tokens(cm), cm, q_shift, b.n_clients, b.batch_cap,
        T_sorted, order, info, status_out, lb_out, n_pad);
    launch_hook("k_estimate_sort_radix", 1, st);
    return cudaGetLastError();
}

HOS_DEFINE_BOUNDS_READER(debug_bounds_offline)

cudaError_t launch_lpt(const hos_batch& b, const uint32_t* T_sorted, const uint32_t* order,
                       const InstInfo* info, int n_pad, int32_t* assign, long long* load,
                       long long* makespan, uint8_t* rank_client, cudaStream_t st) {
    const int M = b.n_clients;
#define HOS_LPT(KPL)                                                                               \
    k_lpt<KPL><<<b.n_inst, 32, 0, st>>>(T_sorted, order, info, b.n_req, n_pad, M, assign, load,    \
                                         makespan, rank_client)
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
                                int32_t* status, uint32_t* ws_T, void* ws_I, uint8_t* ws_C, int32_t* ws_off,
                                int32_t* ws_bad, cudaStream_t st) {
    const size_t smem = local_search_smem(b.n_req, b.n_clients);
    const bool narrow = b.n_req <= 65536;
    const size_t smem_lists = (((size_t)b.n_clients * (LSB_THREADS / 32 + 1) * 4 + 15) & ~(size_t)15) +
                              (load_from_assign ? 0
                                                : (LSB_THREADS / 32) * (narrow ? lists_stage_bytes_per_warp<uint16_t>(b.n_clients)
                                                                               : lists_stage_bytes_per_warp<uint32_t>(b.n_clients)));
    cudaError_t ea = narrow ? allow_max_dynamic_smem(reinterpret_cast<const void*>(k_ls_lists<uint16_t>))
                            : allow_max_dynamic_smem(reinterpret_cast<const void*>(k_ls_lists<uint32_t>));
    if (ea != cudaSuccess) return ea;
    const unsigned grid = (unsigned)(b.n_inst * n_copies);
    launch_hook("k_ls_lists", 0, st);
    if (b.n_req <= 65536)
        k_ls_lists<uint16_t><<<grid, LSB_THREADS, smem_lists, st>>>(
            T_sorted, order, info, b.n_req, n_pad, b.n_clients, n_copies, load_from_assign, assign, load, ws_T,
            static_cast<uint16_t*>(ws_I), ws_C, ws_off, ws_bad);
    else
        k_ls_lists<uint32_t><<<grid, LSB_THREADS, smem_lists, st>>>(
            T_sorted, order, info, b.n_req, n_pad, b.n_clients, n_copies, load_from_assign, assign, load, ws_T,
            static_cast<uint32_t*>(ws_I), ws_C, ws_off, ws_bad);
    launch_hook("k_ls_lists", 1, st);
    // searches in flight per thread: a list of the usual length (and a little more: the packing
    // balances times, not counts), plus the move, should fit one batch of LS_THREADS x nb items
    const long long usual = ((long long)b.n_req / b.n_clients + 1) * 115 / 100;
    const int nb = usual <= 2 * LS_THREADS ? 2 : (usual <= 3 * LS_THREADS ? 3 : LS_BATCH_MAX);
    launch_hook("k_local_search", 0, st);
#define HOS_LS(IDX, NB)                                                                              \
    k_local_search<IDX, NB><<<grid, LS_THREADS, smem, st>>>(                                         \
        T_sorted, order, info, b.n_req, n_pad, b.n_clients, n_copies, rounds, load_from_assign, assign, \
        load, makespan, rounds_applied, ls_log, status, ws_T, static_cast<IDX*>(ws_I), ws_C, ws_off, ws_bad)
    if (narrow) {
        if (nb == 2) HOS_LS(uint16_t, 2); else if (nb == 3) HOS_LS(uint16_t, 3); else HOS_LS(uint16_t, 4);
    } else {
        if (nb == 2) HOS_LS(uint32_t, 2); else if (nb == 3) HOS_LS(uint32_t, 3); else HOS_LS(uint32_t, 4);
    }
#undef HOS_LS
    launch_hook("k_local_search", 1, st);
    return cudaGetLastError();
}

}  // namespace hos
