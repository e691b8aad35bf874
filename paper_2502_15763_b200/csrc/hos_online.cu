// Online scheduling kernels (Section "Online requests and iteration scheduling"):
//   k_queue_build    per-client queues in the order of Algorithm 1
//   k_simulate       iteration-level simulation, one thread per (instance, multiplier, client)
//   k_simulate_steal the same with Algorithm 1's request stealing, one CTA per simulation
//   k_trace_fill     the iteration trace rebuilt from the simulator's event log
//   k_finalize       per-simulation makespan, utilisation, generation speed
//   k_trace_offsets  exclusive scan of the per-client iteration counts
#include "hos_common.cuh"
#include "hos_kernels.h"
#include "hos_sort.cuh"

namespace hos {

constexpr int INST_WIDE = 0x100;         // internal flag in the workspace's per-instance status word

// ---------------------------------------------------------------------------------------
// Queue build: a segmented sort of the instance's requests by (client ascending,
// N^p + N^d descending, index ascending) -- one stable radix sort on the composite key
// client << kb | (2^kb - 1 - (p + o)).  HOS_QUEUE_FCFS sorts by client only.
// ---------------------------------------------------------------------------------------
// FAST: the bucket sort, one CTA per instance; an instance it declines keeps INST_PENDING in its
// status word and the second launch (!FAST, persistent CTAs, radix sort) takes it.
constexpr int INST_PENDING = 0x200;      // internal flag: queues not built yet

template <bool FAST>
__global__ void __launch_bounds__(SORT_THREADS, 1)
k_queue_build(const uint32_t* __restrict__ p, const uint32_t* __restrict__ o,
              const uint32_t* __restrict__ o_est,
              const int32_t* __restrict__ assign, int n_inst, int n_req, int n_clients, long long kv_budget,
              uint32_t p_max, int queue_order, uint2* __restrict__ q_po, uint32_t* __restrict__ q_key,
              uint32_t* __restrict__ q_req,
              int32_t* __restrict__ q_off, unsigned long long* __restrict__ inst_O,
              int32_t* __restrict__ inst_status, int n_pad) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int cbits = bit_width_u32((uint32_t)(n_clients - 1));
    for (int inst = blockIdx.x; inst < n_inst; inst += gridDim.x) {
        if (!FAST) {
            __syncthreads();
            if (!(inst_status[inst] & INST_PENDING)) continue;    // uniform
        }
        const uint32_t* pi = p + (size_t)inst * n_req;
        const uint32_t* oi = o + (size_t)inst * n_req;
        const int32_t* ai = assign + (size_t)inst * n_req;
        const uint32_t* ei = o_est ? o_est + (size_t)inst * n_req : oi;   // the lengths the scheduler sorts by
        // the radix path keeps the keys here, and the clients beside them until the keys are composed
        uint32_t* key = reinterpret_cast<uint32_t*>(smem_raw);
        uint16_t* park = reinterpret_cast<uint16_t*>(smem_raw + align16((size_t)n_req * 4));

        // first pass: checks and sums.  kv_budget here is the most KV one request may need: the
        // fixed reservation, if there is one
        // (the maxima in 32 bits: a sum that does not fit marks the instance bad, and then they are not used)
        unsigned long long sumO = 0;
        uint32_t mx = 0, mxk = 0, mxp = 0;
        int bad = 0;
        for_each_request(pi, oi, ei, ai, n_req, [&](int i, uint32_t pp, uint32_t oo, uint32_t oe, int c) {
            const unsigned long long tot = (unsigned long long)pp + oo;
            const unsigned long long totk = (unsigned long long)pp + oe;
            if (pp == 0 || oo == 0 || oe == 0 || pp > p_max || (long long)tot > kv_budget || totk > 0xFFFFFFFFull ||
                c < 0 || c >= n_clients)
                bad = 1;
            if (!FAST) { key[i] = (uint32_t)totk; park[i] = (uint16_t)(c & 0xFF); }
            sumO += oo;
            mx = max(mx, (uint32_t)tot);
            mxk = max(mxk, (uint32_t)totk);
            mxp = max(mxp, pp);
        });
        // per warp, one barrier, then every warp finishes all four from the warps' values.  The scratch
        // is a part of the sort's shared memory that nothing uses before the sort starts.
        unsigned long long* red = reinterpret_cast<unsigned long long*>(
            FAST ? smem_raw : reinterpret_cast<unsigned char*>(sort_smem_carve<uint16_t>(smem_raw, n_req).cnt));
        uint32_t (*redm)[SORT_WARPS] = reinterpret_cast<uint32_t (*)[SORT_WARPS]>(red + SORT_WARPS);
        sumO = warp_sum_u64(sumO);
        mx = __reduce_max_sync(FULL, mx);
        mxk = __reduce_max_sync(FULL, mxk);
        mxp = __reduce_max_sync(FULL, mxp);
        if (lane_id() == 0) { red[warp_id()] = sumO; redm[0][warp_id()] = mx; redm[1][warp_id()] = mxk; redm[2][warp_id()] = mxp; }
        bad = __syncthreads_or(bad);
        sumO = warp_sum_u64(red[lane_id()]);
        mx = __reduce_max_sync(FULL, redm[0][lane_id()]);
        mxk = __reduce_max_sync(FULL, redm[1][lane_id()]);
        mxp = __reduce_max_sync(FULL, redm[2][lane_id()]);
        __syncthreads();                                  // the scratch is the sort's again
        const int kb = (queue_order == HOS_QUEUE_SORTED) ? bit_width_u32((uint32_t)mxk) : 0;
        // the composite sort key, client above p + (estimated) o, has 32 bits: an estimate so long
        // that it does not fit beside the client bits invalidates the instance (uniform over the CTA)
        if (kb + cbits > 32) bad = 1;
        // bit 8 (internal): some p + o needs more than 16 bits -> the simulator's wide heap entries
        const int32_t st_done = bad ? HOS_ST_INVALID : (mx >= 65536u ? INST_WIDE : 0);
        if (bad) {
            if (threadIdx.x == 0) { inst_O[inst] = sumO; inst_status[inst] = st_done; }
            continue;
        }
        const uint32_t kmask = kb >= 32 ? 0xFFFFFFFFu : ((1u << kb) - 1u);
        uint2* qp = q_po + (size_t)inst * n_pad;
        uint32_t* qr = q_req + (size_t)inst * n_pad;
        uint32_t* qk = q_key ? q_key + (size_t)inst * n_pad : nullptr;
        int32_t* qo = q_off + (size_t)inst * (n_clients + 1);
        if (FAST) {
            // Sort key: the client above the length key 2^kb - 1 - (p + o) (longest first), or above
            // the request index for first-come-first-served queues; ties never arise beyond the
            // index.  The prompt length rides in an entry's spare bits when it fits, so that the queue
            // entries are written without going back to the request tables in queue order (a
            // scattered read per request); with the key p + o the output length follows from it too.
            const bool by_len = kb > 0;
            const int sbits = by_len ? kb : (n_req > 1 ? bit_width_u32((uint32_t)(n_req - 1)) : 1);
            const int nbits = sbits + cbits;             // <= 32 (checked above; 15 + 8 for the index form)
            BucketSort B;
            const int pbits = bit_width_u32((uint32_t)mxp);
            bool ok = bucket_sort_plan(B, smem_raw, n_req, nbits, pbits);
            const bool ride = ok;
            if (!ok) ok = bucket_sort_plan(B, smem_raw, n_req, nbits, 0);
            const bool o_from_key = ride && by_len && kb < 32 && !o_est;
            auto sort_key = [&](int i, uint32_t pp, uint32_t oe, int c) -> uint32_t {
                const uint32_t low = by_len ? kmask - ((pp + oe) & kmask) : (uint32_t)i;
                return (sbits >= 32 ? 0u : ((uint32_t)c << sbits)) | low;
            };
            if (ok) {
                bucket_sort_clear(B);
                for_each_request(pi, oi, ei, ai, n_req, [&](int i, uint32_t pp, uint32_t, uint32_t oe, int c) {
                    bucket_sort_count(B, sort_key(i, pp, oe, c));
                });
                ok = bucket_sort_scan(B, n_req);
            }
            if (!ok) {
                if (threadIdx.x == 0) inst_status[inst] = INST_PENDING;
                continue;
            }
            // the clients' bits are the top bits of the bucket number: a queue starts where its first bucket does
            for (int c = threadIdx.x; c <= n_clients; c += SORT_THREADS)
                qo[c] = c < n_clients ? (int32_t)bucket_sort_start(B, (uint32_t)c << (B.bbits - cbits)) : n_req;
            __syncthreads();
            for_each_request(pi, oi, ei, ai, n_req, [&](int i, uint32_t pp, uint32_t, uint32_t oe, int c) {
                bucket_sort_place(B, sort_key(i, pp, oe, c), (uint32_t)i, ride ? pp : 0u);
            });
            __syncthreads();
            for (int s = threadIdx.x; s < n_req; s += SORT_THREADS) {
                uint32_t k, id, extra;
                const uint32_t r = bucket_sort_rank(B, s, k, id, extra);
                if (!HOS_IN(r, n_req, 301) || !HOS_IN(id, n_req, 302)) continue;
                const uint32_t pp = ride ? extra : pi[id];
                const uint32_t totk = by_len ? kmask - (k & kmask) : 0u;     // p + (estimated) o, when it is the key
                qr[r] = id;
                qp[r] = make_uint2(pp, o_from_key ? totk - pp : oi[id]);
                if (qk) qk[r] = (by_len && kb < 32) ? totk : pp + ei[id];
            }
        } else {
            const int nbits = kb + cbits;
            const bool ride = nbits + bit_width_u32((uint32_t)mxp) <= 32;
            const bool o_from_key = ride && kb > 0 && kb < 32 && !o_est;
            for (int i = threadIdx.x; i < n_req; i += SORT_THREADS) {
                const uint32_t c = (uint32_t)park[i];
                const uint32_t low = (kb >= 32 ? 0u : (c << kb)) | (kmask - (key[i] & kmask));
                key[i] = ride ? (low | (nbits >= 32 ? 0u : (pi[i] << nbits))) : low;
            }
            __syncthreads();
            SortSmem<uint16_t> ss = sort_smem_carve<uint16_t>(smem_raw, n_req);
            const uint16_t* sorted = block_radix_sort_ids<uint16_t>(ss, n_req, nbits, 0u);
            for (int r = threadIdx.x; r < n_req; r += SORT_THREADS) {
                const uint32_t id = sorted[r];
                const uint32_t kw = key[id];
                const uint32_t low = (ride && nbits < 32) ? (kw & ((1u << nbits) - 1u)) : kw;
                const uint32_t pp = (ride && nbits < 32) ? kw >> nbits : pi[id];
                const uint32_t totk = kmask - (low & kmask);             // p + (estimated) o, when it is the key
                qr[r] = id;
                qp[r] = make_uint2(pp, o_from_key ? totk - pp : oi[id]);
                if (qk) qk[r] = kb > 0 && kb < 32 ? totk : pp + ei[id];
                const int c = kb >= 32 ? 0 : (int)(low >> kb);            // 32 key bits leave none for the client: one client
                const uint32_t kprev = r > 0 ? key[sorted[r - 1]] : 0u;
                const int cprev = r > 0 ? (kb >= 32 ? 0 : (int)(((ride && nbits < 32) ? (kprev & ((1u << nbits) - 1u)) : kprev) >> kb)) : -1;
                for (int cc = cprev + 1; cc <= c; ++cc) qo[cc] = r;
                if (r == n_req - 1)
                    for (int cc = c + 1; cc <= n_clients; ++cc) qo[cc] = n_req;
            }
        }
        if (threadIdx.x == 0) { inst_O[inst] = sumO; inst_status[inst] = st_done; }
    }
}

// ---------------------------------------------------------------------------------------
// Iteration-level simulator.  One THREAD per (instance, multiplier, client): the per-client
// recurrence (duration, clock, waited decode time, decision, hash) is scalar work, so every
// lane of a warp runs a client of its own.  The running batch of a client is a 4-ary
// min-heap in shared memory, keyed by the decode-iteration count at which a request retires
// (`fin`) with the request's p + o (`tot`) as payload, laid out [slot][lane] so that lanes
// never collide on a bank whatever slots they touch.  The KV length of a request at count c
// is tot - fin + c, so a decode iteration touches the heap only when someone retires, and
// sum KV is carried along: S += B - sum of retired tot.
// ---------------------------------------------------------------------------------------
constexpr uint32_t EMPTY = 0xFFFFFFFFu;
constexpr int TF_RING = 128;                // log entries in a warp's ring in k_trace_fill (a power of two)
constexpr int TF_AHEAD = 64;                // entries that the ring is filled ahead of their use, at least
// Event logs (what k_trace_fill rebuilds a trace from).  The plain simulator logs at most two
// events per request of the client's own queue, so client c of a simulation owns the entries
// [2 * q_off[c], 2 * q_off[c + 1]) of the simulation's log.  Under stealing a client's events
// are not bounded by its own queue, only their sum over the clients is (every request is
// admitted once and retired once): the clients take chunks of LOG_CHUNK entries from the
// simulation's log as they need them, and a directory lists every client's chunks in order.
constexpr uint32_t LOG_PER_QUEUE = 1u, LOG_CHUNKED = 2u;   // which form a workspace's log has
constexpr int LOG_CHUNK = 32;
constexpr int SIM_QUIET_MAX = 16;         // plain decode iterations per pass of the simulator's loop
constexpr unsigned long long HASH_INIT = 0xCBF29CE484222325ull;
constexpr uint32_t HASH_C1 = 0x9E3779B1u, HASH_C2 = 0x85EBCA77u, HASH_C3 = 0xC2B2AE3Du, HASH_M = 0x27D4EB2Fu;
// Clients are spread over more warps (fewer than 32 per warp) only while an SM gets at most this
// many warps, two per scheduler: spreading pays as long as schedulers would otherwise sit empty
// (800 clients: 0.54 ms as 25 full warps, 0.25 ms one client per warp), not beyond (18,944
// clients: 1.03 ms as 4 full warps per SM, 1.07 ms as 16 warps of 8; 65,536 clients: 1.48 ms
// as 14 full warps per SM, 1.74 ms as 28 warps of 16).
constexpr int SIM_SPREAD_WARPS_PER_SM = 8;

// Heap entries.  Narrow: (fin mod 2^16) << 16 | tot, usable when every p + o of the instance is
// below 2^16 (then fin - cnt < 2^16 too, and entries compare correctly after subtracting
// cnt << 16).  Wide: fin << 32 | tot.  Half the shared memory per client doubles the resident
// warps, and the recurrence is latency-bound.
struct NarrowEntry {
    typedef uint32_t T;
    static __device__ __forceinline__ T make(uint32_t fin, uint32_t tot) { return (fin << 16) | tot; }
    static __device__ __forceinline__ T rel(T x, uint32_t cnt) { return x - (cnt << 16); }
    static __device__ __forceinline__ uint32_t tot(T x) { return x & 0xFFFFu; }
    static __device__ __forceinline__ uint32_t fin(T x, uint32_t cnt) { return cnt + (rel(x, cnt) >> 16); }
    static __device__ __forceinline__ T rebase(T staged, uint32_t cnt) { return staged + (cnt << 16); }
};
struct WideEntry {
    typedef unsigned long long T;
    static __device__ __forceinline__ T make(uint32_t fin, uint32_t tot) { return ((T)fin << 32) | tot; }
    static __device__ __forceinline__ T rel(T x, uint32_t) { return x; }
    static __device__ __forceinline__ uint32_t tot(T x) { return (uint32_t)x; }
    static __device__ __forceinline__ uint32_t fin(T x, uint32_t) { return (uint32_t)(x >> 32); }
    static __device__ __forceinline__ T rebase(T staged, uint32_t cnt) { return staged + ((T)cnt << 32); }
};

template <typename E, bool FULL_WARP>
__global__ void __launch_bounds__(1024)
k_simulate(const uint2* __restrict__ q_po, const int32_t* __restrict__ q_off,
           const int32_t* __restrict__ inst_status, const uint32_t* __restrict__ lambda_q16,
           int n_lambda, int n_clients, int n_pad, long long n_units, int lanes, int cap, uint32_t kv_budget,
           hos_cost_model cm, int q_shift, uint32_t max_iters,
           hos_client_result* __restrict__ cres,
           hos_iter_rec* __restrict__ trace, const long long* __restrict__ trace_off,
           int32_t* __restrict__ status_out, uint4* __restrict__ events, long long ev_stride,
           uint32_t* __restrict__ event_count, uint32_t* __restrict__ log_kind) {
    typedef typename E::T entry_t;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (log_kind && blockIdx.x == 0 && threadIdx.x == 0) *log_kind = LOG_PER_QUEUE;
    // warps of a CTA are independent; each has its own block of cap * lanes heap entries.  Only the
    // first `lanes` lanes of a warp simulate a client: with fewer clients per warp the lanes wait
    // less for each other's events, and a small batch spreads over more SMs.
    // (FULL_WARP: lanes == 32 as a compile-time stride)
    const int stride = FULL_WARP ? 32 : lanes;
    entry_t* heap = reinterpret_cast<entry_t*>(smem_raw) + (size_t)warp_id() * cap * stride + lane_id();
    auto heap_ld = [&](int sl) -> entry_t { return HOS_IN(sl, cap, 311) ? heap[sl * stride] : (entry_t)0; };
    auto heap_st = [&](int sl, entry_t v) { if (HOS_IN(sl, cap, 311)) heap[sl * stride] = v; };
    const long long unit = ((long long)blockIdx.x * (blockDim.x >> 5) + warp_id()) * stride + lane_id();
    const bool in_range = lane_id() < stride && unit < n_units;
    const int c = in_range ? (int)(unit % n_clients) : 0;
    const int l = in_range ? (int)((unit / n_clients) % n_lambda) : 0;
    const int inst = in_range ? (int)(unit / ((long long)n_clients * n_lambda)) : 0;

    const int ist = inst_status[inst];
    const bool mine = in_range && ((ist & INST_WIDE) != 0) == (sizeof(entry_t) == 8);   // else: the other instantiation's
    // the lanes of this warp that simulate a client: they meet at the end of every pass of the loop
    unsigned live = __ballot_sync(FULL, mine && !(ist & HOS_ST_INVALID));
    if (!mine) return;
    if (ist & HOS_ST_INVALID) {
        cres[unit] = hos_client_result{0, 0, 0u, 0u, 0ull, 0.0};
        status_out[unit] = HOS_ST_INVALID;
        if (event_count) event_count[unit] = 0;
        return;
    }
    const int q0 = q_off[(size_t)inst * (n_clients + 1) + c];
    const int qn = q_off[(size_t)inst * (n_clients + 1) + c + 1] - q0;
    const uint2* q = q_po + (size_t)inst * n_pad + q0;
    const uint32_t lam = lambda_q16[l];
    const uint32_t stage_cap = stage_cap_tokens(cm);
    const uint32_t ad = cm.decode_fixed_us, bd = cm.decode_per_seq_us, qd = cm.decode_kv_div;

    long long t = 0, busy = 0;
    uint32_t Cd = 0, cnt = 0, B = 0, S = 0, reserved = 0, n_pre = 0;   // iterations = n_pre + cnt
    uint32_t next_fin = EMPTY;
    int head = 0;
    unsigned long long hash = HASH_INIT;
    uint32_t nA = 0, sumP = 0, sumTot = 0;
    bool grow = true;                        // the candidate prefix may extend
    int32_t status = 0;

    uint4* tr = nullptr;
    uint32_t tr_lim = 0;                     // records that fit the caller's slots
    if (trace) {
        const long long t0 = trace_off[unit];
        const long long capr = trace_off[unit + 1] - t0;
        tr = reinterpret_cast<uint4*>(trace + t0);
        tr_lim = capr > 0x7FFFFFFFll ? 0x7FFFFFFFu : (uint32_t)(capr < 0 ? 0 : capr);
    }
    // event log of this client: one 16-byte entry per logged iteration, at most 2 per request
    uint4* ev = events ? events + (size_t)(inst * n_lambda + l) * ev_stride + (size_t)q0 * 2 : nullptr;
    uint32_t n_ev = 0;
    uint2 nxt = make_uint2(0u, 0u);          // queue entries head + nA and head + nA + 1,
    uint2 nxt2 = make_uint2(0u, 0u);         // fetched ahead of their use
    if (qn > 0) nxt = __ldg(&q[0]);
    if (qn > 1) nxt2 = __ldg(&q[1]);

    // one iteration's bookkeeping: clock, hash, trace
    auto emit = [&](uint32_t dur, uint32_t r1, uint32_t r2, uint32_t r3) {
        const uint32_t it = n_pre + cnt;                 // index of this record (cnt not yet bumped)
        t += dur;
        hash = (hash + dur + (unsigned long long)HASH_C1 * r1 + (unsigned long long)HASH_C2 * r2 +
                (unsigned long long)HASH_C3 * r3) * HASH_M;
        if (it < tr_lim) tr[it] = make_uint4(dur, r1, r2, r3);
    };

    // One decode iteration (one token for every running request), popping every request that
    // retires with it.  Returns the number retired; leaves duration and batch figures in dur, r1, r2.
    // The heap is 4-ary: half the depth of a binary heap, and the four children of a node are
    // independent loads.
    uint32_t dur, r1, r2, r3;
    auto decode_step = [&]() {
        dur = ad + bd * B + (q_shift >= 0 ? (S >> q_shift) : (S / qd));
        r1 = B; r2 = S;
        uint32_t gone_n = 0;
        busy += (long long)dur * B;
        S += B;
        if (cnt + 1 == next_fin) {
            const uint32_t c1 = cnt + 1;
            uint32_t n = B;
            do {                                      // pop every request that retires now
                const uint32_t gone = E::tot(heap_ld(0));
                S -= gone;
                reserved -= gone;
                ++gone_n;
                --n;
                const entry_t x = heap_ld((int)n);
                const entry_t xr = E::rel(x, c1);
                uint32_t i = 0;
                while (true) {
                    const uint32_t ch = 4 * i + 1;
                    if (ch >= n) break;
                    // children beyond the heap's end compare as +infinity
                    entry_t y0 = heap_ld((int)ch), ym = y0;
                    entry_t m = E::rel(y0, c1);
                    uint32_t at = ch;
#pragma unroll
                    for (uint32_t k = 1; k < 4; ++k) {
                        if (ch + k < n) {
                            const entry_t y = heap_ld((int)(ch + k));
                            const entry_t r = E::rel(y, c1);
                            if (r < m) { m = r; ym = y; at = ch + k; }
                        }
                    }
                    if (xr <= m) break;
                    heap_st((int)i, ym);
                    i = at;
                }
                if (n > 0) heap_st((int)i, x);
            } while (n > 0 && E::fin(heap_ld(0), c1) == c1);
            B = n;
            next_fin = n > 0 ? E::fin(heap_ld(0), c1) : EMPTY;
            grow = head + (int)nA < qn;
        }
        r3 = gone_n;
    };
    // Bookkeeping of an event iteration (dur, r1, r2, r3): event log, clock, hash, trace, waited
    // decode time.  False when the clock limit is reached.
    auto finish_event = [&]() {
        if (ev && ((r1 >> 31) || r3 != 0u)) {
            // Something changed: one 16-byte log entry {iteration, tokens, sum KV after it, packed}.
            // A prefill packs flag | head << 16 | (batch after - 1) << 8 | (admitted - 1); a retiring
            // decode packs (retired - 1) << 8 | (batch before - 1).  Batches hold at most 256 requests
            // and queue positions stay below 2^15, durations follow from the tokens.
            const uint32_t packed = (r1 >> 31) ? (0x80000000u | (r3 << 16) | ((B - 1u) << 8) | ((r1 & 0x7FFFFFFFu) - 1u))
                                               : (((r3 - 1u) << 8) | (r1 - 1u));
            if (HOS_IN(n_ev, 2 * qn, 313)) ev[n_ev] = make_uint4(n_pre + cnt, r2, S, packed);
            ++n_ev;
        }
        emit(dur, r1, r2, r3);
        if (r1 >> 31) { Cd = 0; ++n_pre; }
        else { ++cnt; Cd = min(Cd + dur, 0x7FFFFFFFu); }  // both below 2^31: no wrap
        if (t >= (1ll << 39)) { status |= HOS_ST_LIMIT; return false; }
        return true;
    };

    // The event part of a pass: a decode iteration that retires requests, if that is what comes
    // next (the usual way a quiet run ends), then one general "event" iteration (a prefill, or any
    // decode).  The first only does what the second would do with that iteration.  Returns 0 when
    // a quiet run may follow, 1 when the next pass must start with an event again, 2 when the client
    // is done or has hit a limit.
    auto event_part = [&]() -> int {
        if (!grow && B > 0 && cnt + 1 == next_fin && n_pre + cnt != max_iters) {
            // the candidate prefix is current (grow is false), so the decision can be taken here
            const unsigned long long Cp16f = (unsigned long long)prefill_us(cm, sumP) << 16;
            if (nA == 0 || (unsigned long long)lam * Cd <= Cp16f) {
                decode_step();
                if (!finish_event()) return 2;
            }
        }
        if (grow) {
            // candidates: the longest queue prefix that fits the free slots and the KV budget.
            // A retirement only loosens both limits, so the prefix found earlier stays valid.
            // Candidate j waits at heap slot cap-1-j as (o, p+o); B + nA <= cap keeps it clear of
            // the heap itself.
            while (head + (int)nA < qn && B + nA < (uint32_t)cap) {
                const uint32_t tt = nxt.x + nxt.y;
                if (reserved + sumTot + tt > kv_budget) break;   // each term < 2^31 and reserved + sumTot <= budget: no wrap
                if (sumP + nxt.x > stage_cap) break;             // the largest prefill level is full
                heap_st(cap - 1 - (int)nA, E::make(nxt.y, tt));
                sumTot += tt; sumP += nxt.x; ++nA;
                nxt = nxt2;
                if (head + (int)nA + 1 < qn && HOS_IN(q0 + head + (int)nA + 1, n_pad, 312)) nxt2 = __ldg(&q[head + nA + 1]);
            }
            grow = false;
        }
        if (B == 0 && nA == 0) return 2;                 // queue empty and nothing running
        if (n_pre + cnt == max_iters) { status |= HOS_ST_LIMIT; return 2; }

        const uint32_t Cp = prefill_us(cm, sumP);
        const unsigned long long Cp16 = (unsigned long long)Cp << 16;
        const bool want_prefill = nA > 0 && (B == 0 || (unsigned long long)lam * Cd > Cp16);
        // plain decodes (nobody retires, the rule says decode) are the quiet run's business
        if (!want_prefill && cnt + 1 != next_fin) return 0;
        if (want_prefill) {
            // prefill: push the candidates, last staged first (its slot is the lowest, so the
            // growing heap never reaches a candidate that is still waiting)
            for (uint32_t j = 0; j < nA; ++j) {
                const entry_t x = E::rebase(heap_ld(cap - (int)nA + (int)j), cnt);
                const entry_t xr = E::rel(x, cnt);
                uint32_t i = B + j;
                while (i > 0) {
                    const uint32_t par = (i - 1) >> 2;
                    const entry_t y = heap_ld((int)par);
                    if (E::rel(y, cnt) <= xr) break;
                    heap_st((int)i, y);
                    i = par;
                }
                heap_st((int)i, x);
            }
            dur = Cp; r1 = 0x80000000u | nA; r2 = sumP; r3 = (uint32_t)head;
            busy += (long long)Cp * nA;
            S += sumP; B += nA; reserved += sumTot; head += (int)nA;
            nA = 0; sumP = 0; sumTot = 0;
            // slots and KV budget are as full as before, but a stage that stopped at the largest
            // prefill level's capacity has room again
            grow = stage_cap != 0xFFFFFFFFu && head < qn;
            next_fin = E::fin(heap_ld(0), cnt);
        } else {
            decode_step();
        }
        if (!finish_event()) return 2;
        return (grow || B == 0) ? 1 : 0;
    };

    // Every pass of this loop is the event part, then a quiet run of decode iterations in which
    // nobody retires and the decision cannot change.  In steady state a client goes retire ->
    // prefill -> quiet run, so a pass is a whole cycle and the lanes of a warp, which meet again at
    // every pass, spend it in the same code.  A quiet run is cut after SIM_QUIET_MAX iterations, so
    // that the warp does not wait for its longest run; a client whose run was cut skips the event
    // part of the next pass and goes on with its run.
    bool cut = false;                                    // my quiet run was cut and goes on
    while (true) {
        int act = 0;
        if (!cut) act = event_part();
        bool done = act == 2;
        if (act == 0) {
            // quiet run: at most `room` iterations -- up to the next retirement, the iteration limit,
            // and so few that only the last of them can take the clock past its limit (every
            // iteration adds less than 2^31) -- and only while the rule keeps saying "decode"
            const unsigned long long Cp16 = (unsigned long long)prefill_us(cm, sumP) << 16;
            const uint32_t room_t = (uint32_t)(((1ll << 39) - 1 - t) >> 31) + 1u;
            uint32_t room = min(min(next_fin - cnt - 1u, max_iters - (n_pre + cnt)), room_t);
            const bool capped = room > (uint32_t)SIM_QUIET_MAX;
            if (capped) room = SIM_QUIET_MAX;
            const uint32_t lam_run = nA > 0 ? lam : 0u;  // no candidates: nothing to prefill
            const uint32_t base = ad + bd * B;
            const long long t_run = t;
            while (room > 0 && (unsigned long long)lam_run * Cd <= Cp16) {
                const uint32_t dq = base + (q_shift >= 0 ? (S >> q_shift) : (S / qd));
                emit(dq, B, S, 0u);
                ++cnt;
                S += B;
                Cd = min(Cd + dq, 0x7FFFFFFFu);
                --room;
            }
            busy += (t - t_run) * (long long)B;
            if (t >= (1ll << 39)) { status |= HOS_ST_LIMIT; done = true; }
            cut = capped && room == 0 && (unsigned long long)lam_run * Cd <= Cp16;   // the cap ended it, not the rule
        }
        // every lane still simulating arrives here once per pass: the warp starts the next pass together
        live = __ballot_sync(live, !done);
        if (done) break;
    }
    if (tr && n_pre + cnt > tr_lim) status |= HOS_ST_TRACE;
    const uint32_t n_dec = cnt;
    cres[unit] = hos_client_result{t, busy, n_pre, n_dec, hash, 0.0};
    status_out[unit] = status;
    if (event_count) event_count[unit] = n_ev;
}

// ---------------------------------------------------------------------------------------
// Simulation with Algorithm 1's request stealing.  One CTA per (instance, multiplier), one
// thread per client.  Clients advance in global time order (earliest clock first, ties to the
// lower client); a client whose own queue is used up and that still has a free slot takes the
// longest waiting request of the client with the most queued tokens.
//
// Only a stealing client touches other clients' queues, so iterations that provably start
// before any steal can happen run side by side, one thread each; the client at the front of
// the global order takes its turn alone when it might steal (see the horizon H below).
// Iterations that claim nothing commute with everything: plain decodes follow their event
// iteration at once, and a client without a free slot goes on without waiting for its turn.
// ---------------------------------------------------------------------------------------
template <typename E>
__global__ void __launch_bounds__(MAX_CLIENTS)
k_simulate_steal(const uint2* __restrict__ q_po, const uint32_t* __restrict__ q_key,
                 const uint32_t* __restrict__ q_req,
                 const int32_t* __restrict__ q_off, const int32_t* __restrict__ inst_status,
                 const uint32_t* __restrict__ lambda_q16, int n_lambda, int n_clients, int n_req,
                 int n_pad, int cap, uint32_t kv_budget, hos_cost_model cm, int q_shift,
                 uint32_t max_iters, hos_client_result* __restrict__ cres,
                 hos_iter_rec* __restrict__ trace, const long long* __restrict__ trace_off,
                 int32_t* __restrict__ status_out, int32_t* __restrict__ served_by,
                 uint4* __restrict__ events, long long ev_stride, int pool_chunks,
                 uint32_t* __restrict__ chunk_tag, uint32_t* __restrict__ chunk_dir,
                 uint32_t* __restrict__ dir_start, uint32_t* __restrict__ event_count,
                 uint32_t* __restrict__ log_kind) {
    typedef typename E::T entry_t;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ unsigned s_chunks;                         // chunks of the event log handed out so far
    __shared__ uint32_t s_dstart[MAX_CLIENTS];            // first directory entry of each client
    __shared__ uint32_t s_wchunks[MAX_CLIENTS / 32];
    __shared__ int s_ustart[MAX_CLIENTS];                 // first unclaimed position of each queue
    __shared__ unsigned long long s_remain[MAX_CLIENTS];  // p+o still unclaimed in each queue
    __shared__ unsigned long long s_total;                // sum of s_remain
    __shared__ unsigned long long s_horizon;              // earliest possible steal (conservative bound)
    __shared__ unsigned long long s_first;                // earliest possible steal (from the dry run)
    __shared__ unsigned long long s_front;                // earliest unfinished client
    const int sim = blockIdx.x;
    const int inst = sim / n_lambda, l = sim % n_lambda;
    const int c = threadIdx.x;
    const int stride = blockDim.x;
    const long long unit = (long long)sim * n_clients + c;
    const bool is_client = c < n_clients;
    entry_t* heap = reinterpret_cast<entry_t*>(smem_raw) + c;
    auto heap_ld = [&](int sl) -> entry_t { return HOS_IN(sl, cap, 321) ? heap[sl * stride] : (entry_t)0; };
    auto heap_st = [&](int sl, entry_t v) { if (HOS_IN(sl, cap, 321)) heap[sl * stride] = v; };

    const int ist = inst_status[inst];
    if (log_kind && blockIdx.x == 0 && threadIdx.x == 0) *log_kind = LOG_CHUNKED;
    if (((ist & INST_WIDE) != 0) != (sizeof(entry_t) == 8)) return;   // the other instantiation's instance
    if (ist & HOS_ST_INVALID) {
        if (is_client) {
            cres[unit] = hos_client_result{0, 0, 0u, 0u, 0ull, 0.0};
            status_out[unit] = HOS_ST_INVALID;
            if (events) { event_count[unit] = 0; dir_start[unit] = 0; }
        }
        if (served_by)
            for (int i = c; i < n_req; i += stride) served_by[(size_t)sim * n_req + i] = -1;
        return;
    }
    const int32_t* qo = q_off + (size_t)inst * (n_clients + 1);
    const uint2* q = q_po + (size_t)inst * n_pad;          // all queues of the instance, CSR by client
    // queued tokens as the scheduler counts them: p + estimated o when the lengths are estimated
    const uint32_t* qk = q_key ? q_key + (size_t)inst * n_pad : nullptr;
    const uint32_t* qr = q_req + (size_t)inst * n_pad;
    int32_t* served = served_by ? served_by + (size_t)sim * n_req : nullptr;
    const int qend = is_client ? qo[c + 1] : 0;
    const uint32_t lam = lambda_q16[l];
    const uint32_t stage_cap = stage_cap_tokens(cm);
    const uint32_t ad = cm.decode_fixed_us, bd = cm.decode_per_seq_us, qd = cm.decode_kv_div;

    if (is_client) {
        unsigned long long r = 0;
        for (int x = qo[c]; x < qend; ++x) {
            const uint2 po = q[x];
            r += qk ? (unsigned long long)qk[x] : (unsigned long long)po.x + po.y;
        }
        s_ustart[c] = qo[c];
        s_remain[c] = r;
    }
    if (c == 0) { s_total = 0; s_horizon = ~0ull; s_first = ~0ull; s_front = ~0ull; s_chunks = 0u; }
    if (served)                                           // requests nobody gets to (iteration limit)
        for (int i = c; i < n_req; i += stride) served[i] = -1;
    __syncthreads();
    if (is_client) atomicAdd(&s_total, s_remain[c]);

    long long t = 0, busy = 0;
    uint32_t Cd = 0, cnt = 0, B = 0, S = 0, reserved = 0, n_pre = 0;
    uint32_t next_fin = EMPTY, nA = 0, sumP = 0, sumTot = 0, head = 0;
    unsigned long long hash = HASH_INIT;
    int32_t status = 0;
    bool finished = !is_client;
    uint4* tr = nullptr;
    uint32_t tr_lim = 0;
    if (trace && is_client) {
        const long long t0 = trace_off[unit];
        const long long capr = trace_off[unit + 1] - t0;
        tr = reinterpret_cast<uint4*>(trace + t0);
        tr_lim = capr > 0x7FFFFFFFll ? 0x7FFFFFFFu : (uint32_t)(capr < 0 ? 0 : capr);
    }
    // event log: this simulation's pool of chunks, the chunk I am filling, my entries so far
    uint4* const ev_pool = events ? events + (size_t)sim * ev_stride : nullptr;
    uint32_t* const tag_sim = events ? chunk_tag + (size_t)sim * pool_chunks : nullptr;
    uint4* ev_chunk = nullptr;
    uint32_t n_ev = 0;
    bool log_on = false;                                  // not during the dry run
    auto emit = [&](uint32_t dur, uint32_t r1, uint32_t r2, uint32_t r3) {
        const uint32_t it = n_pre + cnt;
        t += dur;
        hash = (hash + dur + (unsigned long long)HASH_C1 * r1 + (unsigned long long)HASH_C2 * r2 +
                (unsigned long long)HASH_C3 * r3) * HASH_M;
        if (it < tr_lim) tr[it] = make_uint4(dur, r1, r2, r3);
    };
    // claim the request at position x of some queue as my next candidate, if it fits.  A dry run
    // keeps its hands off everything the clients share.
    auto claim = [&](int owner, int x, bool dry) -> bool {
        if (!HOS_IN(x, n_req, 322) || !HOS_IN(owner, n_clients, 324)) return false;
        const uint2 po = q[x];
        const uint32_t tt = po.x + po.y;
        if (reserved + sumTot + tt > kv_budget) return false;
        if (sumP + po.x > stage_cap) return false;          // the largest prefill level is full
        heap_st(cap - 1 - (int)nA, E::make(po.y, tt));
        sumTot += tt; sumP += po.x; ++nA;
        if (!dry) {
            const uint32_t tk = qk ? qk[x] : tt;
            s_ustart[owner] = x + 1;
            s_remain[owner] -= tk;
            atomicAdd(&s_total, 0ull - (unsigned long long)tk);
            if (served && HOS_IN(qr[x], n_req, 323)) served[qr[x]] = c;
        }
        return true;
    };
    int u_dry = is_client ? qo[c] : 0;                      // the dry run's own queue position

    // One event iteration of my client -- claims (and, when `may_steal`, requests taken from other
    // queues), the decision, the prefill or decode -- and the plain decodes that follow it while
    // nothing can be claimed.  Sets `finished` when the client is done or hits a limit.
    // One decode iteration (one token for every running request), popping every request that
    // retires with it; leaves the record in dur, r1, r2, r3.
    uint32_t dur, r1, r2, r3;
    auto decode_step = [&]() {
        dur = ad + bd * B + (q_shift >= 0 ? (S >> q_shift) : (S / qd));
        r1 = B; r2 = S; r3 = 0;
        busy += (long long)dur * B;
        S += B;
        if (cnt + 1 == next_fin) {
            const uint32_t c1 = cnt + 1;
            uint32_t n = B;
            do {
                const uint32_t gone = E::tot(heap_ld(0));
                S -= gone;
                reserved -= gone;
                ++r3;
                --n;
                const entry_t x = heap_ld((int)n);
                const entry_t xr = E::rel(x, c1);
                uint32_t i = 0;
                while (true) {
                    const uint32_t ch = 4 * i + 1;
                    if (ch >= n) break;
                    entry_t y0 = heap_ld((int)ch), ym = y0;
                    entry_t m = E::rel(y0, c1);
                    uint32_t at = ch;
#pragma unroll
                    for (uint32_t k = 1; k < 4; ++k) {
                        if (ch + k < n) {
                            const entry_t y = heap_ld((int)(ch + k));
                            const entry_t r = E::rel(y, c1);
                            if (r < m) { m = r; ym = y; at = ch + k; }
                        }
                    }
                    if (xr <= m) break;
                    heap_st((int)i, ym);
                    i = at;
                }
                if (n > 0) heap_st((int)i, x);
            } while (n > 0 && E::fin(heap_ld(0), c1) == c1);
            B = n;
            next_fin = n > 0 ? E::fin(heap_ld(0), c1) : EMPTY;
        }
    };
    // Clock, hash, trace and waited decode time of the iteration in dur, r1, r2, r3; false when the
    // clock limit is reached.
    auto finish_event = [&]() {
        if (log_on && ((r1 >> 31) || r3 != 0u)) {
            // Something changed: a log entry as in k_simulate, {iteration, tokens, sum KV after it,
            // packed}.  Every prefill admits a request and every logged decode retires one, so all
            // the clients' entries together are at most two per request of the instance, and the
            // chunks they start at most that / LOG_CHUNK + one per client: the pool's size.
            if ((n_ev & (LOG_CHUNK - 1)) == 0u) {
                const unsigned ch = atomicAdd(&s_chunks, 1u);
                ev_chunk = nullptr;
                if (HOS_IN(ch, pool_chunks, 325) && ch < (unsigned)pool_chunks) {
                    tag_sim[ch] = ((uint32_t)c << 16) | (n_ev / LOG_CHUNK);
                    ev_chunk = ev_pool + (size_t)ch * LOG_CHUNK;
                }
            }
            const uint32_t packed = (r1 >> 31) ? (0x80000000u | (r3 << 16) | ((B - 1u) << 8) | ((r1 & 0x7FFFFFFFu) - 1u))
                                               : (((r3 - 1u) << 8) | (r1 - 1u));
            if (ev_chunk) ev_chunk[n_ev & (LOG_CHUNK - 1)] = make_uint4(n_pre + cnt, r2, S, packed);
            ++n_ev;
        }
        emit(dur, r1, r2, r3);
        if (r1 >> 31) { Cd = 0; ++n_pre; }
        else { ++cnt; Cd = min(Cd + dur, 0x7FFFFFFFu); }
        if (t >= (1ll << 39)) { status |= HOS_ST_LIMIT; finished = true; return false; }
        return true;
    };
    // `until`: while the client runs side by side with the others (or alone in the dry run), an
    // advance may start with the retiring decode that ends a quiet run and go on to the next event,
    // as long as that one still starts before `until`; 0 when the client runs in its turn of the
    // global order, where every event has to wait for its turn.
    auto advance = [&](bool dry, unsigned long long until) {
        if (until != 0ull && B > 0 && cnt + 1 == next_fin && n_pre + cnt != max_iters) {
            // nothing can be claimed now (no free slot, or the own queue is used up and nothing is
            // left anywhere), so the candidates stay as they are and the rule decides on them
            const int up0 = dry ? u_dry : s_ustart[c];
            const bool no_claim = B + nA >= (uint32_t)cap || (up0 >= qend && (dry || s_total == 0));
            const unsigned long long Cp16f = (unsigned long long)prefill_us(cm, sumP) << 16;
            if (no_claim && (nA == 0 || (unsigned long long)lam * Cd <= Cp16f)) {
                decode_step();
                if (!finish_event()) return;
                // the next event must still be mine to take: before the horizon, and (dry run) before
                // the iteration in which the own queue could be used up
                if ((((unsigned long long)t << 9) | (unsigned)c) >= until) return;
                if (dry && (uint32_t)(qend - u_dry) <= (uint32_t)cap - B - nA) return;
            }
        }
        int up = dry ? u_dry : s_ustart[c];
        while (up < qend && B + nA < (uint32_t)cap) {
            if (!claim(c, up, dry)) break;
            ++up;
        }
        if (dry) u_dry = up;
        if (!dry && up == qend) {
            while (B + nA < (uint32_t)cap && s_total > 0) {    // only reached when running alone
                int d = -1;
                unsigned long long best = 0;
                for (int j = 0; j < n_clients; ++j)
                    if (s_remain[j] > best) { best = s_remain[j]; d = j; }
                if (d < 0 || !claim(d, s_ustart[d], false)) break;
            }
        }
        if (B == 0 && nA == 0) { finished = true; return; }
        if (n_pre + cnt == max_iters) { status |= HOS_ST_LIMIT; finished = true; return; }

        const uint32_t Cp = prefill_us(cm, sumP);
        const unsigned long long Cp16 = (unsigned long long)Cp << 16;
        if (nA > 0 && (B == 0 || (unsigned long long)lam * Cd > Cp16)) {
            for (uint32_t j = 0; j < nA; ++j) {
                const entry_t x = E::rebase(heap_ld(cap - (int)nA + (int)j), cnt);
                const entry_t xr = E::rel(x, cnt);
                uint32_t i = B + j;
                while (i > 0) {
                    const uint32_t par = (i - 1) >> 2;
                    const entry_t y = heap_ld((int)par);
                    if (E::rel(y, cnt) <= xr) break;
                    heap_st((int)i, y);
                    i = par;
                }
                heap_st((int)i, x);
            }
            dur = Cp; r1 = 0x80000000u | nA; r2 = sumP; r3 = head;
            busy += (long long)Cp * nA;
            S += sumP; B += nA; reserved += sumTot; head += nA;
            nA = 0; sumP = 0; sumTot = 0;
            next_fin = E::fin(heap_ld(0), cnt);
        } else {
            decode_step();
        }
        if (!finish_event()) return;
        // plain decodes may follow at once while nothing can be claimed: they touch no queue, so
        // their order against other clients' claims does not matter.  Nothing can be claimed when no
        // slot is free, or when the own queue is used up and no queue has anything left (s_total
        // only ever falls, so a zero read here is final).
        if (B == 0) return;
        if (B + nA < (uint32_t)cap && ((dry ? u_dry : s_ustart[c]) < qend || s_total > 0)) return;
        const uint32_t room_t = (uint32_t)(((1ll << 39) - 1 - t) >> 31) + 1u;
        uint32_t room = min(min(next_fin - cnt - 1u, max_iters - (n_pre + cnt)), room_t);
        const uint32_t lam_run = nA > 0 ? lam : 0u;
        const uint32_t base = ad + bd * B;
        const long long t_run = t;
        while (room > 0 && (unsigned long long)lam_run * Cd <= Cp16) {
            const uint32_t dq = base + (q_shift >= 0 ? (S >> q_shift) : (S / qd));
            emit(dq, B, S, 0u);
            ++cnt;
            S += B;
            Cd = min(Cd + dq, 0x7FFFFFFFu);
            --room;
        }
        busy += (t - t_run) * (long long)B;
        if (t >= (1ll << 39)) { status |= HOS_ST_LIMIT; finished = true; }
    };

    // Dry run: every client alone, until the iteration in which it could use up its own queue
    // (unclaimed requests <= free slots).  As long as nothing has been stolen the real run is these
    // independent runs, so nothing can be stolen before the earliest such iteration, s_first.
    {
        const uint32_t keep_lim = tr_lim;
        tr_lim = 0;                                         // no trace from the dry run
        while (!finished && (uint32_t)(qend - u_dry) > (uint32_t)cap - B - nA) advance(true, ~0ull);
        if (is_client) atomicMin(&s_first, ((unsigned long long)t << 9) | (unsigned)c);
        tr_lim = keep_lim;
        t = 0; busy = 0; Cd = 0; cnt = 0; B = 0; S = 0; reserved = 0; n_pre = 0;
        next_fin = EMPTY; nA = 0; sumP = 0; sumTot = 0; head = 0;
        hash = HASH_INIT; status = 0; finished = !is_client;
        log_on = events != nullptr;
    }

    // After s_first the conservative bound: no iteration lasts less than d_min and a client claims
    // at most `cap` requests per iteration, so a client with u unclaimed own requests cannot use
    // them up -- and so cannot steal -- before es = clock + (ceil(u / cap) - 1) * d_min; with u at least
    // its free slots it cannot steal in its next iteration either, so es >= clock + d_min.  Nothing is
    // stolen before H = max(s_first, min es over the unfinished clients), hence every iteration that
    // starts before H only touches its own client and all of them may run side by side: a client
    // goes on, iteration after iteration, until its clock reaches H (the bound is taken from the
    // state at the start of the step and only gets more conservative as the clients claim their
    // own requests).  When none starts before H, the client at the front of the global order may
    // steal: it runs alone, one iteration.
    // shortest possible iteration: a prefill of one token, or a decode of one request
    const unsigned long long d_min = min((unsigned long long)prefill_us(cm, 1u), (unsigned long long)ad + bd);
    while (true) {
        __syncthreads();                                   // last step's queue updates are visible
        const unsigned long long key = ((unsigned long long)t << 9) | (unsigned)c;
        unsigned long long es_key = ~0ull;
        if (!finished && s_total > s_remain[c]) {          // somebody else still has queued requests
            const unsigned long long u = (unsigned long long)(qend - s_ustart[c]);
            unsigned long long k = u > (unsigned long long)cap ? (u + cap - 1) / cap - 1 : 0ull;
            // and not in its next iteration when its free slots do not outnumber its own requests
            // (it claims those first and steals only with a slot to spare)
            if (k == 0ull && u >= (unsigned long long)((uint32_t)cap - B - nA)) k = 1ull;
            es_key = (((unsigned long long)t + k * d_min) << 9) | (unsigned)c;
        }
        // minima per warp first: one shared-memory update per warp instead of one per client
        unsigned long long wh = es_key, wf = finished ? ~0ull : key;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const unsigned long long oh = __shfl_xor_sync(FULL, wh, d), of = __shfl_xor_sync(FULL, wf, d);
            wh = oh < wh ? oh : wh;
            wf = of < wf ? of : wf;
        }
        if ((c & 31) == 0) {
            if (wh != ~0ull) atomicMin(&s_horizon, wh);
            if (wf != ~0ull) atomicMin(&s_front, wf);
        }
        if (__syncthreads_and(finished)) break;
        const unsigned long long H = max(s_horizon, s_first);
        const unsigned long long front = s_front;
        bool run = !finished && key < H;
        const int ahead = __syncthreads_or(run);           // also orders the reads of the shared keys
        if (!ahead) run = !finished && key == front;       // the front of the global order: may steal
        if (c == 0) { s_horizon = ~0ull; s_front = ~0ull; } // for the next step (after the barrier above)
        if (run) {
            if (ahead) {
                do advance(false, H);
                while (!finished && (((unsigned long long)t << 9) | (unsigned)c) < H);
            } else advance(false, 0ull);
        } else if (!finished) {
            // A client without a free slot claims nothing in its next iteration, whatever that is
            // (a prefill of what it has claimed already, or a decode): the iteration touches no
            // queue and nobody looks at the state it changes, so it needs no turn in the global
            // order.  (What it reads of the queues on the way only decides whether plain decodes
            // may follow at once; a stale value there only postpones them.)
            while (!finished && B + nA == (uint32_t)cap) advance(false, 0ull);
        }
    }
    if (is_client) {
        if (tr && n_pre + cnt > tr_lim) status |= HOS_ST_TRACE;
        cres[unit] = hos_client_result{t, busy, n_pre, cnt, hash, 0.0};
        status_out[unit] = status;
    }
    if (events) {
        // The directory: every client's chunks in the order it filled them, the clients one after
        // the other.  (The loop above ends at a barrier, so every tag written is visible here.)
        const uint32_t mine = is_client ? (n_ev + LOG_CHUNK - 1) / LOG_CHUNK : 0u;
        uint32_t inc = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(FULL, inc, d);
            if (lane_id() >= d) inc += y;
        }
        if (lane_id() == 31) s_wchunks[warp_id()] = inc;
        __syncthreads();
        uint32_t before = 0;
        for (int w = 0; w < warp_id(); ++w) before += s_wchunks[w];
        s_dstart[c] = before + inc - mine;
        if (is_client) {
            event_count[unit] = n_ev;
            dir_start[unit] = before + inc - mine;
        }
        __syncthreads();
        const unsigned total = min(s_chunks, (unsigned)pool_chunks);
        uint32_t* const dir_sim = chunk_dir + (size_t)sim * pool_chunks;
        for (unsigned ch = c; ch < total; ch += stride) {
            const uint32_t tag = tag_sim[ch];
            const uint32_t owner = tag >> 16, seq = tag & 0xFFFFu;
            if (!HOS_IN(owner, n_clients, 326) || owner >= (uint32_t)n_clients) continue;
            const uint32_t at = s_dstart[owner] + seq;
            if (HOS_IN(at, pool_chunks, 327) && at < (uint32_t)pool_chunks) dir_sim[at] = ch;
        }
    }
}

// ---------------------------------------------------------------------------------------
// Trace from the event log.  One warp per (instance, multiplier, client); a lane per iteration.
// Iteration `it` belongs to the last logged iteration k with it_k <= it: it is that record
// itself, or the (it - it_k)-th plain decode after it, with the batch B logged there and
// sum KV = S_k + (it - it_k - 1) * B.  A chunk of 32 consecutive iterations can only reach the
// next 32 log entries, so one coalesced load of their iteration numbers and a bit mask place
// every lane.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
k_trace_fill(const int32_t* __restrict__ q_off, int n_lambda, int n_clients, int n_pad, long long n_units,
             hos_cost_model cm, int q_shift, const hos_client_result* __restrict__ cres,
             const uint4* __restrict__ events, long long ev_stride, const uint32_t* __restrict__ event_count,
             const uint32_t* __restrict__ log_kind, int pool_chunks, const uint32_t* __restrict__ chunk_dir,
             const uint32_t* __restrict__ dir_start,
             hos_iter_rec* __restrict__ trace, const long long* __restrict__ trace_off,
             int32_t* __restrict__ status_out) {
    const long long unit = (long long)blockIdx.x * 4 + warp_id();
    if (unit >= n_units) return;
    const int lane = lane_id();
    const int c = (int)(unit % n_clients);
    const int sim = (int)(unit / n_clients);
    const int inst = sim / n_lambda;
    const int q0 = q_off[(size_t)inst * (n_clients + 1) + c];
    // the client's log: its own stretch of the simulation's log, or (stealing simulator) chunks of
    // LOG_CHUNK entries listed in the directory
    const bool chunked = __ldg(log_kind) == LOG_CHUNKED;
    const uint4* ev = events + (size_t)sim * ev_stride + (chunked ? (size_t)0 : (size_t)q0 * 2);
    const uint32_t* dir = chunk_dir + (size_t)sim * pool_chunks;
    const uint32_t d0 = chunked ? dir_start[unit] : 0u;
    const uint32_t n_ev = event_count[unit];
    const uint32_t n_total = cres[unit].n_prefill_iters + cres[unit].n_decode_iters;
    const long long t0 = trace_off[unit];
    const long long capr = trace_off[unit + 1] - t0;
    uint4* tr = reinterpret_cast<uint4*>(trace + t0);
    const uint32_t lim = capr > (long long)n_total ? n_total : (uint32_t)(capr < 0 ? 0 : capr);
    if (lane == 0 && (long long)n_total > capr) atomicOr(&status_out[unit], HOS_ST_TRACE);
    const uint32_t ad = cm.decode_fixed_us, bd = cm.decode_per_seq_us, qd = cm.decode_kv_div;

    // The log entries pass through a ring in shared memory, filled by asynchronous copies that
    // run TF_AHEAD entries and more ahead of their use: a pass then waits for no load from the
    // log.  The ring holds the entries [k_next - 1, filled); one group of 32 is in flight at most
    // when a pass starts.
    __shared__ uint4 s_ring[4][TF_RING];
    uint4* ring = s_ring[warp_id()];
    uint32_t filled = 0;                       // log entries before `filled` are in the ring or on their way
    auto fill = [&]() {
        const uint32_t kf = filled + lane;
        uint4* dst = &ring[kf & (TF_RING - 1)];
        if (kf < n_ev) {
            const uint4* src = ev + kf;
            if (chunked) {
                // `filled` is a multiple of LOG_CHUNK = 32: the warp's 32 entries are one chunk
                const uint32_t at = d0 + filled / LOG_CHUNK;
                const uint32_t ch = HOS_IN(at, pool_chunks, 341) && at < (uint32_t)pool_chunks ? __ldg(&dir[at]) : 0u;
                src = HOS_IN(ch, pool_chunks, 342) && ch < (uint32_t)pool_chunks ? ev + (size_t)ch * LOG_CHUNK + lane : ev;
            }
            const unsigned sa = (unsigned)__cvta_generic_to_shared(dst);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(sa), "l"(src) : "memory");
        } else {
            *dst = make_uint4(0xFFFFFFFFu, 0u, 0u, 0u);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        filled += 32;
    };
    for (int g = 0; g < TF_AHEAD / 32 + 1; ++g) fill();

    uint32_t k_next = 0;                       // log entries before k_next have it < base
    for (uint32_t base = 0; base < lim; base += 32) {
        const uint32_t it = base + lane;
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        __syncwarp();
        // iteration numbers of the next 32 log entries
        const uint32_t itw = ring[(k_next + lane) & (TF_RING - 1)].x;       // 0xFFFFFFFF past the log's end
        const uint32_t dw = itw - base;                                  // >= 0 by construction
        const uint32_t mask = __reduce_or_sync(FULL, dw < 32u ? (1u << dw) : 0u);
        const uint32_t upto = mask & (0xFFFFFFFFu >> (31 - lane));       // logged iterations <= it
        const uint32_t k = k_next + __popc(upto) - 1u;                   // iteration 0 is always logged
        if (it < lim) {
            const uint4 st = ring[k & (TF_RING - 1)];  // {iteration, tokens, sum KV after it, packed}
            const bool pre = st.w >> 31;
            const bool logged = st.x == it;
            const uint32_t lo8 = (st.w & 0xFFu) + 1u, hi8 = ((st.w >> 8) & 0xFFu) + 1u;
            // a decode record either way -- the logged (retiring) one, or a plain one after the logged
            // iteration -- from one formula; only a logged prefill takes a branch
            const uint32_t Bk = logged ? lo8 : (pre ? hi8 : lo8 - hi8);  // batch of this iteration
            const uint32_t Sk = logged ? st.y : st.z + (it - st.x - 1u) * Bk;
            uint4 rec = make_uint4(ad + bd * Bk + (q_shift >= 0 ? (Sk >> q_shift) : (Sk / qd)), Bk, Sk,
                                   logged ? hi8 : 0u);
            if (logged && pre)
                rec = make_uint4(prefill_us(cm, st.y), 0x80000000u | lo8, st.y, (st.w >> 16) & 0x7FFFu);
            tr[it] = rec;
        }
        k_next += __popc(mask);
        __syncwarp();                           // every lane has read its entries before slots are refilled
        if (filled - k_next < (uint32_t)TF_AHEAD + 32u) fill();
        else asm volatile("cp.async.commit_group;" ::: "memory");        // keeps "all but the newest group" exact
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}


// ---------------------------------------------------------------------------------------
// Per-simulation figures: makespan = max over clients, busy = sum, utilisation = busy slot
// time over offered slot time, generation speed = output tokens per second of makespan.
// One warp per (instance, multiplier).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
k_finalize(int n_sims, int n_lambda, int n_clients, int cap,
           const unsigned long long* __restrict__ inst_O, hos_client_result* __restrict__ cres,
           hos_sim_result* __restrict__ sres) {
    const int sim = blockIdx.x * 4 + warp_id();
    if (sim >= n_sims) return;
    const int lane = lane_id();
    hos_client_result* cr = cres + (size_t)sim * n_clients;
    long long mk = 0;
    unsigned long long busy = 0;
    for (int j = lane; j < n_clients; j += 32) {
        mk = cr[j].makespan_us > mk ? cr[j].makespan_us : mk;
        busy += (unsigned long long)cr[j].busy_slot_us;
    }
    mk = warp_max_i64(mk);
    busy = warp_sum_u64(busy);
    const double dm = (double)mk;
    for (int j = lane; j < n_clients; j += 32)
        cr[j].utilisation = mk > 0 ? (double)cr[j].busy_slot_us / ((double)cap * dm) : 0.0;
    if (lane == 0) {
        hos_sim_result r;
        r.makespan_us = mk;
        r.busy_slot_us = (long long)busy;
        r.utilisation = mk > 0 ? (double)(long long)busy / (((double)n_clients * (double)cap) * dm) : 0.0;
        r.tokens_per_s = mk > 0 ? ((double)inst_O[sim / n_lambda] * 1.0e6) / dm : 0.0;
        sres[sim] = r;
    }
}

// Exclusive scan of the iteration counts.  Every CTA owns a slice of whole tiles of 1,024 units; it
// first adds up all counts before its slice (no CTA waits for another and no scratch memory is
// needed; the counts are a few MB in L2), then scans its slice tile by tile.
__global__ void __launch_bounds__(1024)
k_trace_offsets(const hos_client_result* __restrict__ cres, long long n_units, long long slice,
                long long* __restrict__ trace_off) {
    __shared__ unsigned long long wsum[2][32];
    __shared__ unsigned long long s_before;
    auto count = [&](long long x) {
        return x < n_units ? (unsigned long long)cres[x].n_prefill_iters + cres[x].n_decode_iters : 0ull;
    };
    const long long x0 = slice * blockIdx.x, x1 = min(n_units, x0 + slice);
    if (blockIdx.x == 0 && threadIdx.x == 0) trace_off[0] = 0;
    if (x0 >= n_units) return;                                            // the whole CTA: a slice past the end
    if (threadIdx.x == 0) s_before = 0;
    __syncthreads();
    {
        unsigned long long part = 0;
        long long x = threadIdx.x;
        for (; x + 7 * 1024 < x0; x += 8 * 1024) {
            unsigned long long v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = count(x + j * 1024);
#pragma unroll
            for (int j = 0; j < 8; ++j) part += v[j];
        }
        for (; x < x0; x += 1024) part += count(x);
        part = warp_sum_u64(part);
        if (lane_id() == 0 && part != 0) atomicAdd(&s_before, part);
    }
    __syncthreads();
    unsigned long long carry = s_before;                                  // units before this tile
    int buf = 0;
    for (long long base = x0; base < x1; base += 1024, buf ^= 1) {
        const long long x = base + threadIdx.x;
        const unsigned long long mine = count(x);
        unsigned long long inc = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long y = __shfl_up_sync(FULL, inc, d);
            if (lane_id() >= d) inc += y;
        }
        if (lane_id() == 31) wsum[buf][warp_id()] = inc;
        __syncthreads();
        // every warp scans the 32 warp sums itself: one barrier per tile (the two buffers keep a
        // fast warp's next tile away from the sums that a slow warp still reads)
        const unsigned long long w = wsum[buf][lane_id()];
        unsigned long long winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long y = __shfl_up_sync(FULL, winc, d);
            if (lane_id() >= d) winc += y;
        }
        const unsigned long long before = __shfl_sync(FULL, winc - w, warp_id());
        if (x < x1) trace_off[x + 1] = (long long)(carry + before + inc);
        carry += __shfl_sync(FULL, winc, 31);
    }
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------
// Slots and KV budget the simulators run with (see launch_simulate).
static int sim_slots(const hos_batch& b) {
    if (!b.kv_reserve_tokens) return b.batch_cap;
    const long long fit = b.kv_budget / (long long)b.kv_reserve_tokens;
    return (int)(fit < (long long)b.batch_cap ? fit : (long long)b.batch_cap);
}
static uint32_t sim_budget(const hos_batch& b) { return b.kv_reserve_tokens ? 0x7FFFFFFFu : (uint32_t)b.kv_budget; }

HOS_DEFINE_BOUNDS_READER(debug_bounds_online)

size_t queue_build_smem(int n_req) { return sort_smem_bytes<uint16_t>(n_req); }

cudaError_t launch_queue_build(const hos_batch& b, const int32_t* assign, uint32_t p_max, int queue_order, uint2* q_po,
                               uint32_t* q_key, uint32_t* q_req, int32_t* q_off, unsigned long long* inst_O,
                               int32_t* inst_status, int n_pad, cudaStream_t st) {
    cudaError_t e = allow_max_dynamic_smem(reinterpret_cast<const void*>(k_queue_build<true>));
    if (e != cudaSuccess) return e;
    if ((e = allow_max_dynamic_smem(reinterpret_cast<const void*>(k_queue_build<false>))) != cudaSuccess) return e;
    const long long most = b.kv_reserve_tokens ? (long long)b.kv_reserve_tokens : (long long)b.kv_budget;
    launch_hook("k_queue_build", 0, st);
    k_queue_build<true><<<b.n_inst, SORT_THREADS, bucket_sort_smem_bytes(b.n_req), st>>>(
        b.p, b.o, b.o_est, assign, b.n_inst, b.n_req, b.n_clients, most, p_max, queue_order, q_po,
        b.o_est ? q_key : nullptr, q_req, q_off, inst_O, inst_status, n_pad);
    launch_hook("k_queue_build", 1, st);
    int n_sm = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    launch_hook("k_queue_build_radix", 0, st);
    k_queue_build<false><<<b.n_inst < n_sm ? b.n_inst : n_sm, SORT_THREADS, queue_build_smem(b.n_req), st>>>(
        b.p, b.o, b.o_est, assign, b.n_inst, b.n_req, b.n_clients, most, p_max, queue_order, q_po,
        b.o_est ? q_key : nullptr, q_req, q_off, inst_O, inst_status, n_pad);
    launch_hook("k_queue_build_radix", 1, st);
    return cudaGetLastError();
}

cudaError_t launch_simulate(const hos_batch& b, const hos_cost_model& cm, const uint32_t* lambda_q16,
                            int n_lambda, uint32_t max_iters, const uint2* q_po, const int32_t* q_off,
                            const int32_t* inst_status, int n_pad, hos_client_result* cres,
                            hos_iter_rec* trace, const long long* trace_off, int32_t* status,
                            const EventLog& log, cudaStream_t st) {
    const long long n_units = (long long)b.n_inst * n_lambda * b.n_clients;
    // A fixed reservation of R tokens per request admits floor(budget / R) requests at most and
    // nothing else: the simulator runs with that many slots and no KV limit.
    const int cap = sim_slots(b);
    const uint32_t kv = sim_budget(b);
    int q_shift = -1;                                    // power-of-two KV divisor -> shift
    if ((cm.decode_kv_div & (cm.decode_kv_div - 1)) == 0)
        for (q_shift = 0; (1u << q_shift) != cm.decode_kv_div; ++q_shift) {}
    // Both instantiations are launched; each one runs the instances whose entries it can hold and
    // returns at once for the others (the flag is per instance, on the device).
    //
    // Launch shape.  The recurrence is latency-bound and shared memory (one heap per client) limits
    // what is resident, so what matters is that everything runs at once, on as many SMs as possible,
    // with as few clients per warp as that allows (the lanes of a warp wait for each other's events).
    // `lanes` clients per warp: the smallest power of two for which all warps are resident in one
    // wave and, below 32, an SM holds at most SIM_SPREAD_WARPS_PER_SM of them.  Every CTA
    // costs 1 KB of shared memory on top of its heaps; if not even 32 lanes make one wave, one-warp
    // CTAs are used, which free their SM slot as soon as they finish.
    int n_sm = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    struct Shape { int lanes, wpc; unsigned grid; size_t smem; };
    auto shape_for = [&](size_t entry_bytes) {
        const size_t budget = 227 * 1024, fixed = 1024;
        Shape best{32, 1, 0, 0};
        bool found = false;
        for (int lanes = 32; lanes >= 1; lanes >>= 1) {
            const long long n_warps = (n_units + lanes - 1) / lanes;
            const size_t per_warp = (size_t)cap * lanes * entry_bytes;
            const long long per_sm = (n_warps + n_sm - 1) / n_sm;              // warps an SM must hold
            if (lanes < 32 && per_sm > SIM_SPREAD_WARPS_PER_SM) break;
            const long long ctas = (per_sm + 31) / 32;                         // CTAs per SM
            const long long wpc = (per_sm + ctas - 1) / ctas;
            if ((size_t)ctas * ((size_t)wpc * per_warp + fixed) > budget) break;
            best = Shape{lanes, (int)wpc, (unsigned)((n_warps + wpc - 1) / wpc), (size_t)wpc * per_warp};
            found = true;
        }
        if (!found) {
            const long long n_warps = (n_units + 31) / 32;
            best = Shape{32, 1, (unsigned)n_warps, (size_t)cap * 32 * entry_bytes};
        }
        return best;
    };
    const Shape sn = shape_for(sizeof(uint32_t)), sw = shape_for(sizeof(unsigned long long));
    auto kern_n = sn.lanes == 32 ? k_simulate<NarrowEntry, true> : k_simulate<NarrowEntry, false>;
    auto kern_w = sw.lanes == 32 ? k_simulate<WideEntry, true> : k_simulate<WideEntry, false>;
    cudaError_t e = allow_max_dynamic_smem(reinterpret_cast<const void*>(kern_n));
    if (e != cudaSuccess) return e;
    e = allow_max_dynamic_smem(reinterpret_cast<const void*>(kern_w));
    if (e != cudaSuccess) return e;
    launch_hook("k_simulate", 0, st);
    kern_n<<<sn.grid, 32 * sn.wpc, sn.smem, st>>>(
        q_po, q_off, inst_status, lambda_q16, n_lambda, b.n_clients, n_pad, n_units, sn.lanes, cap,
        kv, cm, q_shift, max_iters, cres, trace, trace_off, status, log.events, log.ev_stride, log.event_count,
        log.kind);
    launch_hook("k_simulate", 1, st);
    if (b.kv_budget >= 65536) {                          // otherwise no p + o can reach 2^16
        launch_hook("k_simulate_wide", 0, st);
        kern_w<<<sw.grid, 32 * sw.wpc, sw.smem, st>>>(
            q_po, q_off, inst_status, lambda_q16, n_lambda, b.n_clients, n_pad, n_units, sw.lanes, cap,
            kv, cm, q_shift, max_iters, cres, trace, trace_off, status, log.events, log.ev_stride,
            log.event_count, log.kind);
        launch_hook("k_simulate_wide", 1, st);
    }
    return cudaGetLastError();
}

int event_log_chunks(int n_pad, int n_clients) { return (2 * n_pad + LOG_CHUNK - 1) / LOG_CHUNK + n_clients; }
int event_log_chunk_entries() { return LOG_CHUNK; }

size_t simulate_steal_smem(int n_clients, int cap, bool wide) {
    const int threads = (n_clients + 31) & ~31;
    return (size_t)cap * threads * (wide ? sizeof(unsigned long long) : sizeof(uint32_t));
}

cudaError_t launch_simulate_steal(const hos_batch& b, const hos_cost_model& cm, const uint32_t* lambda_q16,
                                  int n_lambda, uint32_t max_iters, const uint2* q_po, const uint32_t* q_key,
                                  const uint32_t* q_req,
                                  const int32_t* q_off, const int32_t* inst_status, int n_pad,
                                  hos_client_result* cres, hos_iter_rec* trace, const long long* trace_off,
                                  int32_t* status, int32_t* served_by, const EventLog& log, cudaStream_t st) {
    const int threads = (b.n_clients + 31) & ~31;
    const int cap = sim_slots(b);
    const uint32_t kv = sim_budget(b);
    const unsigned grid = (unsigned)(b.n_inst * n_lambda);
    int q_shift = -1;
    if ((cm.decode_kv_div & (cm.decode_kv_div - 1)) == 0)
        for (q_shift = 0; (1u << q_shift) != cm.decode_kv_div; ++q_shift) {}
    const size_t smem_n = simulate_steal_smem(b.n_clients, cap, false);
    const size_t smem_w = simulate_steal_smem(b.n_clients, cap, true);
    cudaError_t e = allow_max_dynamic_smem(reinterpret_cast<const void*>(k_simulate_steal<NarrowEntry>));
    if (e != cudaSuccess) return e;
    launch_hook("k_simulate_steal", 0, st);
    k_simulate_steal<NarrowEntry><<<grid, threads, smem_n, st>>>(
        q_po, b.o_est ? q_key : nullptr, q_req, q_off, inst_status, lambda_q16, n_lambda, b.n_clients, b.n_req, n_pad, cap,
        kv, cm, q_shift, max_iters, cres, trace, trace_off, status, served_by, log.events, log.ev_stride,
        log.pool_chunks, log.chunk_tag, log.chunk_dir, log.dir_start, log.event_count, log.kind);
    launch_hook("k_simulate_steal", 1, st);
    if (b.kv_budget >= 65536) {                          // otherwise no p + o can reach 2^16
        e = allow_max_dynamic_smem(reinterpret_cast<const void*>(k_simulate_steal<WideEntry>));
        if (e != cudaSuccess) return e;
        launch_hook("k_simulate_steal_wide", 0, st);
        k_simulate_steal<WideEntry><<<grid, threads, smem_w, st>>>(
            q_po, b.o_est ? q_key : nullptr, q_req, q_off, inst_status, lambda_q16, n_lambda, b.n_clients, b.n_req, n_pad, cap,
            kv, cm, q_shift, max_iters, cres, trace, trace_off, status, served_by, log.events, log.ev_stride,
            log.pool_chunks, log.chunk_tag, log.chunk_dir, log.dir_start, log.event_count, log.kind);
        launch_hook("k_simulate_steal_wide", 1, st);
    }
    return cudaGetLastError();
}

cudaError_t launch_trace_fill(const hos_batch& b, const hos_cost_model& cm, int n_lambda,
                              const int32_t* q_off, int n_pad, const hos_client_result* cres,
                              const EventLog& log, hos_iter_rec* trace,
                              const long long* trace_off, int32_t* status, cudaStream_t st) {
    const long long n_units = (long long)b.n_inst * n_lambda * b.n_clients;
    int q_shift = -1;
    if ((cm.decode_kv_div & (cm.decode_kv_div - 1)) == 0)
        for (q_shift = 0; (1u << q_shift) != cm.decode_kv_div; ++q_shift) {}
    launch_hook("k_trace_fill", 0, st);
    k_trace_fill<<<(unsigned)((n_units + 3) / 4), 128, 0, st>>>(q_off, n_lambda, b.n_clients, n_pad, n_units,
                                                                cm, q_shift, cres, log.events, log.ev_stride,
                                                                log.event_count, log.kind, log.pool_chunks,
                                                                log.chunk_dir, log.dir_start,
                                                                trace, trace_off, status);
    launch_hook("k_trace_fill", 1, st);
    return cudaGetLastError();
}

cudaError_t launch_finalize(const hos_batch& b, int n_lambda, const unsigned long long* inst_O,
                            hos_client_result* cres, hos_sim_result* sres, cudaStream_t st) {
    const int n_sims = b.n_inst * n_lambda;
    launch_hook("k_finalize", 0, st);
    k_finalize<<<(n_sims + 3) / 4, 128, 0, st>>>(n_sims, n_lambda, b.n_clients, b.batch_cap, inst_O,
                                                 cres, sres);
    launch_hook("k_finalize", 1, st);
    return cudaGetLastError();
}

cudaError_t launch_trace_offsets(const hos_client_result* cres, long long n_units, long long* trace_off,
                                 cudaStream_t st) {
    launch_hook("k_trace_offsets", 0, st);
    // at most one CTA per SM of the largest part, each with whole tiles of 1,024 units
    const long long tiles = (n_units + 1023) / 1024;
    const long long ctas = tiles < 1 ? 1 : (tiles < 148 ? tiles : 148);
    const long long slice = (tiles + ctas - 1) / ctas * 1024;
    k_trace_offsets<<<(unsigned)ctas, 1024, 0, st>>>(cres, n_units, slice, trace_off);
    launch_hook("k_trace_offsets", 1, st);
    return cudaGetLastError();
}

}  // namespace hos
