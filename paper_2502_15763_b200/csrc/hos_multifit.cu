// A stronger packing for the offline model (Eq. 26-30): MULTIFIT (Coffman, Garey and Johnson,
// 1978) -- bisection on a common capacity C, first-fit decreasing as the feasibility test.
//
//   k_multifit   one CTA per instance.  The bisection's probes are first-fit decreasing passes
//                over the whole sorted request table, each a dependent chain (a request goes to
//                the LOWEST client with room, so every step needs the loads the step before
//                left).  Seven warps run the seven probes of the next three levels of the
//                bisection tree side by side -- the capacity that would be probed after
//                success/success, success/failure, ... -- and one thread then walks the three
//                levels: the same probe sequence as the step-by-step bisection, in a third of
//                the passes.  That is for small batches, where the chain's latency is all there
//                is; a batch that fills the GPU anyway is bound by instruction issue, and there
//                the four speculative probes in seven that are thrown away cost more than the
//                shorter chain saves, so larger batches resolve two levels per round (three
//                warps) or one (the plain bisection).  A last pass packs at the capacity found
//                and writes it where it beats the makespan it finds there (the caller presets
//                that to the largest value and chooses between the packings afterwards).
#include "hos_common.cuh"
#include "hos_kernels.h"

namespace hos {

constexpr int MF_LEVELS_MAX = 3;                     // bisection levels resolved per round, at most
constexpr int MF_NODES_MAX = (1 << MF_LEVELS_MAX) - 1;   // probes per round, one warp each

// One first-fit decreasing pass by one warp: client j = k * 32 + lane keeps its load in load[k].
// Returns false at the first request that fits nowhere.  With RECORD, rc[r] gets the client of
// the request of rank r.  L is the load type: 32 bits when the capacity fits, else 64.
template <int KPL, typename L, bool RECORD>
__device__ __forceinline__ bool first_fit_pass(const uint32_t* __restrict__ Ts, int n, int n_clients, L C,
                                               L (&load)[KPL], uint8_t* rc) {
    const int lane = lane_id();
    bool valid[KPL];
#pragma unroll
    for (int k = 0; k < KPL; ++k) { load[k] = 0; valid[k] = k * 32 + lane < n_clients; }
    uint32_t tv_next = lane < n ? __ldg(&Ts[lane]) : 0u;
    for (int r0 = 0; r0 < n; r0 += 32) {
        const uint32_t tv = tv_next;
        const int rn = r0 + 32 + lane;
        tv_next = rn < n ? __ldg(&Ts[rn]) : 0u;      // the next 32 requests arrive during these
        const int steps = min(32, n - r0);
        uint32_t mine = 0;
        for (int s = 0; s < steps; ++s) {
            const L t = (L)__shfl_sync(FULL, tv, s);
            int j = -1;
#pragma unroll
            for (int k = 0; k < KPL; ++k) {
                // load <= C always, so C - load does not wrap whatever t is
                const unsigned b = __ballot_sync(FULL, valid[k] && t <= C - load[k]);
                if (j < 0 && b != 0u) {
                    const int l = __ffs(b) - 1;
                    j = k * 32 + l;
                    if (lane == l) load[k] += t;
                }
            }
            if (j < 0) return false;                 // uniform over the warp
            if (RECORD && lane == s) mine = (uint32_t)j;
        }
        if (RECORD && r0 + lane < n) rc[r0 + lane] = (uint8_t)mine;
    }
    return true;
}

template <int KPL, typename L>
__device__ void multifit_instance(const uint32_t* __restrict__ Ts, const uint32_t* __restrict__ od, int n,
                                  int n_clients, unsigned long long sum_T, uint32_t max_T, int max_steps, int levels,
                                  int32_t* __restrict__ asg, long long* __restrict__ load_out,
                                  long long* __restrict__ makespan_out, uint8_t* __restrict__ rank_client,
                                  int32_t* __restrict__ packer_out, uint8_t* s_rc) {
    __shared__ unsigned long long s_lo, s_hi;
    __shared__ int s_steps, s_ok[MF_NODES_MAX], s_take;
    const int nodes = (1 << levels) - 1;
    const int warp = warp_id(), lane = lane_id();
    const unsigned long long M = (unsigned long long)n_clients;
    if (threadIdx.x == 0) {
        // the authors' interval: no packing beats C_L, first-fit decreasing always succeeds at C_U
        const unsigned long long lo = max((sum_T + M - 1ull) / M, (unsigned long long)max_T);
        const unsigned long long hi = max((2ull * sum_T + M - 1ull) / M, (unsigned long long)max_T);
        s_lo = lo; s_hi = hi; s_steps = 0; s_take = 0;
    }
    __syncthreads();
    L load[KPL];
    while (true) {
        const unsigned long long lo0 = s_lo, hi0 = s_hi;
        const int steps0 = s_steps;
        if (lo0 >= hi0 || steps0 >= max_steps) break;            // uniform: shared values
        if (warp < nodes) {
            // my node of the tree: depth d, path bits from the top (0 = the probe above succeeded)
            const int d = warp == 0 ? 0 : (warp < 3 ? 1 : 2);
            const int path = warp - ((1 << d) - 1);
            unsigned long long lo = lo0, hi = hi0;
            bool active = steps0 + d < max_steps;
            for (int e = d - 1; e >= 0 && active; --e) {
                if (lo >= hi) { active = false; break; }
                const unsigned long long C = lo + (hi - lo) / 2;
                if ((path >> e) & 1) lo = C + 1; else hi = C;
            }
            active = active && lo < hi;
            if (active) {
                const unsigned long long C = lo + (hi - lo) / 2;
                const bool ok = first_fit_pass<KPL, L, false>(Ts, n, n_clients, (L)C, load, nullptr);
                if (lane == 0) s_ok[warp] = ok ? 1 : 0;
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long lo = lo0, hi = hi0;
            int steps = steps0, node = 0;
            for (int d = 0; d < levels && lo < hi && steps < max_steps; ++d) {
                const unsigned long long C = lo + (hi - lo) / 2;
                const bool ok = s_ok[node] != 0;
                if (ok) hi = C; else lo = C + 1;
                node = 2 * node + (ok ? 1 : 2);
                ++steps;
            }
            s_lo = lo; s_hi = hi; s_steps = steps;
        }
        __syncthreads();
    }
    // the packing at the capacity found; taken only when strictly better than what is there
    if (warp == 0) {
        const bool ok = first_fit_pass<KPL, L, true>(Ts, n, n_clients, (L)s_hi, load, s_rc);
        unsigned long long mx = 0;
#pragma unroll
        for (int k = 0; k < KPL; ++k)
            if (k * 32 + lane < n_clients) mx = max(mx, (unsigned long long)load[k]);
        mx = warp_max_u64(mx);
        const bool take = ok && (long long)mx < makespan_out[blockIdx.x];
        if (take) {
#pragma unroll
            for (int k = 0; k < KPL; ++k)
                if (k * 32 + lane < n_clients) load_out[(size_t)blockIdx.x * n_clients + k * 32 + lane] = (long long)load[k];
        }
        __syncwarp();
        if (lane == 0) {
            if (take) makespan_out[blockIdx.x] = (long long)mx;
            if (packer_out) packer_out[blockIdx.x] = take ? 1 : 0;
            s_take = take ? 1 : 0;
        }
    }
    __syncthreads();
    if (s_take) {
        for (int r = threadIdx.x; r < n; r += blockDim.x) {
            const uint8_t c = s_rc[r];
            if (!HOS_IN(od[r], n, 401) || !HOS_IN(c, n_clients, 402)) continue;
            asg[od[r]] = (int32_t)c;
            if (rank_client) rank_client[r] = c;
        }
    }
}

template <int KPL>
__global__ void __launch_bounds__(32 * MF_NODES_MAX)
k_multifit(const uint32_t* __restrict__ T_sorted, const uint32_t* __restrict__ order,
           const InstInfo* __restrict__ info, int n_req, int n_pad, int n_clients, int max_steps, int levels,
           int32_t* __restrict__ assign, long long* __restrict__ load_out, long long* __restrict__ makespan_out,
           uint8_t* __restrict__ rank_client, int32_t* __restrict__ packer_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int inst = blockIdx.x;
    const InstInfo inf = info[inst];
    if (inf.status) {
        if (threadIdx.x == 0 && packer_out) packer_out[inst] = 0;
        return;
    }
    const uint32_t* Ts = T_sorted + (size_t)inst * n_pad;
    const uint32_t* od = order + (size_t)inst * n_pad;
    int32_t* asg = assign + (size_t)inst * n_req;
    uint8_t* rc = rank_client ? rank_client + (size_t)inst * n_pad : nullptr;
    const unsigned long long M = (unsigned long long)n_clients;
    const unsigned long long hi = max((2ull * inf.sum_T + M - 1ull) / M, (unsigned long long)inf.max_T);
    if (hi <= 0xFFFFFFFFull)
        multifit_instance<KPL, uint32_t>(Ts, od, n_req, n_clients, inf.sum_T, inf.max_T, max_steps, levels, asg, load_out,
                                         makespan_out, rc, packer_out, smem_raw);
    else
        multifit_instance<KPL, unsigned long long>(Ts, od, n_req, n_clients, inf.sum_T, inf.max_T, max_steps, levels, asg,
                                                   load_out, makespan_out, rc, packer_out, smem_raw);
}

// Keeps, per instance, the better of two finished packings: the alternative replaces the primary
// one when its packing exists (alt_ok) and its largest load is strictly smaller.
__global__ void __launch_bounds__(256)
k_pick_packing(int n_req, int n_clients, int rounds, const int32_t* __restrict__ alt_ok,
               const int32_t* __restrict__ alt_assign, const long long* __restrict__ alt_load,
               const long long* __restrict__ alt_makespan, const int32_t* __restrict__ alt_rounds,
               const hos_ls_move* __restrict__ alt_log, int32_t* __restrict__ assign, long long* __restrict__ load,
               long long* __restrict__ makespan, int32_t* __restrict__ rounds_applied,
               hos_ls_move* __restrict__ ls_log, int32_t* __restrict__ packer) {
    const int inst = blockIdx.x;
    const bool take = alt_ok[inst] != 0 && alt_makespan[inst] < makespan[inst];   // uniform over the CTA
    __syncthreads();                                     // everyone has read the old makespan
    if (threadIdx.x == 0 && packer) packer[inst] = take ? 1 : 0;
    if (!take) return;
    for (int i = threadIdx.x; i < n_req; i += blockDim.x) assign[(size_t)inst * n_req + i] = alt_assign[(size_t)inst * n_req + i];
    for (int j = threadIdx.x; j < n_clients; j += blockDim.x) load[(size_t)inst * n_clients + j] = alt_load[(size_t)inst * n_clients + j];
    if (ls_log)
        for (int r = threadIdx.x; r < rounds; r += blockDim.x) ls_log[(size_t)inst * rounds + r] = alt_log[(size_t)inst * rounds + r];
    if (threadIdx.x == 0) { makespan[inst] = alt_makespan[inst]; rounds_applied[inst] = alt_rounds[inst]; }
}

cudaError_t launch_pick_packing(const hos_batch& b, int rounds, const int32_t* alt_ok, const int32_t* alt_assign,
                                const long long* alt_load, const long long* alt_makespan, const int32_t* alt_rounds,
                                const hos_ls_move* alt_log, int32_t* assign, long long* load, long long* makespan,
                                int32_t* rounds_applied, hos_ls_move* ls_log, int32_t* packer, cudaStream_t st) {
    launch_hook("k_pick_packing", 0, st);
    k_pick_packing<<<b.n_inst, 256, 0, st>>>(b.n_req, b.n_clients, rounds, alt_ok, alt_assign, alt_load, alt_makespan,
                                             alt_rounds, alt_log, assign, load, makespan, rounds_applied, ls_log, packer);
    launch_hook("k_pick_packing", 1, st);
    return cudaGetLastError();
}

HOS_DEFINE_BOUNDS_READER(debug_bounds_multifit)

cudaError_t launch_multifit(const hos_batch& b, const uint32_t* T_sorted, const uint32_t* order,
                            const InstInfo* info, int n_pad, int max_steps, int32_t* assign, long long* load,
                            long long* makespan, uint8_t* rank_client, int32_t* packer, cudaStream_t st) {
    const int M = b.n_clients;
    const size_t smem = ((size_t)b.n_req + 15) & ~(size_t)15;
    // as many levels per round (1, 3 or 7 warps per instance) as leave the schedulers room: up to
    // about six warps per scheduler over the whole batch
    int n_sm = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    int levels = MF_LEVELS_MAX;
    while (levels > 1 && (long long)b.n_inst * ((1 << levels) - 1) > 24ll * n_sm) --levels;
    const int threads = 32 * ((1 << levels) - 1);
#define HOS_MF(KPL)                                                                                        \
    k_multifit<KPL><<<b.n_inst, threads, smem, st>>>(T_sorted, order, info, b.n_req, n_pad, M, max_steps,  \
                                                     levels, assign, load, makespan, rank_client, packer)
    launch_hook("k_multifit", 0, st);
    if (M <= 32) HOS_MF(1);
    else if (M <= 64) HOS_MF(2);
    else if (M <= 128) HOS_MF(4);
    else HOS_MF(8);
#undef HOS_MF
    launch_hook("k_multifit", 1, st);
    return cudaGetLastError();
}

}  // namespace hos
