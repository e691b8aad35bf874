/*
 * hos -- batched evaluation of the hybrid offline-online LLM-inference scheduler
 * of arXiv 2502.15763 on one NVIDIA B200 (sm_100a).
 *
 * C ABI.  Conventions shared by every call:
 *   - `hos_batch`, `hos_cost_model` and every `const T*` marked HOST are read on
 *     the host during the call.  Every other pointer is DEVICE memory owned by
 *     the caller; the library allocates nothing, keeps no results or data between calls,
 *     enqueues its kernels on `stream` (a cudaStream_t passed as void*) and
 *     returns without synchronising.  Results are valid once `stream` has
 *     reached the point of the call's return.
 *   - Tables are row-major.  A batch holds `n_inst` independent scheduling
 *     instances of the same shape: `n_req` requests, `n_clients` clients, each
 *     client with `batch_cap` slots and `kv_budget` KV tokens.
 *   - Return value: HOS_OK or a negative HOS_E_* code found on the host before
 *     anything is enqueued (bad sizes, null pointers, workspace too small,
 *     unsupported shape, CUDA launch error).  Problems that depend on the data
 *     (a zero length, a request larger than the KV budget, an iteration limit,
 *     a trace buffer that is too small) never trap: they set bits of the
 *     per-unit `status` word on the device and the unit's results are zeroed
 *     (HOS_ST_INVALID) or truncated (HOS_ST_LIMIT, HOS_ST_TRACE).
 *   - Workspaces are scratch: contents are undefined before and after a call;
 *     base must be 256-byte aligned.  Two calls that share a workspace or an
 *     output buffer must be ordered on the stream.
 *   - Shape limits of this library: n_clients <= 256, batch_cap <= 256,
 *     n_req <= 24384, kv_budget < 2^31, estimated times T_i < 2^32; for the lower bounds
 *     also n_req * R^2 / 2 < 2^63, R = the most KV tokens one request may need
 *     (kv_reserve_tokens if set, else kv_budget).
 *   - Calls may come from several host threads at once (each with its own stream, workspace
 *     and outputs).  The only things the library remembers are idempotent per-device set-up
 *     facts (a kernel's shared-memory allowance, the address of the built-in scratch), kept
 *     under a lock.
 */
#ifndef HOS_H
#define HOS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    HOS_OK            =  0,
    HOS_E_INVALID     = -1,   /* null pointer, non-positive size, inconsistent arguments        */
    HOS_E_WORKSPACE   = -2,   /* workspace smaller than hos_*_workspace_bytes, or misaligned     */
    HOS_E_CUDA        = -3,   /* a CUDA runtime call failed (see cudaGetLastError)               */
    HOS_E_UNSUPPORTED = -4,   /* shape outside the limits listed above                           */
    HOS_E_TOO_LARGE   = -5    /* batch needs more scratch than hos_lower_bound_static has built in */
};

/* bits of the per-unit device status words */
enum {
    HOS_ST_LIMIT   = 1,       /* iteration limit or 2^39 us clock limit reached; results partial */
    HOS_ST_TRACE   = 2,       /* more iterations than trace slots; extra records dropped         */
    HOS_ST_INVALID = 4,       /* instance data invalid (p_i = 0, o_i = 0, p_i + o_i > kv_budget,
                                 T_i >= 2^32, assignment outside [0, n_clients), or a queue key
                                 p_i + o_est_i too long to sit beside the client number in 32
                                 bits: bit_width(max p + o_est) + bit_width(n_clients - 1) > 32) */
    HOS_ST_RANGE   = 8        /* a lower bound of this instance does not fit 64 bits (products of
                                 coefficients and token sums that are each inside their limits);
                                 its hos_lb is zeroed, everything else is unaffected             */
};

enum { HOS_QUEUE_SORTED = 0, HOS_QUEUE_FCFS = 1 };

/* Integer-microsecond cost model.  The paper profiles both stage times as affine in the
 * token counts (Numerical Experiment, "Experiment settings"); the KV term comes from the
 * synthetic workloads' definition.  prefill iteration = prefill_fixed_us + prefill_per_token_us * sum p;
 * decode iteration = decode_fixed_us + decode_per_seq_us * B + floor(sum KV / decode_kv_div);
 * estimated request time T_i = est_per_prompt_token * p_i + est_per_output_token * o_i.
 * Requires decode_fixed_us >= 1, decode_kv_div >= 1, and both iteration durations < 2^31
 * for any admissible batch. */
#define HOS_MAX_LEVELS 8
typedef struct hos_cost_model {
    uint32_t prefill_fixed_us, prefill_per_token_us;
    uint32_t decode_fixed_us, decode_per_seq_us, decode_kv_div;
    uint32_t est_per_prompt_token, est_per_output_token;
    /* Stepped prefill cost, Eq. 5-7: with n_levels > 0 (at most HOS_MAX_LEVELS) a prefill stage is
     * at the smallest level l whose capacity level_cap_tokens[l] (N^cap_l, strictly ascending)
     * holds its prompt tokens and lasts level_time_us[l] (T^p_l, non-decreasing, < 2^31); the two
     * prefill_* coefficients are then unused, no stage takes more than the largest level's
     * tokens, and a prompt longer than that makes its instance HOS_ST_INVALID.  n_levels = 0:
     * the affine cost above. */
    uint32_t n_levels;
    uint32_t level_cap_tokens[HOS_MAX_LEVELS];
    uint32_t level_time_us[HOS_MAX_LEVELS];
} hos_cost_model;

/* HOST struct; p and o are DEVICE tables [n_inst][n_req] of prompt lengths N^p_i and output
 * lengths N^d_i (both >= 1, Notation table of the paper).
 *
 * Output lengths that are only estimated (Section "Problem formulation": the number of output
 * tokens is not known before inference; the offline model works on an estimate of it): o_est,
 * nullable, is a DEVICE table of the same shape with the lengths the scheduler believes (>= 1).
 * With it, the estimated times T_i, the offline packing, the queue order of Algorithm 1 and its
 * count of queued tokens use o_est, while the simulation decodes the true o_i tokens, and the
 * lower bounds of the simulated makespan use the true lengths.  A request's KV need is then not
 * known at admission, so every request reserves kv_reserve_tokens from admission to retirement
 * (the paper's experiment reserves the blocks of the maximum input plus output for each
 * request); a request with p_i + o_i above that makes its instance HOS_ST_INVALID.
 * kv_reserve_tokens = 0: a request reserves p_i + o_i (requires o_est = NULL);
 * kv_reserve_tokens must not exceed kv_budget. */
typedef struct hos_batch {
    int32_t n_inst, n_req, n_clients, batch_cap;
    int64_t kv_budget;
    const uint32_t* p;
    const uint32_t* o;
    const uint32_t* o_est;
    uint32_t kv_reserve_tokens;
} hos_batch;

/* One local-search round: request i left the critical client for client k; u >= 0 came back
 * in exchange (swap), u = -1 is a plain move; v = max of the two changed loads afterwards.
 * A round that found no improving step is {-1, -1, -1, current maximum load}. */
typedef struct hos_ls_move { int32_t i, u, k; int64_t v; } hos_ls_move;

/* Lower bounds of one instance.  lb_pack (units of T) bounds the optimum of the offline
 * model, Eq. 26-30: max(ceil(sum_T / M), max_T, pair_T), pair_T = T_(M) + T_(M+1) when
 * n_req > M.  lb_sim_us bounds every simulated makespan: max(work, chain_us), where work
 * is Eq. 32's t^p* + t^d* for M clients (tp_star_us, td_star_us are the two terms, each
 * rounded up) and chain_us is the longest request served alone.  With prefill levels t^p* is
 * max(T^p_1 * ceil(n_req / batch_cap), min_l floor(P / N^cap_l) * T^p_l), valid for any level
 * table; tp_paper_us is Eq. 31 as printed, T^p_L * floor(P / N^cap_L) for the largest level (not
 * divided by the number of clients; 0 without levels). */
typedef struct hos_lb {
    int64_t lb_pack, sum_T, max_T, pair_T;
    int64_t lb_sim_us, tp_star_us, td_star_us, chain_us;
    int64_t tp_paper_us;
} hos_lb;

typedef struct hos_client_result {
    int64_t  makespan_us;        /* this client's clock when its last request retired        */
    int64_t  busy_slot_us;       /* sum over iterations of duration * requests advanced       */
    uint32_t n_prefill_iters, n_decode_iters;
    uint64_t trace_hash;         /* checksum of the trace records in order (a multiply-add
                                    recurrence mod 2^64), produced with or without the trace  */
    double   utilisation;        /* busy_slot_us / (batch_cap * makespan of the simulation)   */
} hos_client_result;

typedef struct hos_sim_result {
    int64_t makespan_us;         /* max over clients                                          */
    int64_t busy_slot_us;        /* sum over clients                                          */
    double  utilisation;         /* busy / (n_clients * batch_cap * makespan)                 */
    double  tokens_per_s;        /* sum o_i * 1e6 / makespan                                  */
} hos_sim_result;

/* One iteration of one client.  prefill: {duration, 2^31 | admitted requests, sum of their
 * prompt tokens, queue position of the first admitted}.  decode: {duration, B, sum of KV
 * lengths before the step, requests retired by the step}. */
typedef struct hos_iter_rec { uint32_t dur_us, kind_n, tokens, aux; } hos_iter_rec;

/*
 * Offline request scheduling, Eq. 26-30 (Minimizing-Makespan Bin Packing): T_i, per-instance
 * order by (T descending, index ascending), longest-first list scheduling onto the least
 * loaded client (ties: lowest client), then `ls_rounds` rounds of local search, each applying
 * the single move or pairwise swap off the most loaded client that minimises
 * (v, i, k, u) lexicographically, if v is below the current maximum load.
 *   assign         [n_inst][n_req]     out  client of every request (-1 in invalid instances)
 *   load           [n_inst][n_clients] out  sum of T_i per client
 *   makespan_est   [n_inst]            out  max_j load
 *   rounds_applied [n_inst]            out  local-search rounds that changed the assignment
 *   ls_log         [n_inst][ls_rounds] out, nullable
 *   lb             [n_inst]            out, nullable: the lower bounds of hos_lower_bound, from the
 *                                      sort this call does anyway (saves the separate call its own)
 *   status         [n_inst]            out  0, HOS_ST_INVALID, or HOS_ST_RANGE (with lb)
 */
int hos_offline_pack(const hos_batch* batch, const hos_cost_model* cm, int ls_rounds,
                     int32_t* assign, int64_t* load, int64_t* makespan_est,
                     int32_t* rounds_applied, hos_ls_move* ls_log, hos_lb* lb, int32_t* status,
                     void* ws, size_t ws_bytes, void* stream);

/*
 * hos_offline_pack with a stronger packing before the local search.  The paper solves Eq. 26-30
 * to optimality with a MIP solver (Numerical Experiment: "offline" and "offline + online" runs);
 * this call narrows the gap to that optimum with MULTIFIT (Coffman, Garey, Johnson 1978):
 * bisection on a common capacity C over [max(ceil(sum T / M), max T), max(ceil(2 sum T / M), max T)],
 * at most `multifit_steps` probes (>= 1; 64 always converges), each probe a first-fit decreasing
 * pass (every request, longest first, to the lowest client where load + T <= C; success halves the
 * interval from above, failure from below).  Both packings -- the longest-first list schedule and
 * the first-fit decreasing one at the capacity found -- are improved by the same `ls_rounds`
 * rounds of local search, and every instance keeps the better result: the list schedule's unless
 * the other's largest load is strictly smaller (so the result is never worse than
 * hos_offline_pack's).
 *   packer [n_inst] out, nullable: 1 where the MULTIFIT packing was kept, 0 where the list
 *   schedule was.  Everything else as in hos_offline_pack, except the workspace:
 *   hos_offline_multifit_workspace_bytes (room for the second packing).
 */
int hos_offline_pack_multifit(const hos_batch* batch, const hos_cost_model* cm, int multifit_steps,
                              int ls_rounds, int32_t* assign, int64_t* load, int64_t* makespan_est,
                              int32_t* rounds_applied, hos_ls_move* ls_log, hos_lb* lb, int32_t* status,
                              int32_t* packer, void* ws, size_t ws_bytes, void* stream);

/*
 * Local-search rounds only, from given assignments (same rule as in hos_offline_pack).
 * Every instance carries `n_copies` independent assignments (for instance one per
 * multiplier value of a sweep); request data are shared by the copies.
 *   assign [n_inst][n_copies][n_req] in/out;  load, makespan_est, rounds_applied, ls_log
 *   are laid out [n_inst][n_copies][...];  load is recomputed from assign on entry.
 *   status [n_inst] out.
 */
int hos_local_search(const hos_batch* batch, const hos_cost_model* cm, int n_copies, int ls_rounds,
                     int32_t* assign, int64_t* load, int64_t* makespan_est,
                     int32_t* rounds_applied, hos_ls_move* ls_log, int32_t* status,
                     void* ws, size_t ws_bytes, void* stream);

/* Theoretical lower bounds, Eq. 31-32 and the relaxations of Eq. 26-30.  out [n_inst],
 * status [n_inst]. */
int hos_lower_bound(const hos_batch* batch, const hos_cost_model* cm, hos_lb* out, int32_t* status,
                    void* ws, size_t ws_bytes, void* stream);

/*
 * Online scheduling.  Queues: the requests of each client in the order of Algorithm 1
 * (N^p + N^d descending, ties by index; HOS_QUEUE_FCFS: index order).  Then one simulation
 * per (instance, multiplier, client): every iteration either prefills the longest
 * admissible queue prefix (batch cap and KV budget, p+o reserved per request) or decodes one
 * token for every running request; with candidates and a non-empty batch it prefills iff
 * lambda * C_d > C_p (Section "Online requests and iteration scheduling": C_p = cost of
 * that prefill, C_d = decode time waited since the last prefill; lambda = 1.0 is the
 * paper's rule), lambda in Q16.16.
 *   assign     [n_inst][n_req]                  in
 *   lambda_q16 [n_lambda]                       in (DEVICE)
 *   cres       [n_inst][n_lambda][n_clients]    out
 *   sres       [n_inst][n_lambda]               out
 *   status     [n_inst][n_lambda][n_clients]    out  HOS_ST_* bits
 *   trace      nullable; with trace_off [n_inst*n_lambda*n_clients + 1] (DEVICE, ascending):
 *              unit x = (inst*n_lambda + l)*n_clients + c writes its iterations, in order, to
 *              trace[trace_off[x] .. trace_off[x+1]).  Sizes come from a first call with
 *              trace = NULL (n_prefill_iters + n_decode_iters) and hos_trace_offsets, or from
 *              any upper bound the caller chooses.  (With sizes from a first call, hos_trace_fill
 *              below is the cheaper way to get the trace.)
 *   max_iters  at most this many iterations per client (then HOS_ST_LIMIT).
 *   keep_events  non-zero: also leave in `ws` the log of the iterations in which something
 *              changes (prefills and decodes that retire requests; at most two per request),
 *              from which hos_trace_fill rebuilds the full trace without simulating again.
 *              Needs the larger workspace of hos_online_workspace_bytes(.., keep_events = 1).
 */
int hos_online_simulate(const hos_batch* batch, const int32_t* assign, const hos_cost_model* cm,
                        const uint32_t* lambda_q16, int n_lambda, int queue_order, uint32_t max_iters,
                        hos_client_result* cres, hos_sim_result* sres,
                        hos_iter_rec* trace, const int64_t* trace_off, int32_t* status,
                        int keep_events, void* ws, size_t ws_bytes, void* stream);

/*
 * Online scheduling with the second part of Algorithm 1 ("sorting and online preemptive
 * method"): the clients of an instance are advanced together in global time order (earliest
 * clock first, ties to the lower client), and a client whose own queue is used up while it
 * still has a free slot takes the longest waiting request (the head of the queue) of the
 * client with the most queued tokens, sum of p+o (ties to the lower client), as long as it
 * fits its KV budget.  A request counts as taken from the moment a client has picked it as a
 * candidate for its next prefill.  Everything else -- queues, iteration rule, results, trace,
 * status bits -- is as in hos_online_simulate.
 *   served_by [n_inst][n_lambda][n_req]  out, nullable: the client that served each request.
 *   keep_events  as in hos_online_simulate: the event log stays in `ws` for hos_trace_fill.  Here
 *              a client's logged iterations are not bounded by its own queue, only all clients'
 *              together by two per request of the instance; the log is handed out in chunks.
 *              Same workspace size as for hos_online_simulate with keep_events.
 * Limit of this library: n_clients (rounded up to 32) * batch_cap heap entries of one simulation
 * must fit one CTA's shared memory (HOS_E_UNSUPPORTED otherwise).
 */
int hos_online_simulate_steal(const hos_batch* batch, const int32_t* assign, const hos_cost_model* cm,
                              const uint32_t* lambda_q16, int n_lambda, int queue_order,
                              uint32_t max_iters, hos_client_result* cres, hos_sim_result* sres,
                              hos_iter_rec* trace, const int64_t* trace_off, int32_t* status,
                              int32_t* served_by, int keep_events, void* ws, size_t ws_bytes,
                              void* stream);

/*
 * The iteration trace from the event log of a hos_online_simulate or hos_online_simulate_steal
 * call made with keep_events != 0 (the workspace records which of the two wrote it): between two logged iterations a client only decodes, with a constant
 * batch and sum KV growing by B per iteration, so every record in between follows from the
 * log (same records, bit for bit, as a traced simulation).  `batch`, `cm`, `n_lambda`, `cres`
 * and `ws` must be those of that call, and `ws` untouched since.  trace / trace_off as in
 * hos_online_simulate; status [n_units] gets HOS_ST_TRACE OR-ed in where the slots are too few.
 * The usual sequence: simulate (trace = NULL, keep_events = 1) -> hos_trace_offsets ->
 * allocate -> hos_trace_fill.
 */
int hos_trace_fill(const hos_batch* batch, const hos_cost_model* cm, int n_lambda,
                   const hos_client_result* cres, hos_iter_rec* trace, const int64_t* trace_off,
                   int32_t* status, const void* ws, size_t ws_bytes, void* stream);

/*
 * The lower bounds again, for callers that must not allocate.  (The paper has no counterpart:
 * this is a packaging variant of hos_lower_bound, same results bit for bit.)
 *
 * Who needs it: a scheduler that runs next to an inference engine usually finds the device
 * already carved up -- the engine reserved nearly all of HBM for weights and KV cache at
 * start-up, so a cudaMalloc may fail, and even a successful one synchronises the device in the
 * middle of a serving loop.  The same holds for plug-ins that live inside another framework's
 * memory pool and have no allocator of their own.  Such callers pass only inputs and outputs;
 * the scratch that hos_lower_bound asks its caller for sits in a fixed array of
 * HOS_STATIC_SCRATCH_BYTES inside the library's device image.  Every GPU that loads the
 * library carries that array until the process exits, whether or not this call is used.
 *
 *   - The call itself allocates and frees nothing, on host or device.
 *   - Size limit: hos_lower_bound_workspace_bytes(batch) must not exceed
 *     HOS_STATIC_SCRATCH_BYTES (about n_inst * n_req <= 1,000,000 requests); larger batches
 *     get HOS_E_TOO_LARGE and nothing is enqueued.  Split them, or use hos_lower_bound.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and remembers it.  Make that first call outside any stream capture.
 *   - All calls on one device share the one array and find the previous call's leftovers in
 *     it; the kernels overwrite everything they later read, so no clearing is needed.  Two
 *     calls that may run at the same time on the same GPU (different streams, or different
 *     host threads without ordering) race on the array: order them on one stream.
 * out [n_inst], status [n_inst] as in hos_lower_bound.
 */
#define HOS_STATIC_SCRATCH_BYTES (8u << 20)
int hos_lower_bound_static(const hos_batch* batch, const hos_cost_model* cm, hos_lb* out,
                           int32_t* status, void* stream);

/* trace_off[0] = 0, trace_off[x+1] = trace_off[x] + iterations of unit x (exclusive scan of
 * n_prefill_iters + n_decode_iters over cres[0..n_units)).  The trace protocol of
 * hos_online_simulate; no counterpart in the paper beyond the Gantt figures of its Numerical
 * Experiment section. */
int hos_trace_offsets(const hos_client_result* cres, int64_t n_units, int64_t* trace_off,
                      void* stream);

size_t hos_offline_workspace_bytes(const hos_batch* batch, int n_copies, int ls_rounds);
size_t hos_offline_multifit_workspace_bytes(const hos_batch* batch, int ls_rounds);
size_t hos_lower_bound_workspace_bytes(const hos_batch* batch);
size_t hos_online_workspace_bytes(const hos_batch* batch, int n_lambda, int keep_events);

const char* hos_strerror(int code);

/*
 * Measurement aid (no counterpart in the paper).  When a hook is set, every kernel launch of
 * the library is bracketed by hook(kernel_name, 0, stream, user) and
 * hook(kernel_name, 1, stream, user), called on the host from the launching thread, so that
 * a caller can record CUDA events on the launching stream and count launches.  Process-wide
 * and not thread-safe: set it only while no other thread is inside the library; pass NULL
 * to remove it.  It is never consulted for any decision of the hot path.
 */
/*
 * Memory-safety aid (no counterpart in the paper).  The library can be built with
 * -DHOS_DEBUG_BOUNDS (libhos_debug.so): every data-dependent index into shared or global
 * memory is then checked, an index out of range is counted and its access skipped -- nothing
 * faults -- and this call synchronises the device and returns the number of violations on the
 * current device since the library was loaded (first, nullable: {site number, index, limit} of
 * the first one).  The ordinary build has no checks and returns -1.
 */
long long hos_debug_bounds_violations(long long* first);

typedef void (*hos_launch_hook)(const char* kernel, int phase, void* stream, void* user);
void hos_set_launch_hook(hos_launch_hook hook, void* user);

#ifdef __cplusplus
}
#endif
#endif /* HOS_H */
