/*
 * CPU oracle for the hybrid offline-online scheduler (arXiv 2502.15763).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, single-threaded C, written step by step
 * from the paper's definitions; it shares no code, header, table or constant
 * generator with the CUDA library and is never used by the product path.
 * Every function works on ONE scheduling instance held in host memory.
 *
 * Parity pins: every function below is pinned by tests that do not use the
 * oracle itself (hand-worked traces, closed forms, brute-force optima, the
 * paper's printed cost examples, conservation laws).  The paper's outcome
 * figures (80.2 % -> 89.1 % utilisation, 201.00 s -> 190.58 s) depend on a
 * data set and model outputs that are not available: parity unpinned for
 * those, only the sign of the hybrid-vs-baseline gain is checked.
 */
#ifndef HOS_ORACLE_H
#define HOS_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Integer-microsecond cost coefficients (Section "Experiment settings": both
 * stage times are affine in the token counts). */
typedef struct {
    uint32_t prefill_fixed_us;      /* a_p */
    uint32_t prefill_per_token_us;  /* b_p */
    uint32_t decode_fixed_us;       /* a_d */
    uint32_t decode_per_seq_us;     /* b_d */
    uint32_t decode_kv_div;         /* q: decode adds floor(sum KV / q) */
    uint32_t est_per_prompt_token;  /* e_p */
    uint32_t est_per_output_token;  /* e_o */
    /* Eq. 5-7: with n_levels > 0 a prefill stage is at the smallest level l whose capacity
     * N^cap_l holds its tokens and lasts T^p_l (a_p, b_p unused); no stage exceeds the largest. */
    uint32_t n_levels;
    uint32_t level_cap[8];          /* N^cap_l, ascending */
    uint32_t level_time[8];         /* T^p_l, non-decreasing */
} ora_cost;

typedef struct { int32_t i, u, k; int64_t v; } ora_move;

typedef struct {
    int64_t lb_pack, sum_T, max_T, pair_T;
    int64_t lb_sim_us, tp_star_us, td_star_us, chain_us;
    int64_t tp_paper_us;            /* Eq. 31 as printed: T^p_L * floor(sum N^p / N^cap_L); 0 without levels */
} ora_lb;

typedef struct { uint32_t dur_us, kind_n, tokens, aux; } ora_rec;

typedef struct {
    int64_t  makespan_us;
    int64_t  busy_slot_us;
    uint32_t n_prefill_iters, n_decode_iters;
    uint64_t trace_hash;
    int32_t  status;          /* bit 0: iteration / clock limit hit; bit 1: trace buffer too small */
} ora_client;

enum { ORA_QUEUE_SORTED = 0, ORA_QUEUE_FCFS = 1 };

/* T_i = e_p p_i + e_o o_i  (the "estimated decode completion time" of Eq. 26-30). */
void ora_estimate(int n, const uint32_t* p, const uint32_t* o, const ora_cost* c, int64_t* T);

/* order = request indices by (T descending, index ascending). */
void ora_order(int n, const int64_t* T, int32_t* order);

/* Longest-processing-time list scheduling onto M clients (feasible for Eq. 27-28). */
void ora_lpt(int n, int M, const int64_t* T, const int32_t* order, int32_t* assign, int64_t* load);

/* Up to `rounds` rounds of best single move / pairwise swap off the critical client.
 * log (nullable) gets one entry per round; returns the number of applied rounds. */
int ora_local_search(int n, int M, const int64_t* T, int32_t* assign, int64_t* load,
                     int rounds, ora_move* log);

/* MULTIFIT (Coffman, Garey, Johnson 1978) for the same model: bisection on a common capacity C
 * with first-fit decreasing as the feasibility test, at most max_steps probes; the packing is the
 * first-fit decreasing one at the smallest capacity found.  Returns 1 when it exists. */
int ora_multifit(int n, int M, const int64_t* T, const int32_t* order, int max_steps,
                 int32_t* assign, int64_t* load, int64_t* C_final);

/* Optimum of Eq. 26-30 by exhaustive enumeration (M^n assignments; tiny instances only). */
int64_t ora_optimal_makespan(int n, int M, const int64_t* T);

/* Lower bounds (Eq. 31-32 restated for the affine cost model and M clients of `cap` slots). */
void ora_lower_bound(int n, int M, int cap, const uint32_t* p, const uint32_t* o,
                     const ora_cost* c, ora_lb* out);

/* Per-client queues (Algorithm 1, first part): CSR q_off[M+1], q_req[n]. */
/* (o here is what the scheduler sorts by: the output lengths it knows, exact or estimated.) */
void ora_queue_build(int n, int M, const int32_t* assign, const uint32_t* p, const uint32_t* o,
                     int mode, int32_t* q_off, int32_t* q_req);

/* Iteration-level simulation of one client's queue (PD competition + continuous batching,
 * decision rule of the "Online requests and iteration scheduling" section). */
void ora_simulate_client(int qn, const int32_t* q_req, const uint32_t* p, const uint32_t* o,
                         const ora_cost* c, int cap, int64_t kv_budget, int64_t kv_reserve,
                         uint32_t lambda_q16, uint32_t max_iters, ora_client* res, ora_rec* trace,
                         int64_t trace_cap);

/* The same simulation with Algorithm 1's second part: all M clients of one instance advance in
 * global time order (earliest clock first, ties to the lower client); a client whose own queue
 * is exhausted and that still has a free slot takes the head of the queue of the client with
 * the most queued tokens (ties to the lower client).  q_off/q_req: queues from ora_queue_build.
 * res [M]; traces [M] (nullable, each with trace_cap[c] slots); served_by [n] (nullable) gets the
 * client that finally served each request. */
void ora_simulate_steal(int n, int M, const int32_t* q_off, const int32_t* q_req,
                        const uint32_t* p, const uint32_t* o, const uint32_t* o_key, const ora_cost* c,
                        int cap, int64_t kv_budget, int64_t kv_reserve, uint32_t lambda_q16,
                        uint32_t max_iters,
                        ora_client* res, ora_rec** traces, const int64_t* trace_cap,
                        int32_t* served_by);

#ifdef __cplusplus
}
#endif
#endif
