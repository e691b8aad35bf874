// Internal launch interface between the C-ABI layer and the kernel translation units.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "hos.h"

namespace hos {

struct InstInfo;

// Bounds-checked build: add this translation unit's violation count (no-ops otherwise).
void debug_bounds_offline(unsigned long long* count, long long* first);
void debug_bounds_online(unsigned long long* count, long long* first);
void debug_bounds_multifit(unsigned long long* count, long long* first);

// Calls the user's launch hook, if one is set (see hos_set_launch_hook).
void launch_hook(const char* kernel, int phase, cudaStream_t st);

// Lets `func` be launched with any dynamic shared memory size up to what an SM offers beside the
// kernel's static shared memory.  Done once per kernel and device and never lowered, so that
// host threads that launch different shapes at the same time cannot undo each other's setting.
cudaError_t allow_max_dynamic_smem(const void* func);

size_t estimate_sort_smem(int n_req);
size_t local_search_smem(int n_req, int n_clients);
size_t queue_build_smem(int n_req);

cudaError_t launch_estimate_sort(const hos_batch& b, const hos_cost_model& cm, uint32_t* T_sorted,
                                 uint32_t* order, InstInfo* info, int32_t* status_out, hos_lb* lb_out, int n_pad,
                                 cudaStream_t st);
cudaError_t launch_lpt(const hos_batch& b, const uint32_t* T_sorted, const uint32_t* order,
                       const InstInfo* info, int n_pad, int32_t* assign, long long* load,
                       long long* makespan, uint8_t* rank_client, cudaStream_t st);
cudaError_t launch_multifit(const hos_batch& b, const uint32_t* T_sorted, const uint32_t* order,
                            const InstInfo* info, int n_pad, int max_steps, int32_t* assign, long long* load,
                            long long* makespan, uint8_t* rank_client, int32_t* packer, cudaStream_t st);
cudaError_t launch_pick_packing(const hos_batch& b, int rounds, const int32_t* alt_ok, const int32_t* alt_assign,
                                const long long* alt_load, const long long* alt_makespan, const int32_t* alt_rounds,
                                const hos_ls_move* alt_log, int32_t* assign, long long* load, long long* makespan,
                                int32_t* rounds_applied, hos_ls_move* ls_log, int32_t* packer, cudaStream_t st);
cudaError_t launch_local_search(const hos_batch& b, const uint32_t* T_sorted, const uint32_t* order,
                                const InstInfo* info, int n_pad, int n_copies, int rounds,
                                bool load_from_assign, int32_t* assign, long long* load,
                                long long* makespan, int32_t* rounds_applied, hos_ls_move* ls_log,
                                int32_t* status, uint32_t* ws_T, void* ws_I, uint8_t* ws_C, int32_t* ws_off,
                                int32_t* ws_bad, cudaStream_t st);
size_t local_search_index_bytes(int n_req);
cudaError_t launch_queue_build(const hos_batch& b, const int32_t* assign, uint32_t p_max, int queue_order, uint2* q_po,
                               uint32_t* q_key, uint32_t* q_req, int32_t* q_off, unsigned long long* inst_O,
                               int32_t* inst_status, int n_pad, cudaStream_t st);
// The event log of a simulation call, in the caller's workspace (all null without a log).  A
// simulation owns `ev_stride` = pool_chunks * event_log_chunk_entries() entries of `events`: the
// plain simulator gives client c the entries from 2 * q_off[c] on; the stealing simulator hands
// them out in chunks and lists every client's chunks in `chunk_dir` from `dir_start[unit]` on.
struct EventLog {
    uint4* events;              // [n_sims][ev_stride]
    long long ev_stride;
    uint32_t* event_count;      // [n_units]
    uint32_t* kind;             // one word: which simulator wrote the log
    int pool_chunks;            // chunks per simulation
    uint32_t* chunk_tag;        // [n_sims][pool_chunks]  owner << 16 | number within the owner's log
    uint32_t* chunk_dir;        // [n_sims][pool_chunks]  chunks by owner, then by number
    uint32_t* dir_start;        // [n_units]
};
int event_log_chunks(int n_pad, int n_clients);
int event_log_chunk_entries();
cudaError_t launch_simulate(const hos_batch& b, const hos_cost_model& cm, const uint32_t* lambda_q16,
                            int n_lambda, uint32_t max_iters, const uint2* q_po, const int32_t* q_off,
                            const int32_t* inst_status, int n_pad, hos_client_result* cres,
                            hos_iter_rec* trace, const long long* trace_off, int32_t* status,
                            const EventLog& log, cudaStream_t st);
size_t simulate_steal_smem(int n_clients, int cap, bool wide);
cudaError_t launch_simulate_steal(const hos_batch& b, const hos_cost_model& cm, const uint32_t* lambda_q16,
                                  int n_lambda, uint32_t max_iters, const uint2* q_po, const uint32_t* q_key,
                                  const uint32_t* q_req,
                                  const int32_t* q_off, const int32_t* inst_status, int n_pad,
                                  hos_client_result* cres, hos_iter_rec* trace, const long long* trace_off,
                                  int32_t* status, int32_t* served_by, const EventLog& log, cudaStream_t st);
cudaError_t launch_trace_fill(const hos_batch& b, const hos_cost_model& cm, int n_lambda,
                              const int32_t* q_off, int n_pad, const hos_client_result* cres,
                              const EventLog& log, hos_iter_rec* trace,
                              const long long* trace_off, int32_t* status, cudaStream_t st);
cudaError_t launch_finalize(const hos_batch& b, int n_lambda, const unsigned long long* inst_O,
                            hos_client_result* cres, hos_sim_result* sres, cudaStream_t st);
cudaError_t launch_trace_offsets(const hos_client_result* cres, long long n_units, long long* trace_off,
                                 cudaStream_t st);

}  // namespace hos
