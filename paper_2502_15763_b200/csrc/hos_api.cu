// C-ABI layer: argument validation, workspace carving, kernel sequencing.
#include <cuda_runtime.h>

#include <mutex>
#include <unordered_map>

#include "hos.h"
#include "hos_common.cuh"
#include "hos_kernels.h"

namespace {

using namespace hos;

constexpr size_t WS_ALIGN = 256;
inline size_t up(size_t x) { return (x + WS_ALIGN - 1) & ~(WS_ALIGN - 1); }
inline int pad4(int n) { return (n + 3) & ~3; }
inline int bit_width_host(unsigned long long v) { int b = 0; while (v) { ++b; v >>= 1; } return b; }

int check_batch(const hos_batch* b) {
    if (!b || !b->p || !b->o) return HOS_E_INVALID;
    if (b->n_inst < 1 || b->n_req < 1 || b->n_clients < 1 || b->batch_cap < 1 || b->kv_budget < 1)
        return HOS_E_INVALID;
    if (b->n_clients > MAX_CLIENTS || b->batch_cap > MAX_CAP || b->n_req > MAX_REQ ||
        b->kv_budget >= (1ll << 31))
        return HOS_E_UNSUPPORTED;
    if ((long long)b->n_inst * (long long)pad4(b->n_req) >= (1ll << 40)) return HOS_E_UNSUPPORTED;
    // estimated output lengths need the fixed reservation; a reservation must fit the budget
    if (b->o_est && b->kv_reserve_tokens == 0) return HOS_E_INVALID;
    if ((long long)b->kv_reserve_tokens > (long long)b->kv_budget) return HOS_E_INVALID;
    return HOS_OK;
}

int check_cost(const hos_cost_model* cm, const hos_batch* b) {
    if (!cm) return HOS_E_INVALID;
    if (cm->decode_fixed_us < 1 || cm->decode_kv_div < 1) return HOS_E_INVALID;
    if (cm->n_levels > HOS_MAX_LEVELS) return HOS_E_INVALID;
    for (uint32_t l = 0; l < cm->n_levels; ++l) {
        if (cm->level_cap_tokens[l] < 1 || cm->level_time_us[l] >= (1u << 31)) return HOS_E_INVALID;
        if (l > 0 && (cm->level_cap_tokens[l] <= cm->level_cap_tokens[l - 1] ||
                      cm->level_time_us[l] < cm->level_time_us[l - 1]))
            return HOS_E_INVALID;
    }
    // longest possible iterations must stay below 2^31 us
    const unsigned long long kv = (unsigned long long)b->kv_budget;
    const unsigned long long pre = cm->n_levels ? 0ull :
        cm->prefill_fixed_us + (unsigned long long)cm->prefill_per_token_us * kv;
    const unsigned long long dec = cm->decode_fixed_us +
                                   (unsigned long long)cm->decode_per_seq_us * (unsigned long long)b->batch_cap +
                                   kv / cm->decode_kv_div;
    if (pre >= (1ull << 31) || dec >= (1ull << 31)) return HOS_E_INVALID;
    return HOS_OK;
}

// The lower bounds add up o_i * p_i + o_i (o_i - 1) / 2 <= (p_i + o_i)^2 / 2 over the requests of an
// instance in 64 bits: the largest admissible request bounds that sum.
int check_lb_range(const hos_batch* b) {
    const unsigned long long most = b->kv_reserve_tokens ? b->kv_reserve_tokens : (unsigned long long)b->kv_budget;
    const unsigned __int128 worst = (unsigned __int128)most * most / 2 * (unsigned long long)b->n_req;
    return worst >> 63 ? HOS_E_UNSUPPORTED : HOS_OK;
}

int check_ws(const void* ws, size_t have, size_t need) {
    if (!ws || have < need || (reinterpret_cast<uintptr_t>(ws) & (WS_ALIGN - 1))) return HOS_E_WORKSPACE;
    return HOS_OK;
}

struct OfflineWs {
    uint32_t* T_sorted;
    uint32_t* order;
    InstInfo* info;
    uint32_t* ls_T;             // local search, per (instance, copy): the member lists' T
    void* ls_I;                 // and request indices
    uint8_t* ls_C;              // and the client of every rank of the sorted order
    int32_t* ls_off;            // list offsets, n_clients + 1 per (instance, copy)
    int32_t* ls_bad;            // per (instance, copy): assignment outside [0, n_clients)
    size_t bytes;
};
OfflineWs carve_offline(const hos_batch* b, void* ws, int n_copies, int ls_rounds) {
    OfflineWs w;
    const size_t rows = (size_t)b->n_inst * pad4(b->n_req);
    unsigned char* base = static_cast<unsigned char*>(ws);
    size_t off = 0;
    w.T_sorted = reinterpret_cast<uint32_t*>(base + off); off += up(rows * 4);
    w.order = reinterpret_cast<uint32_t*>(base + off);    off += up(rows * 4);
    w.info = reinterpret_cast<InstInfo*>(base + off);     off += up((size_t)b->n_inst * sizeof(InstInfo));
    w.ls_T = nullptr; w.ls_I = nullptr; w.ls_C = nullptr; w.ls_off = nullptr; w.ls_bad = nullptr;
    if (ls_rounds > 0) {
        const size_t units = rows * (size_t)(n_copies > 0 ? n_copies : 1);
        w.ls_T = reinterpret_cast<uint32_t*>(base + off);  off += up(units * 4);
        w.ls_I = base + off;                               off += up(units * local_search_index_bytes(b->n_req));
        w.ls_C = base + off;                               off += up(units);
        const size_t n_units = (size_t)b->n_inst * (size_t)(n_copies > 0 ? n_copies : 1);
        w.ls_off = reinterpret_cast<int32_t*>(base + off); off += up(n_units * (size_t)(b->n_clients + 1) * 4);
        w.ls_bad = reinterpret_cast<int32_t*>(base + off); off += up(n_units * 4);
    }
    w.bytes = off;
    return w;
}

struct OnlineWs {
    uint2* q_po;
    uint32_t* q_key;            // p + estimated o per queue position (only with hos_batch::o_est)
    uint32_t* q_req;
    int32_t* q_off;
    unsigned long long* inst_O;
    int32_t* inst_status;
    EventLog log;               // all null without keep_events
    size_t bytes;
};
OnlineWs carve_online(const hos_batch* b, void* ws, int n_lambda, int keep_events) {
    OnlineWs w;
    const size_t rows = (size_t)b->n_inst * pad4(b->n_req);
    unsigned char* base = static_cast<unsigned char*>(ws);
    size_t off = 0;
    w.q_po = reinterpret_cast<uint2*>(base + off);                off += up(rows * 8);
    w.q_req = reinterpret_cast<uint32_t*>(base + off);            off += up(rows * 4);
    w.q_key = nullptr;
    if (b->o_est) { w.q_key = reinterpret_cast<uint32_t*>(base + off); off += up(rows * 4); }
    w.q_off = reinterpret_cast<int32_t*>(base + off);             off += up((size_t)b->n_inst * (b->n_clients + 1) * 4);
    w.inst_O = reinterpret_cast<unsigned long long*>(base + off); off += up((size_t)b->n_inst * 8);
    w.inst_status = reinterpret_cast<int32_t*>(base + off);       off += up((size_t)b->n_inst * 4);
    w.log = EventLog{nullptr, 0, nullptr, nullptr, 0, nullptr, nullptr, nullptr};
    if (keep_events) {
        const size_t sims = (size_t)b->n_inst * (size_t)n_lambda;
        const size_t chunks = (size_t)event_log_chunks(pad4(b->n_req), b->n_clients);
        w.log.pool_chunks = (int)chunks;
        w.log.ev_stride = (long long)(chunks * event_log_chunk_entries());
        w.log.kind = reinterpret_cast<uint32_t*>(base + off);         off += up(4);
        w.log.event_count = reinterpret_cast<uint32_t*>(base + off);  off += up(sims * b->n_clients * 4);
        w.log.dir_start = reinterpret_cast<uint32_t*>(base + off);    off += up(sims * b->n_clients * 4);
        w.log.chunk_tag = reinterpret_cast<uint32_t*>(base + off);    off += up(sims * chunks * 4);
        w.log.chunk_dir = reinterpret_cast<uint32_t*>(base + off);    off += up(sims * chunks * 4);
        w.log.events = reinterpret_cast<uint4*>(base + off);          off += up(sims * (size_t)w.log.ev_stride * 16);
    }
    w.bytes = off;
    return w;
}

inline int cuda_rc(cudaError_t e) { return e == cudaSuccess ? HOS_OK : HOS_E_CUDA; }

hos_launch_hook g_hook = nullptr;
void* g_hook_user = nullptr;

}  // namespace

namespace hos {
cudaError_t allow_max_dynamic_smem(const void* func) {
    static std::mutex mu;
    static std::unordered_map<const void*, unsigned long long> done;      // kernel -> devices already set
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    unsigned long long& mask = done[func];
    if (dev >= 0 && dev < 64 && ((mask >> dev) & 1ull)) return cudaSuccess;
    cudaFuncAttributes attr;
    if ((e = cudaFuncGetAttributes(&attr, func)) != cudaSuccess) return e;
    const int room = (int)SMEM_LIMIT - (int)attr.sharedSizeBytes;
    if ((e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, room)) != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) mask |= 1ull << dev;
    return cudaSuccess;
}

void launch_hook(const char* kernel, int phase, cudaStream_t st) {
    if (g_hook) g_hook(kernel, phase, static_cast<void*>(st), g_hook_user);
}
}  // namespace hos

extern "C" {

size_t hos_offline_workspace_bytes(const hos_batch* b, int n_copies, int ls_rounds) {
    if (!b || b->n_inst < 1 || b->n_req < 1) return 0;
    return carve_offline(b, nullptr, n_copies, ls_rounds).bytes;
}
size_t hos_lower_bound_workspace_bytes(const hos_batch* b) {
    if (!b || b->n_inst < 1 || b->n_req < 1) return 0;
    return carve_offline(b, nullptr, 1, 0).bytes;
}
size_t hos_online_workspace_bytes(const hos_batch* b, int n_lambda, int keep_events) {
    if (!b || b->n_inst < 1 || b->n_req < 1 || b->n_clients < 1 || n_lambda < 1) return 0;
    return carve_online(b, nullptr, n_lambda, keep_events).bytes;
}

namespace {
// Buffers of the alternative packing (MULTIFIT start), behind the ordinary offline workspace.
struct AltWs {
    int32_t* assign; long long* load; long long* makespan; int32_t* rounds; hos_ls_move* log; int32_t* ok;
    size_t bytes;
};
AltWs carve_alt(const hos_batch* b, void* ws, size_t at, int ls_rounds) {
    AltWs a;
    unsigned char* base = static_cast<unsigned char*>(ws);
    size_t off = at;
    const size_t n = (size_t)b->n_inst;
    a.assign = reinterpret_cast<int32_t*>(base + off);      off += up(n * (size_t)b->n_req * 4);
    a.load = reinterpret_cast<long long*>(base + off);      off += up(n * (size_t)b->n_clients * 8);
    a.makespan = reinterpret_cast<long long*>(base + off);  off += up(n * 8);
    a.rounds = reinterpret_cast<int32_t*>(base + off);      off += up(n * 4);
    a.ok = reinterpret_cast<int32_t*>(base + off);          off += up(n * 4);
    a.log = reinterpret_cast<hos_ls_move*>(base + off);     off += up(n * (size_t)(ls_rounds > 0 ? ls_rounds : 0) * sizeof(hos_ls_move));
    a.bytes = off;
    return a;
}

int offline_pack_impl(const hos_batch* b, const hos_cost_model* cm, int multifit_steps, int ls_rounds,
                      int32_t* assign, int64_t* load, int64_t* makespan_est, int32_t* rounds_applied,
                      hos_ls_move* ls_log, hos_lb* lb, int32_t* status, int32_t* packer, void* ws,
                      size_t ws_bytes, void* stream) {
    int rc = check_batch(b);
    if (rc) return rc;
    if ((rc = check_cost(cm, b))) return rc;
    if (!assign || !load || !makespan_est || !rounds_applied || !status || ls_rounds < 0 || multifit_steps < 0)
        return HOS_E_INVALID;
    if (lb && (rc = check_lb_range(b))) return rc;
    if (estimate_sort_smem(b->n_req) > SMEM_LIMIT) return HOS_E_UNSUPPORTED;
    const OfflineWs w = carve_offline(b, ws, 1, ls_rounds);
    const AltWs alt = carve_alt(b, ws, w.bytes, ls_rounds);
    if ((rc = check_ws(ws, ws_bytes, multifit_steps > 0 ? alt.bytes : w.bytes))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_pad = pad4(b->n_req);
    long long* ld = reinterpret_cast<long long*>(load);
    long long* mk = reinterpret_cast<long long*>(makespan_est);
    auto search = [&](int32_t* a, long long* l, long long* m, int32_t* applied, hos_ls_move* log) {
        if (ls_rounds == 0) return cuda_rc(cudaMemsetAsync(applied, 0, (size_t)b->n_inst * sizeof(int32_t), st));
        return cuda_rc(launch_local_search(*b, w.T_sorted, w.order, w.info, n_pad, 1, ls_rounds, false, a, l, m, applied,
                                           log, status, w.ls_T, w.ls_I, w.ls_C, w.ls_off, w.ls_bad, st));
    };
    if ((rc = cuda_rc(launch_estimate_sort(*b, *cm, w.T_sorted, w.order, w.info, status, lb, n_pad, st)))) return rc;
    if ((rc = cuda_rc(launch_lpt(*b, w.T_sorted, w.order, w.info, n_pad, assign, ld, mk, w.ls_C, st)))) return rc;
    if ((rc = search(assign, ld, mk, rounds_applied, ls_log))) return rc;
    if (multifit_steps == 0) return HOS_OK;
    // The MULTIFIT packing, improved by the same local search, in buffers of its own; then the better
    // of the two per instance.  (The packing kernel writes where its result beats the makespan it
    // finds: with that preset to the largest value, wherever first-fit decreasing succeeded.)
    if ((rc = cuda_rc(cudaMemsetAsync(alt.makespan, 0x7F, (size_t)b->n_inst * sizeof(long long), st)))) return rc;
    if ((rc = cuda_rc(launch_multifit(*b, w.T_sorted, w.order, w.info, n_pad, multifit_steps, alt.assign, alt.load,
                                      alt.makespan, w.ls_C, alt.ok, st))))
        return rc;
    if ((rc = search(alt.assign, alt.load, alt.makespan, alt.rounds, ls_log ? alt.log : nullptr))) return rc;
    return cuda_rc(launch_pick_packing(*b, ls_rounds, alt.ok, alt.assign, alt.load, alt.makespan, alt.rounds, alt.log,
                                       assign, ld, mk, rounds_applied, ls_log, packer, st));
}
}  // namespace

int hos_offline_pack(const hos_batch* b, const hos_cost_model* cm, int ls_rounds, int32_t* assign,
                     int64_t* load, int64_t* makespan_est, int32_t* rounds_applied,
                     hos_ls_move* ls_log, hos_lb* lb, int32_t* status, void* ws, size_t ws_bytes,
                     void* stream) {
    return offline_pack_impl(b, cm, 0, ls_rounds, assign, load, makespan_est, rounds_applied, ls_log, lb, status,
                             nullptr, ws, ws_bytes, stream);
}

size_t hos_offline_multifit_workspace_bytes(const hos_batch* b, int ls_rounds) {
    if (!b || b->n_inst < 1 || b->n_req < 1 || b->n_clients < 1 || ls_rounds < 0) return 0;
    return carve_alt(b, nullptr, carve_offline(b, nullptr, 1, ls_rounds).bytes, ls_rounds).bytes;
}

int hos_offline_pack_multifit(const hos_batch* b, const hos_cost_model* cm, int multifit_steps, int ls_rounds,
                              int32_t* assign, int64_t* load, int64_t* makespan_est, int32_t* rounds_applied,
                              hos_ls_move* ls_log, hos_lb* lb, int32_t* status, int32_t* packer, void* ws,
                              size_t ws_bytes, void* stream) {
    if (multifit_steps < 1) return HOS_E_INVALID;
    return offline_pack_impl(b, cm, multifit_steps, ls_rounds, assign, load, makespan_est, rounds_applied, ls_log,
                             lb, status, packer, ws, ws_bytes, stream);
}

int hos_local_search(const hos_batch* b, const hos_cost_model* cm, int n_copies, int ls_rounds,
                     int32_t* assign, int64_t* load, int64_t* makespan_est, int32_t* rounds_applied,
                     hos_ls_move* ls_log, int32_t* status, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_batch(b);
    if (rc) return rc;
    if ((rc = check_cost(cm, b))) return rc;
    if (!assign || !load || !makespan_est || !rounds_applied || !status || ls_rounds < 0 || n_copies < 1)
        return HOS_E_INVALID;
    if ((long long)b->n_inst * n_copies > 0x7FFFFFFFll) return HOS_E_UNSUPPORTED;
    if (estimate_sort_smem(b->n_req) > SMEM_LIMIT) return HOS_E_UNSUPPORTED;
    if ((rc = check_ws(ws, ws_bytes, hos_offline_workspace_bytes(b, n_copies, ls_rounds)))) return rc;
    const OfflineWs w = carve_offline(b, ws, n_copies, ls_rounds);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_pad = pad4(b->n_req);
    if ((rc = cuda_rc(launch_estimate_sort(*b, *cm, w.T_sorted, w.order, w.info, status, nullptr, n_pad, st)))) return rc;
    return cuda_rc(launch_local_search(*b, w.T_sorted, w.order, w.info, n_pad, n_copies, ls_rounds, true,
                                       assign, reinterpret_cast<long long*>(load),
                                       reinterpret_cast<long long*>(makespan_est), rounds_applied,
                                       ls_log, status, w.ls_T, w.ls_I, w.ls_C, w.ls_off, w.ls_bad, st));
}

int hos_lower_bound(const hos_batch* b, const hos_cost_model* cm, hos_lb* out, int32_t* status, void* ws,
                    size_t ws_bytes, void* stream) {
    int rc = check_batch(b);
    if (rc) return rc;
    if ((rc = check_cost(cm, b))) return rc;
    if (!out || !status) return HOS_E_INVALID;
    if ((rc = check_lb_range(b))) return rc;
    if (estimate_sort_smem(b->n_req) > SMEM_LIMIT) return HOS_E_UNSUPPORTED;
    if ((rc = check_ws(ws, ws_bytes, hos_lower_bound_workspace_bytes(b)))) return rc;
    const OfflineWs w = carve_offline(b, ws, 1, 0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_pad = pad4(b->n_req);
    return cuda_rc(launch_estimate_sort(*b, *cm, nullptr, nullptr, w.info, status, out, n_pad, st));
}

int hos_online_simulate(const hos_batch* b, const int32_t* assign, const hos_cost_model* cm,
                        const uint32_t* lambda_q16, int n_lambda, int queue_order, uint32_t max_iters,
                        hos_client_result* cres, hos_sim_result* sres, hos_iter_rec* trace,
                        const int64_t* trace_off, int32_t* status, int keep_events, void* ws,
                        size_t ws_bytes, void* stream) {
    int rc = check_batch(b);
    if (rc) return rc;
    if ((rc = check_cost(cm, b))) return rc;
    if (!assign || !lambda_q16 || n_lambda < 1 || !cres || !sres || !status) return HOS_E_INVALID;
    if (queue_order != HOS_QUEUE_SORTED && queue_order != HOS_QUEUE_FCFS) return HOS_E_INVALID;
    if (trace && !trace_off) return HOS_E_INVALID;
    if (queue_build_smem(b->n_req) > SMEM_LIMIT) return HOS_E_UNSUPPORTED;
    if (bit_width_host((unsigned long long)b->kv_budget) + bit_width_host((unsigned long long)(b->n_clients - 1)) > 32)
        return HOS_E_UNSUPPORTED;
    if ((long long)b->n_inst * n_lambda > 0x7FFFFFFFll / 4) return HOS_E_UNSUPPORTED;
    if ((rc = check_ws(ws, ws_bytes, hos_online_workspace_bytes(b, n_lambda, keep_events)))) return rc;
    const OnlineWs w = carve_online(b, ws, n_lambda, keep_events);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_pad = pad4(b->n_req);
    if (max_iters > 0x7FFFFFFFu) max_iters = 0x7FFFFFFFu;
    if ((rc = cuda_rc(launch_queue_build(*b, assign, stage_cap_tokens(*cm), queue_order, w.q_po, w.q_key, w.q_req, w.q_off, w.inst_O,
                                         w.inst_status, n_pad, st))))
        return rc;
    if ((rc = cuda_rc(launch_simulate(*b, *cm, lambda_q16, n_lambda, max_iters, w.q_po, w.q_off,
                                      w.inst_status, n_pad, cres, trace,
                                      reinterpret_cast<const long long*>(trace_off), status, w.log, st))))
        return rc;
    return cuda_rc(launch_finalize(*b, n_lambda, w.inst_O, cres, sres, st));
}

int hos_online_simulate_steal(const hos_batch* b, const int32_t* assign, const hos_cost_model* cm,
                              const uint32_t* lambda_q16, int n_lambda, int queue_order, uint32_t max_iters,
                              hos_client_result* cres, hos_sim_result* sres, hos_iter_rec* trace,
                              const int64_t* trace_off, int32_t* status, int32_t* served_by, int keep_events,
                              void* ws, size_t ws_bytes, void* stream) {
    int rc = check_batch(b);
    if (rc) return rc;
    if ((rc = check_cost(cm, b))) return rc;
    if (!assign || !lambda_q16 || n_lambda < 1 || !cres || !sres || !status) return HOS_E_INVALID;
    if (queue_order != HOS_QUEUE_SORTED && queue_order != HOS_QUEUE_FCFS) return HOS_E_INVALID;
    if (trace && !trace_off) return HOS_E_INVALID;
    if (queue_build_smem(b->n_req) > SMEM_LIMIT) return HOS_E_UNSUPPORTED;
    if (bit_width_host((unsigned long long)b->kv_budget) + bit_width_host((unsigned long long)(b->n_clients - 1)) > 32)
        return HOS_E_UNSUPPORTED;
    if ((long long)b->n_inst * n_lambda > 0x7FFFFFFFll / 4) return HOS_E_UNSUPPORTED;
    // every client's heap of one simulation shares a CTA's shared memory
    const bool may_be_wide = b->kv_budget >= 65536;
    if (simulate_steal_smem(b->n_clients, b->batch_cap, may_be_wide) + 8 * 1024 > SMEM_LIMIT) return HOS_E_UNSUPPORTED;
    if ((rc = check_ws(ws, ws_bytes, hos_online_workspace_bytes(b, n_lambda, keep_events)))) return rc;
    const OnlineWs w = carve_online(b, ws, n_lambda, keep_events);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_pad = pad4(b->n_req);
    if (max_iters > 0x7FFFFFFFu) max_iters = 0x7FFFFFFFu;
    if ((rc = cuda_rc(launch_queue_build(*b, assign, stage_cap_tokens(*cm), queue_order, w.q_po, w.q_key, w.q_req, w.q_off, w.inst_O,
                                         w.inst_status, n_pad, st))))
        return rc;
    if ((rc = cuda_rc(launch_simulate_steal(*b, *cm, lambda_q16, n_lambda, max_iters, w.q_po, w.q_key, w.q_req, w.q_off,
                                            w.inst_status, n_pad, cres, trace,
                                            reinterpret_cast<const long long*>(trace_off), status, served_by,
                                            w.log, st))))
        return rc;
    return cuda_rc(launch_finalize(*b, n_lambda, w.inst_O, cres, sres, st));
}

int hos_trace_fill(const hos_batch* b, const hos_cost_model* cm, int n_lambda, const hos_client_result* cres,
                   hos_iter_rec* trace, const int64_t* trace_off, int32_t* status, const void* ws,
                   size_t ws_bytes, void* stream) {
    int rc = check_batch(b);
    if (rc) return rc;
    if ((rc = check_cost(cm, b))) return rc;
    if (!cres || !trace || !trace_off || !status || n_lambda < 1) return HOS_E_INVALID;
    if ((long long)b->n_inst * n_lambda > 0x7FFFFFFFll / 4) return HOS_E_UNSUPPORTED;
    if ((rc = check_ws(ws, ws_bytes, hos_online_workspace_bytes(b, n_lambda, 1)))) return rc;
    const OnlineWs w = carve_online(b, const_cast<void*>(ws), n_lambda, 1);
    return cuda_rc(launch_trace_fill(*b, *cm, n_lambda, w.q_off, pad4(b->n_req), cres, w.log,
                                     trace, reinterpret_cast<const long long*>(trace_off), status,
                                     static_cast<cudaStream_t>(stream)));
}

int hos_trace_offsets(const hos_client_result* cres, int64_t n_units, int64_t* trace_off, void* stream) {
    if (!cres || !trace_off || n_units < 0) return HOS_E_INVALID;
    return cuda_rc(launch_trace_offsets(cres, (long long)n_units, reinterpret_cast<long long*>(trace_off),
                                        static_cast<cudaStream_t>(stream)));
}

long long hos_debug_bounds_violations(long long* first) {
#ifdef HOS_DEBUG_BOUNDS
    unsigned long long count = 0;
    long long f[3] = {0, 0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) return HOS_E_CUDA;
    debug_bounds_offline(&count, f);
    debug_bounds_online(&count, f);
    debug_bounds_multifit(&count, f);
    if (first) { first[0] = f[0]; first[1] = f[1]; first[2] = f[2]; }
    return (long long)count;
#else
    (void)first;
    return -1;
#endif
}

void hos_set_launch_hook(hos_launch_hook hook, void* user) {
    g_hook = hook;
    g_hook_user = user;
}

const char* hos_strerror(int code) {
    switch (code) {
        case HOS_OK: return "ok";
        case HOS_E_INVALID: return "invalid argument";
        case HOS_E_WORKSPACE: return "workspace missing, too small or not 256-byte aligned";
        case HOS_E_CUDA: return "CUDA runtime error";
        case HOS_E_UNSUPPORTED: return "shape outside the supported limits";
        case HOS_E_TOO_LARGE: return "batch exceeds the built-in scratch of hos_lower_bound_static";
        default: return "unknown error code";
    }
}

}  // extern "C"
