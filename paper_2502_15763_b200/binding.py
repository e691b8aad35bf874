"""ctypes binding of libhos.so: same names as the C entry points, argument marshalling only.

Every array argument is a torch CUDA tensor (torch supplies device memory and
the current stream); every result is a torch CUDA tensor.  Structured results
are returned as uint8 tensors of shape [..., sizeof(struct)] whose host copy can
be viewed with the numpy dtypes below (`view_struct`).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))

HOS_QUEUE_SORTED, HOS_QUEUE_FCFS = 0, 1
HOS_ST_LIMIT, HOS_ST_TRACE, HOS_ST_INVALID, HOS_ST_RANGE = 1, 2, 4, 8

LS_MOVE_DTYPE = np.dtype([("i", "<i4"), ("u", "<i4"), ("k", "<i4"), ("v", "<i8")], align=True)
LB_DTYPE = np.dtype([(n, "<i8") for n in ("lb_pack", "sum_T", "max_T", "pair_T", "lb_sim_us",
                                           "tp_star_us", "td_star_us", "chain_us", "tp_paper_us")])
CLIENT_RESULT_DTYPE = np.dtype([("makespan_us", "<i8"), ("busy_slot_us", "<i8"),
                                ("n_prefill_iters", "<u4"), ("n_decode_iters", "<u4"),
                                ("trace_hash", "<u8"), ("utilisation", "<f8")])
SIM_RESULT_DTYPE = np.dtype([("makespan_us", "<i8"), ("busy_slot_us", "<i8"),
                             ("utilisation", "<f8"), ("tokens_per_s", "<f8")])
ITER_REC_DTYPE = np.dtype([("dur_us", "<u4"), ("kind_n", "<u4"), ("tokens", "<u4"), ("aux", "<u4")])

_SYMBOLS = ("hos_offline_pack", "hos_local_search", "hos_lower_bound", "hos_online_simulate",
            "hos_trace_offsets", "hos_offline_workspace_bytes", "hos_lower_bound_workspace_bytes",
            "hos_online_workspace_bytes", "hos_strerror", "hos_set_launch_hook",
            "hos_lower_bound_static", "hos_trace_fill", "hos_online_simulate_steal",
            "hos_offline_pack_multifit", "hos_debug_bounds_violations", "hos_offline_multifit_workspace_bytes")

LAUNCH_HOOK = C.CFUNCTYPE(None, C.c_char_p, C.c_int, C.c_void_p, C.c_void_p)


class HosError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {hos_strerror(code)} ({code})")


class _CostModel(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in (
        "prefill_fixed_us", "prefill_per_token_us", "decode_fixed_us", "decode_per_seq_us",
        "decode_kv_div", "est_per_prompt_token", "est_per_output_token", "n_levels")] + [
        ("level_cap_tokens", C.c_uint32 * 8), ("level_time_us", C.c_uint32 * 8)]


class _Batch(C.Structure):
    _fields_ = [("n_inst", C.c_int32), ("n_req", C.c_int32), ("n_clients", C.c_int32),
                ("batch_cap", C.c_int32), ("kv_budget", C.c_int64),
                ("p", C.c_void_p), ("o", C.c_void_p), ("o_est", C.c_void_p),
                ("kv_reserve_tokens", C.c_uint32)]


_lib = None


def lib_path() -> str:
    return os.path.join(_PKG, "libhos.so")


def lib():
    """Load libhos.so (building it first if the sources are newer).  Raises if it cannot be had.
    With HOS_LIB_VARIANT=debug in the environment the bounds-checked build libhos_debug.so is
    loaded instead (see hos_debug_bounds_violations)."""
    global _lib
    if _lib is None:
        from . import _build
        debug = os.environ.get("HOS_LIB_VARIANT", "") == "debug"
        path = _build.build(debug=debug)
        L = C.CDLL(path)
        L.hos_debug_bounds_violations.restype = C.c_longlong
        for name in ("hos_offline_workspace_bytes", "hos_lower_bound_workspace_bytes",
                     "hos_online_workspace_bytes", "hos_offline_multifit_workspace_bytes"):
            getattr(L, name).restype = C.c_size_t
        L.hos_strerror.restype = C.c_char_p
        for name in ("hos_offline_pack", "hos_local_search", "hos_lower_bound",
                     "hos_online_simulate", "hos_trace_offsets", "hos_lower_bound_static", "hos_trace_fill",
                     "hos_online_simulate_steal", "hos_offline_pack_multifit"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def hos_set_launch_hook(fn):
    """fn(kernel_name: bytes, phase: int, stream: int, user) around every kernel launch; None removes it.

    Returns the ctypes callback object, which the caller must keep alive while it is set."""
    L = lib()
    if fn is None:
        L.hos_set_launch_hook(None, None)
        return None
    cb = LAUNCH_HOOK(fn)
    L.hos_set_launch_hook(cb, None)
    return cb


def hos_debug_bounds_violations():
    """(count, (site, index, limit) of the first) out-of-range indexes caught by the bounds-checked
    build on the current device since it was loaded; count is -1 in the ordinary build."""
    first = (C.c_longlong * 3)()
    n = lib().hos_debug_bounds_violations(first)
    return int(n), tuple(int(x) for x in first)


def exported_symbols() -> Sequence[str]:
    return _SYMBOLS


def hos_strerror(code: int) -> str:
    return lib().hos_strerror(C.c_int(code)).decode()


def _torch():
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("paper_2502_15763_b200 needs a CUDA device; there is no CPU fallback")
    return torch


def _dev(t, dtype, what: str):
    torch = _torch()
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{what}: expected a contiguous CUDA tensor of {dtype}")
    return t


def _ptr(t) -> C.c_void_p:
    return C.c_void_p(t.data_ptr() if t is not None else None)


def _stream():
    return C.c_void_p(_torch().cuda.current_stream().cuda_stream)


def _batch(p, o, n_clients: int, batch_cap: int, kv_budget: int, o_est=None, kv_reserve: int = 0) -> _Batch:
    """o_est: optional table of estimated output lengths (same shape as o); kv_reserve: KV tokens
    every request reserves (required with o_est), 0 = p + o."""
    torch = _torch()
    # uint32 tables travel as int32 tensors (same bits)
    p = _dev(p, torch.int32, "p")
    o = _dev(o, torch.int32, "o")
    if p.dim() != 2 or p.shape != o.shape:
        raise ValueError("p and o must be [n_inst][n_req] tables of the same shape")
    if o_est is not None:
        o_est = _dev(o_est, torch.int32, "o_est")
        if o_est.shape != o.shape:
            raise ValueError("o_est must have the shape of o")
    return _Batch(p.shape[0], p.shape[1], n_clients, batch_cap, kv_budget, p.data_ptr(), o.data_ptr(),
                  o_est.data_ptr() if o_est is not None else None, int(kv_reserve))


def _cost(cm: Sequence) -> _CostModel:
    """cm: the seven coefficients, optionally followed by the prefill levels ((cap_tokens, time_us), ...)."""
    c = _CostModel(*[int(x) for x in cm[:7]])
    levels = list(cm[7]) if len(cm) > 7 else []
    if len(levels) > 8:
        raise ValueError("at most 8 prefill levels")
    c.n_levels = len(levels)
    for l, (cap_tokens, time_us) in enumerate(levels):
        c.level_cap_tokens[l] = int(cap_tokens)
        c.level_time_us[l] = int(time_us)
    return c


def _workspace(nbytes: int, like):
    torch = _torch()
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=like.device)


def _check(rc: int, where: str):
    if rc != 0:
        raise HosError(rc, where)


def view_struct(t, dtype: np.dtype) -> np.ndarray:
    """Host copy of a [..., sizeof] uint8 result tensor viewed as a structured numpy array."""
    a = t.detach().cpu().numpy()
    return a.view(dtype).reshape(a.shape[:-1])


def hos_offline_pack(p, o, n_clients: int, batch_cap: int, kv_budget: int, cost_model, ls_rounds: int = 0,
                     want_log: bool = False, ws=None, out=None, want_lb: bool = False, o_est=None, kv_reserve: int = 0,
                     multifit_steps: int = 0):
    """Eq. 26-30: estimate, order, LPT, `ls_rounds` local-search rounds.  Returns a dict of tensors.

    multifit_steps > 0 calls hos_offline_pack_multifit instead (MULTIFIT packing kept where it beats
    the list schedule) and adds 'packer' (int32 [n_inst]) to the result.

    out: optional dict with preallocated 'assign', 'load', 'makespan_est', 'rounds_applied', 'status'
    (for instance row slices of larger tensors) to write into instead of new tensors, optionally 'lb'.
    want_lb: also return the lower bounds (uint8 [n_inst][64]) computed from the same sort."""
    torch = _torch()
    b = _batch(p, o, n_clients, batch_cap, kv_budget, o_est, kv_reserve)
    cm = _cost(cost_model)
    L = lib()
    need = (L.hos_offline_multifit_workspace_bytes(C.byref(b), C.c_int(ls_rounds)) if multifit_steps > 0
            else L.hos_offline_workspace_bytes(C.byref(b), C.c_int(1), C.c_int(ls_rounds)))
    ws = ws if ws is not None and ws.numel() >= need else _workspace(need, p)
    dev = p.device
    if out is not None:
        assign = _dev(out["assign"], torch.int32, "out.assign")
        load = _dev(out["load"], torch.int64, "out.load")
        makespan = _dev(out["makespan_est"], torch.int64, "out.makespan_est")
        applied = _dev(out["rounds_applied"], torch.int32, "out.rounds_applied")
        status = _dev(out["status"], torch.int32, "out.status")
        if (tuple(assign.shape) != (b.n_inst, b.n_req) or tuple(load.shape) != (b.n_inst, n_clients)
                or makespan.numel() != b.n_inst or applied.numel() != b.n_inst or status.numel() != b.n_inst):
            raise ValueError("out tensors do not match the batch")
    else:
        assign = torch.empty((b.n_inst, b.n_req), dtype=torch.int32, device=dev)
        load = torch.empty((b.n_inst, n_clients), dtype=torch.int64, device=dev)
        makespan = torch.empty((b.n_inst,), dtype=torch.int64, device=dev)
        applied = torch.empty((b.n_inst,), dtype=torch.int32, device=dev)
        status = torch.empty((b.n_inst,), dtype=torch.int32, device=dev)
    log = (torch.empty((b.n_inst, ls_rounds, LS_MOVE_DTYPE.itemsize), dtype=torch.uint8, device=dev)
           if want_log and ls_rounds > 0 else None)
    lb = None
    if out is not None and out.get("lb") is not None:
        lb = _dev(out["lb"], torch.uint8, "out.lb")
    elif want_lb:
        lb = torch.empty((b.n_inst, LB_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    packer = None
    if multifit_steps > 0:
        packer = torch.empty((b.n_inst,), dtype=torch.int32, device=dev)
        rc = L.hos_offline_pack_multifit(C.byref(b), C.byref(cm), C.c_int(multifit_steps), C.c_int(ls_rounds),
                                         _ptr(assign), _ptr(load), _ptr(makespan), _ptr(applied), _ptr(log),
                                         _ptr(lb), _ptr(status), _ptr(packer), _ptr(ws), C.c_size_t(ws.numel()),
                                         _stream())
        _check(rc, "hos_offline_pack_multifit")
    else:
        rc = L.hos_offline_pack(C.byref(b), C.byref(cm), C.c_int(ls_rounds), _ptr(assign), _ptr(load),
                                _ptr(makespan), _ptr(applied), _ptr(log), _ptr(lb), _ptr(status), _ptr(ws),
                                C.c_size_t(ws.numel()), _stream())
        _check(rc, "hos_offline_pack")
    return dict(assign=assign, load=load, makespan_est=makespan, rounds_applied=applied, ls_log=log,
                lb=lb, status=status, packer=packer)


def hos_local_search(p, o, n_clients: int, batch_cap: int, kv_budget: int, cost_model, assign,
                     ls_rounds: int, want_log: bool = False, ws=None, o_est=None, kv_reserve: int = 0):
    """Local-search rounds from given assignments [n_inst][n_copies][n_req] (modified in place)."""
    torch = _torch()
    b = _batch(p, o, n_clients, batch_cap, kv_budget, o_est, kv_reserve)
    cm = _cost(cost_model)
    assign = _dev(assign, torch.int32, "assign")
    if assign.dim() != 3 or assign.shape[0] != b.n_inst or assign.shape[2] != b.n_req:
        raise ValueError("assign must be [n_inst][n_copies][n_req]")
    n_copies = assign.shape[1]
    L = lib()
    need = L.hos_offline_workspace_bytes(C.byref(b), C.c_int(n_copies), C.c_int(ls_rounds))
    ws = ws if ws is not None else _workspace(need, p)
    dev = p.device
    load = torch.empty((b.n_inst, n_copies, n_clients), dtype=torch.int64, device=dev)
    makespan = torch.empty((b.n_inst, n_copies), dtype=torch.int64, device=dev)
    applied = torch.empty((b.n_inst, n_copies), dtype=torch.int32, device=dev)
    status = torch.empty((b.n_inst,), dtype=torch.int32, device=dev)
    log = (torch.empty((b.n_inst, n_copies, ls_rounds, LS_MOVE_DTYPE.itemsize), dtype=torch.uint8, device=dev)
           if want_log and ls_rounds > 0 else None)
    rc = L.hos_local_search(C.byref(b), C.byref(cm), C.c_int(n_copies), C.c_int(ls_rounds), _ptr(assign),
                            _ptr(load), _ptr(makespan), _ptr(applied), _ptr(log), _ptr(status), _ptr(ws),
                            C.c_size_t(ws.numel()), _stream())
    _check(rc, "hos_local_search")
    return dict(assign=assign, load=load, makespan_est=makespan, rounds_applied=applied, ls_log=log,
                status=status)


def hos_lower_bound(p, o, n_clients: int, batch_cap: int, kv_budget: int, cost_model, ws=None, o_est=None, kv_reserve: int = 0):
    """Eq. 31-32 and the packing relaxations; returns {'lb': uint8 [n_inst][64], 'status': ...}."""
    torch = _torch()
    b = _batch(p, o, n_clients, batch_cap, kv_budget, o_est, kv_reserve)
    cm = _cost(cost_model)
    L = lib()
    need = L.hos_lower_bound_workspace_bytes(C.byref(b))
    ws = ws if ws is not None else _workspace(need, p)
    out = torch.empty((b.n_inst, LB_DTYPE.itemsize), dtype=torch.uint8, device=p.device)
    status = torch.empty((b.n_inst,), dtype=torch.int32, device=p.device)
    rc = L.hos_lower_bound(C.byref(b), C.byref(cm), _ptr(out), _ptr(status), _ptr(ws),
                           C.c_size_t(ws.numel()), _stream())
    _check(rc, "hos_lower_bound")
    return dict(lb=out, status=status)


def hos_lower_bound_static(p, o, n_clients: int, batch_cap: int, kv_budget: int, cost_model, o_est=None, kv_reserve: int = 0):
    """hos_lower_bound without a caller workspace: for code that may not allocate device memory
    (the scratch is a fixed array inside the library; batches beyond it raise HosError -5).
    The result tensors here are the caller's outputs; the C call itself allocates nothing."""
    torch = _torch()
    b = _batch(p, o, n_clients, batch_cap, kv_budget, o_est, kv_reserve)
    cm = _cost(cost_model)
    out = torch.empty((b.n_inst, LB_DTYPE.itemsize), dtype=torch.uint8, device=p.device)
    status = torch.empty((b.n_inst,), dtype=torch.int32, device=p.device)
    rc = lib().hos_lower_bound_static(C.byref(b), C.byref(cm), _ptr(out), _ptr(status), _stream())
    _check(rc, "hos_lower_bound_static")
    return dict(lb=out, status=status)


def hos_trace_offsets(cres, n_units: Optional[int] = None):
    """Exclusive scan of the per-client iteration counts -> int64 [n_units + 1]."""
    torch = _torch()
    cres = _dev(cres, torch.uint8, "cres")
    n = int(cres.numel() // CLIENT_RESULT_DTYPE.itemsize) if n_units is None else int(n_units)
    off = torch.empty((n + 1,), dtype=torch.int64, device=cres.device)
    _check(lib().hos_trace_offsets(_ptr(cres), C.c_int64(n), _ptr(off), _stream()), "hos_trace_offsets")
    return off


def hos_online_simulate(p, o, n_clients: int, batch_cap: int, kv_budget: int, cost_model, assign,
                        lambda_q16, queue_order: int = HOS_QUEUE_SORTED, max_iters: int = 0x7FFFFFFF,
                        trace=None, trace_off=None, keep_events: bool = False, ws=None, o_est=None, kv_reserve: int = 0):
    """Queues + iteration simulation for every (instance, multiplier, client).

    trace: None, or a uint8 tensor [n_records][16] with trace_off (int64 [n_units + 1]).
    keep_events: leave the event log in the returned workspace `ws` for hos_trace_fill.
    """
    torch = _torch()
    b = _batch(p, o, n_clients, batch_cap, kv_budget, o_est, kv_reserve)
    cm = _cost(cost_model)
    assign = _dev(assign, torch.int32, "assign")
    if tuple(assign.shape) != (b.n_inst, b.n_req):
        raise ValueError("assign must be [n_inst][n_req]")
    lambda_q16 = _dev(lambda_q16, torch.int32, "lambda_q16")       # uint32 bits
    n_lambda = int(lambda_q16.numel())
    L = lib()
    need = L.hos_online_workspace_bytes(C.byref(b), C.c_int(n_lambda), C.c_int(int(keep_events)))
    ws = ws if ws is not None else _workspace(need, p)
    dev = p.device
    cres = torch.empty((b.n_inst, n_lambda, n_clients, CLIENT_RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    sres = torch.empty((b.n_inst, n_lambda, SIM_RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    status = torch.empty((b.n_inst, n_lambda, n_clients), dtype=torch.int32, device=dev)
    if trace is not None:
        trace = _dev(trace, torch.uint8, "trace")
        trace_off = _dev(trace_off, torch.int64, "trace_off")
        if trace_off.numel() != b.n_inst * n_lambda * n_clients + 1:
            raise ValueError("trace_off must have n_units + 1 entries")
    rc = L.hos_online_simulate(C.byref(b), _ptr(assign), C.byref(cm), _ptr(lambda_q16), C.c_int(n_lambda),
                               C.c_int(queue_order), C.c_uint32(max_iters), _ptr(cres), _ptr(sres),
                               _ptr(trace), _ptr(trace_off), _ptr(status), C.c_int(int(keep_events)), _ptr(ws),
                               C.c_size_t(ws.numel()), _stream())
    _check(rc, "hos_online_simulate")
    return dict(cres=cres, sres=sres, status=status, ws=ws)


def hos_online_simulate_steal(p, o, n_clients: int, batch_cap: int, kv_budget: int, cost_model, assign,
                              lambda_q16, queue_order: int = HOS_QUEUE_SORTED, max_iters: int = 0x7FFFFFFF,
                              trace=None, trace_off=None, want_served_by: bool = False, keep_events: bool = False,
                              ws=None, o_est=None, kv_reserve: int = 0):
    """hos_online_simulate with Algorithm 1's request stealing between the clients of an instance.

    keep_events: leave the event log in the returned workspace `ws` for hos_trace_fill.
    """
    torch = _torch()
    b = _batch(p, o, n_clients, batch_cap, kv_budget, o_est, kv_reserve)
    cm = _cost(cost_model)
    assign = _dev(assign, torch.int32, "assign")
    if tuple(assign.shape) != (b.n_inst, b.n_req):
        raise ValueError("assign must be [n_inst][n_req]")
    lambda_q16 = _dev(lambda_q16, torch.int32, "lambda_q16")
    n_lambda = int(lambda_q16.numel())
    L = lib()
    need = L.hos_online_workspace_bytes(C.byref(b), C.c_int(n_lambda), C.c_int(int(keep_events)))
    ws = ws if ws is not None else _workspace(need, p)
    dev = p.device
    cres = torch.empty((b.n_inst, n_lambda, n_clients, CLIENT_RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    sres = torch.empty((b.n_inst, n_lambda, SIM_RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    status = torch.empty((b.n_inst, n_lambda, n_clients), dtype=torch.int32, device=dev)
    served = torch.empty((b.n_inst, n_lambda, b.n_req), dtype=torch.int32, device=dev) if want_served_by else None
    if trace is not None:
        trace = _dev(trace, torch.uint8, "trace")
        trace_off = _dev(trace_off, torch.int64, "trace_off")
        if trace_off.numel() != b.n_inst * n_lambda * n_clients + 1:
            raise ValueError("trace_off must have n_units + 1 entries")
    rc = L.hos_online_simulate_steal(C.byref(b), _ptr(assign), C.byref(cm), _ptr(lambda_q16), C.c_int(n_lambda),
                                     C.c_int(queue_order), C.c_uint32(max_iters), _ptr(cres), _ptr(sres),
                                     _ptr(trace), _ptr(trace_off), _ptr(status), _ptr(served),
                                     C.c_int(int(keep_events)), _ptr(ws), C.c_size_t(ws.numel()), _stream())
    _check(rc, "hos_online_simulate_steal")
    return dict(cres=cres, sres=sres, status=status, served_by=served, ws=ws)


def hos_trace_fill(p, o, n_clients: int, batch_cap: int, kv_budget: int, cost_model, n_lambda: int,
                   sim, trace, trace_off, o_est=None, kv_reserve: int = 0):
    """The full iteration trace from the event log of `sim`, the dict returned by
    hos_online_simulate or hos_online_simulate_steal (..., keep_events=True) for the same batch.  ORs HOS_ST_TRACE into
    sim["status"] where the slots are too few.  Returns `trace`."""
    torch = _torch()
    b = _batch(p, o, n_clients, batch_cap, kv_budget, o_est, kv_reserve)
    cm = _cost(cost_model)
    trace = _dev(trace, torch.uint8, "trace")
    trace_off = _dev(trace_off, torch.int64, "trace_off")
    if trace_off.numel() != b.n_inst * n_lambda * n_clients + 1:
        raise ValueError("trace_off must have n_units + 1 entries")
    ws = sim["ws"]
    rc = lib().hos_trace_fill(C.byref(b), C.byref(cm), C.c_int(n_lambda), _ptr(sim["cres"]), _ptr(trace),
                              _ptr(trace_off), _ptr(sim["status"]), _ptr(ws), C.c_size_t(ws.numel()), _stream())
    _check(rc, "hos_trace_fill")
    return trace
