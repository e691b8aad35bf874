#!/usr/bin/env python
"""Benchmark of the batched scheduler evaluation (offline pack + lower bound + online simulation).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c0..c4] [--impl ours|reference]

One step is one pass of the whole path over one batch of synthetic instances:
hos_offline_pack (sort, lower bounds, LPT, local search) -> hos_online_simulate
(with its event log) -> hos_trace_offsets -> hos_trace_fill (the iteration trace).  Prints ONE JSON line.
With N > 1 (under torchrun) every rank runs the same number of instances with its own seeds
(weak scaling, no data-path collective); the time is the max over ranks.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workload import Workload, workload  # noqa: E402

METRIC = "instances/sec"
UNIT = "instances/s"
DTYPE = "int64"            # integer microseconds / Q16.16; utilisation is one f64 division
L2_FLUSH_BYTES = 256 << 20

# algorithmic bytes per unit of work of each kernel (what a streaming implementation of that
# step alone must move once); the estimate + sort kernel also carries the lower bounds' 64 B per instance
BYTES_PER_REQ = {"k_estimate_sort": 16, "k_lpt": 12, "k_queue_build": 16, "k_ls_lists": 15, "k_multifit": 9}
# What bounds each kernel (counters in profiles/).  "hbm": streaming, set against the measured copy
# bandwidth.  "alu": the iteration recurrence, integer operations of the method against the int32
# lanes.  "issue": dependent chains on data that stays on chip (DRAM idle); warp instructions
# issued against the schedulers' issue slots.
BOUND = {"k_simulate": "alu", "k_simulate_steal": "alu", "k_lpt": "issue", "k_local_search": "issue",
         "k_multifit": "issue"}
# integer operations of one simulated iteration as the method states it: duration (3), busy slot
# time (2), clock (1), waited decode time (2), sum of KV lengths (1), decision compare in Q16.16 (3),
# trace hash (9), counters (3)
INT_OPS_PER_ITERATION = 24
# Counters of one ncu capture (DRAM bytes and warp instructions per unit of work and kernel),
# written by paper_2502_15763_b200/profile_summary.py; ignored once the library sources changed.
NCU_COUNTERS = os.path.join(ROOT, "profiles", "ncu_counters_c4x296.json")


def ncu_counters():
    """(counters per kernel, shape of the captured workload, note): {} with the reason when the file
    is missing or stale."""
    try:
        doc = json.load(open(NCU_COUNTERS))
    except (OSError, ValueError):
        return {}, None, "no counter file"
    from paper_2502_15763_b200 import _build
    if doc.get("source_hash") != _build.source_hash():
        return {}, None, "kernels changed since the counters were taken"
    return doc.get("kernels", {}), doc.get("shape"), "ncu capture of " + doc.get("workload", "?")


def describe(w: Workload) -> str:
    return (f"{w.name}: {w.n_inst} instances x {w.n_req} requests, {w.n_clients} clients, batch cap "
            f"{w.batch_cap}, KV budget {w.kv_budget}, {len(w.lambdas_q16)} multiplier value(s), "
            f"{w.ls_rounds} local-search rounds")


def rank_workload(name: str, rank: int, instances: int = 0) -> Workload:
    """Rank r evaluates the same number of instances with seeds shifted by r * n_inst."""
    w = workload(name)
    if instances > 0:
        w = w.subset(0, min(instances, w.n_inst))
    if rank == 0:
        return w
    seeds = tuple(s + rank * w.n_inst for s in w.seeds)
    return Workload(w.name, seeds, w.n_req, w.n_clients, w.batch_cap, w.kv_budget, w.dist_p, w.dist_o,
                    w.lambdas_q16, w.ls_rounds, w.cost_model, w.est_sigma, w.kv_reserve)


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.monotonic(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        """Median SM clock and the throttle reasons seen between t0 and t1 (time.monotonic() around the
        timed steps); the sampler runs from before the warm-up steps, and a timed region too short for
        a sample of its own reports the samples taken under the same load since the warm-up began."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        inside = [r for ts, r in self.rows if t0 <= ts <= t1]
        window = "timed steps" if inside else "warm-up and timed steps"
        for row in (inside or [r for _, r in self.rows]):
            parts = [x.strip() for x in row.split(",")]
            if len(parts) != 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "window": window, "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
class Pipeline:
    """Device buffers of one workload and the step that runs the whole path through the C ABI."""

    def __init__(self, w: Workload, device):
        import torch
        import paper_2502_15763_b200 as hos
        self.torch, self.hos, self.w, self.dev = torch, hos, w, device
        p, o = w.lengths()
        self.p_host = torch.from_numpy(p.view(np.int32)).pin_memory()
        self.o_host = torch.from_numpy(o.view(np.int32)).pin_memory()
        self.lam_host = torch.from_numpy(np.asarray(w.lambdas_q16, dtype=np.uint32).view(np.int32)).pin_memory()
        self.p = self.p_host.to(device)
        self.o = self.o_host.to(device)
        est = w.estimates()                  # None unless the workload schedules on estimated lengths
        self.est_host = None if est is None else torch.from_numpy(est.view(np.int32)).pin_memory()
        self.est = None if est is None else self.est_host.to(device)
        self.kw = dict(o_est=self.est, kv_reserve=w.kv_reserve)
        self.lam = self.lam_host.to(device)
        self.ws_off = None
        self.ws_on = None
        self.trace = None
        self.out = None
        self.n_iters = 0
        self.up = None
        self.down = None
        self.sets = None
        self.trace_free = None
        self.trace_host = None

    def tables(self):
        return dict(p=self.p, o=self.o, est=self.est, lam=self.lam)

    def args(self, t=None):
        w = self.w
        t = t or self.tables()
        return (t["p"], t["o"], w.n_clients, w.batch_cap, w.kv_budget, w.cost_model)

    def offline(self, t=None):
        hos, w = self.hos, self.w
        t = t or self.tables()
        sweep = len(w.lambdas_q16) > 1
        # a multiplier sweep runs its local-search rounds per (instance, multiplier) copy, in online()
        return hos.hos_offline_pack(*self.args(t), 0 if sweep else w.ls_rounds, ws=self.ws_off, want_lb=True,
                                    o_est=t["est"], kv_reserve=w.kv_reserve)

    def step(self, t=None):
        return self.online(self.offline(t), t)

    def prepare(self):
        """Workspaces (allocated once; the library itself allocates nothing)."""
        import ctypes as C
        from paper_2502_15763_b200 import binding as B
        b = B._batch(*self.args()[:5], self.est, self.w.kv_reserve)
        L = self.hos.lib()
        n_off = L.hos_offline_workspace_bytes(C.byref(b), len(self.w.lambdas_q16), self.w.ls_rounds)
        n_on = L.hos_online_workspace_bytes(C.byref(b), len(self.w.lambdas_q16), 1)
        self.ws_off = self.torch.empty(n_off, dtype=self.torch.uint8, device=self.dev)
        self.ws_on = self.torch.empty(n_on, dtype=self.torch.uint8, device=self.dev)

    def online(self, pk, t=None):
        """Lower bound, simulation with event log, trace offsets, trace (and the sweep's local search)."""
        hos, w = self.hos, self.w
        t = t or self.tables()
        kw = dict(o_est=t["est"], kv_reserve=w.kv_reserve)
        lb = dict(lb=pk["lb"])                      # Eq. 31-32 bounds, computed inside hos_offline_pack
        s1 = hos.hos_online_simulate(*self.args(t), pk["assign"], t["lam"], hos.HOS_QUEUE_SORTED,
                                     keep_events=True, ws=self.ws_on, **kw)
        off = hos.hos_trace_offsets(s1["cres"])
        if self.trace is None:                      # first (warm-up) step sizes the trace buffer
            self.n_iters = int(off[-1].item())
            self.trace = self.torch.empty((max(self.n_iters, 1), 16), dtype=self.torch.uint8, device=self.dev)
        if self.trace_free is not None:             # the last step's trace is still on its way to the host
            self.torch.cuda.current_stream().wait_event(self.trace_free)
        hos.hos_trace_fill(*self.args(t), len(w.lambdas_q16), s1, self.trace, off, **kw)
        self.out = dict(pk=pk, lb=lb, sim=s1, off=off)
        if len(w.lambdas_q16) > 1 and w.ls_rounds > 0:
            copies = pk["assign"][:, None, :].expand(-1, len(w.lambdas_q16), -1).contiguous()
            self.out["ls"] = hos.hos_local_search(*self.args(t), copies, w.ls_rounds, ws=self.ws_off, **kw)
        return self.out

    @staticmethod
    def results(r):
        """What a step hands back to the host: assignment, loads, estimate, status, bounds, client and
        simulation results (the iteration trace stays on the device)."""
        pk, sim = r["pk"], r["sim"]
        return (pk["assign"], pk["load"], pk["makespan_est"], pk["status"], r["lb"]["lb"],
                sim["cres"], sim["sres"], sim["status"])

    def e2e_run(self, steps, host_out, flush, with_trace=False):
        """`steps` steps from pinned host tables to pinned host results, as a stream of batches.

        Every step uploads its own tables and downloads its own results.  There are two sets of device
        tables: while step k computes, the tables of step k+1 go up and results go down (separate
        streams, both copy directions at once; the offline results of step k already while its online
        part runs).  Returns the device time from the start of
        the first upload to the end of the last download (ms) and the bytes per step each way."""
        torch = self.torch
        main = torch.cuda.current_stream()
        if self.up is None:
            self.up, self.down = torch.cuda.Stream(), torch.cuda.Stream()
            spare = {k: (None if v is None else torch.empty_like(v)) for k, v in self.tables().items()}
            self.sets = [self.tables(), spare]
        host = dict(p=self.p_host, o=self.o_host, est=self.est_host, lam=self.lam_host)
        read = [None, None]                         # the step that last read a set of tables has finished
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(main)
        self.up.wait_stream(main)
        self.down.wait_stream(main)
        for k in range(steps):
            t = self.sets[k & 1]
            with torch.cuda.stream(self.up):
                if read[k & 1] is not None:
                    self.up.wait_event(read[k & 1])
                for name, h in host.items():
                    if h is not None:
                        t[name].copy_(h, non_blocking=True)
                arrived = torch.cuda.Event()
                arrived.record(self.up)
            main.wait_event(arrived)
            if flush is not None:
                flush.fill_(1)
            pk = self.offline(t)
            packed = torch.cuda.Event()
            packed.record(main)
            res = self.results(self.online(pk, t))
            done = torch.cuda.Event()
            done.record(main)
            read[k & 1] = done
            if not host_out:                        # first call: learn the result shapes
                host_out.extend(torch.empty(d.shape, dtype=d.dtype).pin_memory() for d in res)
            n_early = 5                             # the offline results go down while the online part runs
            with torch.cuda.stream(self.down):
                for i, (h, d) in enumerate(zip(host_out, res)):
                    if i == 0:
                        self.down.wait_event(packed)
                    if i == n_early:
                        self.down.wait_event(done)
                    h.copy_(d, non_blocking=True)
                    d.record_stream(self.down)      # the allocator must not hand it out again before the copy ends
                if with_trace:                      # the iteration trace too: the next fill waits for this copy
                    if self.trace_host is None:
                        self.trace_host = torch.empty(self.trace.shape, dtype=torch.uint8).pin_memory()
                    self.trace_host.copy_(self.trace, non_blocking=True)
                    self.trace_free = torch.cuda.Event()
                    self.trace_free.record(self.down)
        main.wait_stream(self.down)
        main.wait_stream(self.up)
        end.record(main)
        torch.cuda.synchronize()
        self.trace_free = None
        h2d = sum(h.numel() * h.element_size() for h in host.values() if h is not None)
        d2h = sum(h.numel() * h.element_size() for h in host_out)
        if with_trace:
            d2h += self.trace_host.numel()
        return start.elapsed_time(end), h2d, d2h


def timed_steps(torch, fn, steps, flush):
    """Sum of per-step CUDA-event times (ms); L2 is flushed between steps outside the timed spans."""
    spans = []
    for _ in range(steps):
        if flush is not None:
            flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        spans.append((a, b))
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in spans)


def kernel_profile(torch, hos, pipe, steps, flush):
    """Per-kernel device time from CUDA events recorded by the library's launch hook."""
    events = []

    def hook(name, phase, stream, user):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()                                  # the binding launches on torch's current stream
        events.append((name.decode(), phase, ev))

    cb = hos.hos_set_launch_hook(hook)
    try:
        for _ in range(steps):
            if flush is not None:
                flush.fill_(1)
            pipe.step()
        torch.cuda.synchronize()
    finally:
        hos.hos_set_launch_hook(None)
    del cb
    table, order, pending = {}, [], {}
    for name, phase, ev in events:
        if phase == 0:
            pending[name] = ev
        else:
            ms = pending.pop(name).elapsed_time(ev)
            if name not in table:
                table[name] = [0, 0.0]
                order.append(name)
            table[name][0] += 1
            table[name][1] += ms
    return {n: {"launches_per_step": table[n][0] / steps, "ms_per_launch": table[n][1] / table[n][0]}
            for n in order}


def algorithmic_bytes(w: Workload, name: str, pipe) -> float:
    """Bytes one launch of `name` must move at least (see the design notes for the per-unit figures)."""
    n_req_total = w.n_inst * w.n_req
    if name in BYTES_PER_REQ:
        extra = 64 * w.n_inst if name == "k_estimate_sort" else 0
        copies = len(w.lambdas_q16) if name == "k_ls_lists" and len(w.lambdas_q16) > 1 else 1
        return BYTES_PER_REQ[name] * n_req_total * copies + extra
    if name == "k_local_search":
        return float(executed_rounds(w, pipe)) * (8 * w.n_req + 8 * w.n_clients)
    if name == "k_simulate":
        n_sims = w.n_inst * len(w.lambdas_q16)
        # reads the queue entries, writes the client results
        return 8.0 * w.n_req * n_sims + 48.0 * n_sims * w.n_clients
    if name == "k_trace_fill":
        return 16.0 * pipe.n_iters
    if name == "k_finalize":
        return 40.0 * w.n_inst * len(w.lambdas_q16) * w.n_clients
    if name == "k_trace_offsets":
        return 48.0 * w.n_inst * len(w.lambdas_q16) * w.n_clients
    return 0.0


def executed_rounds(w: Workload, pipe) -> int:
    """Local-search rounds that were evaluated in the last step (the round that finds nothing counts)."""
    src = pipe.out.get("ls") or pipe.out["pk"]
    if w.ls_rounds <= 0:
        return 0
    applied = src["rounds_applied"].to("cpu").numpy().astype(np.int64)
    return int(np.minimum(applied + 1, w.ls_rounds).sum())


# Shortest a local-search round can be with its phases in sequence and nothing else on the SM
# (cycles; the derivation is in the design notes): copy of the critical list (one global round
# trip, ~600), nine dependent shared-memory probes (~270), evaluation of both neighbours (~100),
# two CTA-wide minima with a barrier between (~300), load update and next extremes (~300), list
# patch by search and shift (~550), two barriers (~100).
LS_ROUND_MIN_CYCLES = 2200


def input_sha256(pipe) -> str:
    """SHA-256 of the request tables this rank evaluates (p, o and, if used, the estimates)."""
    import hashlib
    h = hashlib.sha256()
    for t in (pipe.p_host, pipe.o_host, pipe.est_host):
        if t is not None:
            h.update(t.numpy().tobytes())
    return h.hexdigest()


def struct_view(t, dtype):
    from paper_2502_15763_b200.binding import view_struct
    return view_struct(t, dtype)


def study_report(hos, pipe, w: Workload) -> dict:
    """The 100-case study (Section "Numerical experiment"): hybrid scheduling (longest-first packing,
    queues sorted by length, multiplier 1.0) against the two baselines (requests dealt round-robin
    in arrival order, first-come-first-served queues; prefill-first, and never preempting a decode)."""
    import torch
    from workload import LAMBDA_NEVER_PREEMPT, LAMBDA_ONE, LAMBDA_PREFILL_FIRST
    args = pipe.args()
    pk = hos.hos_offline_pack(*args, w.ls_rounds, want_lb=True, **pipe.kw)
    lam = lambda *v: torch.from_numpy(np.asarray(v, dtype=np.uint32).view(np.int32)).to(pipe.dev)
    hyb = hos.hos_online_simulate(*args, pk["assign"], lam(LAMBDA_ONE), hos.HOS_QUEUE_SORTED, **pipe.kw)
    rr = (torch.arange(w.n_req, dtype=torch.int32, device=pipe.dev) % w.n_clients)[None, :].repeat(w.n_inst, 1).contiguous()
    base = hos.hos_online_simulate(*args, rr, lam(LAMBDA_PREFILL_FIRST, LAMBDA_NEVER_PREEMPT), hos.HOS_QUEUE_FCFS,
                                   **pipe.kw)
    h = struct_view(hyb["sres"], hos.SIM_RESULT_DTYPE)[:, 0]
    b = struct_view(base["sres"], hos.SIM_RESULT_DTYPE)
    lb = struct_view(pk["lb"], hos.LB_DTYPE)
    uh, up, un = h["utilisation"], b["utilisation"][:, 0], b["utilisation"][:, 1]
    r4 = lambda a: [round(float(x), 4) for x in a]
    return {
        "instances": w.n_inst,
        "mean_utilisation": {"hybrid": float(uh.mean()), "fcfs_prefill_first": float(up.mean()),
                             "fcfs_never_preempt": float(un.mean())},
        "mean_makespan_s": {"hybrid": float(h["makespan_us"].mean()) / 1e6,
                            "fcfs_prefill_first": float(b["makespan_us"][:, 0].mean()) / 1e6,
                            "fcfs_never_preempt": float(b["makespan_us"][:, 1].mean()) / 1e6,
                            "lower_bound": float(lb["lb_sim_us"].mean()) / 1e6},
        "gain_vs_prefill_first": {"percentage_points": float((uh - up).mean() * 100), "ratio": float((uh / up).mean()),
                                  "instances_improved": int((uh > up).sum())},
        "gain_vs_never_preempt": {"percentage_points": float((uh - un).mean() * 100), "ratio": float((uh / un).mean()),
                                  "instances_improved": int((uh > un).sum())},
        "tokens_per_s_gain_vs_prefill_first": float((h["tokens_per_s"] - b["tokens_per_s"][:, 0]).mean()),
        "paper_context": "the paper's own 100-case study on its data reports +8.0 % utilisation and +100.63 tokens/s",
        "per_instance": {"utilisation_hybrid": r4(uh), "utilisation_fcfs_prefill_first": r4(up),
                         "utilisation_fcfs_never_preempt": r4(un),
                         "makespan_over_lower_bound": r4(h["makespan_us"] / lb["lb_sim_us"])},
    }


def sweep_report(torch, hos, pipe, w: Workload, flush) -> dict:
    """The multiplier sweep's local search both ways: one private copy of the packing per (instance,
    multiplier), as the workload states it, and once per instance (the copies agree bit for bit)."""
    pk = pipe.out["pk"]
    nl = len(w.lambdas_q16)
    copies = pk["assign"][:, None, :].expand(-1, nl, -1).contiguous()
    one = pk["assign"][:, None, :].contiguous()
    run_all = lambda: hos.hos_local_search(*pipe.args(), copies.clone(), w.ls_rounds, ws=pipe.ws_off, **pipe.kw)
    run_one = lambda: hos.hos_local_search(*pipe.args(), one.clone(), w.ls_rounds, ws=pipe.ws_off, **pipe.kw)
    run_all(); run_one()
    torch.cuda.synchronize()
    ms_all = timed_steps(torch, run_all, 5, flush) / 5
    ms_one = timed_steps(torch, run_one, 5, flush) / 5
    return {"as_executed": {"searches": w.n_inst * nl, "rounds_each": w.ls_rounds, "ms": ms_all,
                            "rounds_per_s": w.n_inst * nl * w.ls_rounds / (ms_all * 1e-3)},
            "deduplicated": {"searches": w.n_inst, "rounds_each": w.ls_rounds, "ms": ms_one,
                             "rounds_per_s": w.n_inst * w.ls_rounds / (ms_one * 1e-3)},
            "note": "times include the clone of the assignments and the sort that hos_local_search does itself"}


def packing_gap_report(torch, hos, pipe, w: Workload, flush) -> dict:
    """makespan_est - lb_pack with the list schedule and with MULTIFIT before the same local search."""
    rounds = w.ls_rounds if len(w.lambdas_q16) == 1 else 0
    out = {}
    for key, steps in (("lpt", 0), ("multifit", 64)):
        run = lambda: hos.hos_offline_pack(*pipe.args(), rounds, ws=pipe.ws_off, want_lb=True, multifit_steps=steps,
                                           **pipe.kw)
        r = run()
        torch.cuda.synchronize()
        ms_ = timed_steps(torch, run, 3, flush) / 3
        lb = struct_view(r["lb"], hos.LB_DTYPE)["lb_pack"]
        mk = r["makespan_est"].cpu().numpy()
        gap = mk - lb
        out[key] = {"ms_per_call": ms_, "mean_gap": float(gap.mean()), "max_gap": int(gap.max()),
                    "mean_relative_gap": float((gap / np.maximum(lb, 1)).mean()), "at_lower_bound": int((gap == 0).sum()),
                    "local_search_rounds": rounds}
        if steps:
            out[key]["instances_taking_multifit"] = int(r["packer"].sum().item())
    return out


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except (OSError, KeyError, ValueError):
            pass
    return 6650.0, "fallback"


def oracle_sample(w: Workload, n_sample: int, repeats: int = 1):
    """Time the CPU oracle (one thread) on the first n_sample instances, `repeats` times over: the whole path."""
    from oracle import hos_oracle as ora
    sub = w.subset(0, n_sample)
    p, o = sub.lengths()
    est = sub.estimates()
    t0 = time.perf_counter()
    iters = 0
    for k in [k for _ in range(repeats) for k in range(sub.n_inst)]:
        sweep = len(w.lambdas_q16) > 1
        pk = ora.offline_pack(p[k], o[k] if est is None else est[k], w.n_clients, w.cost_model,
                              0 if sweep else w.ls_rounds)
        ora.lower_bound(p[k], o[k], w.n_clients, w.batch_cap, w.cost_model)
        for lam in w.lambdas_q16:
            s = ora.simulate(pk["assign"], p[k], o[k], w.n_clients, w.cost_model, w.batch_cap, w.kv_budget,
                             lam, ora.QUEUE_SORTED, want_trace=True, o_est=None if est is None else est[k],
                             kv_reserve=w.kv_reserve)
            iters += sum(c.n_prefill_iters + c.n_decode_iters for c in s.clients)
            if sweep and w.ls_rounds > 0:      # local search on a private copy per multiplier value
                ora.local_search(pk["T"], pk["assign"], pk["load"], w.ls_rounds)
    dt = time.perf_counter() - t0
    return sub.n_inst * repeats / dt, iters / dt, dt


def sample_size(w: Workload, budget_s: float = 12.0) -> int:
    """Instances of the workload (from its start, at most all of them) that take the oracle about
    budget_s seconds on one core, from the time of the first one."""
    t0 = time.perf_counter()
    oracle_sample(w, 1)
    per_inst = max(time.perf_counter() - t0, 1e-4)
    return max(1, min(w.n_inst, int(budget_s / per_inst)))


def run_ours(args):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    import paper_2502_15763_b200 as hos
    hos.lib()

    w = rank_workload(args.workload, rank, args.instances)
    pipe = Pipeline(w, dev)
    pipe.prepare()
    input_bytes = 2 * w.n_inst * w.n_req * 4
    flush = None
    if input_bytes <= (128 << 20):
        flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 1)):
        pipe.step()
    barrier()
    t0 = time.monotonic()
    ms = timed_steps(torch, pipe.step, args.steps, flush)
    barrier()
    clocks = sampler.stop(t0, time.monotonic()) if rank == 0 else None
    ms_t = torch.tensor([ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(ms_t, op=dist.ReduceOp.MAX)
    ms = float(ms_t.item())

    # end to end: pinned host tables in, pinned host results out, every step
    host_out = []
    h2d, d2h, ms_e2e = 0, 0, 0.0
    if not args.skip_e2e:
        pipe.e2e_run(max(args.warmup, 3), host_out, flush)
        barrier()
        ms_e2e, h2d, d2h = pipe.e2e_run(args.steps, host_out, flush)
        barrier()
        for h, d in zip(host_out, pipe.results(pipe.step())):
            if not torch.equal(h, d.cpu()):
                raise SystemExit("bench: the end-to-end results differ from those of the device-resident step")
    e_t = torch.tensor([ms_e2e], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(e_t, op=dist.ReduceOp.MAX)
    ms_e2e = float(e_t.item())

    # the widened path: the same batch with Algorithm 1's request stealing between clients
    steal_ms = None
    if rank == 0 and not args.skip_steal:
        run_steal = lambda: hos.hos_online_simulate_steal(*pipe.args(), pipe.out["pk"]["assign"], pipe.lam,
                                                          hos.HOS_QUEUE_SORTED, ws=pipe.ws_on, **pipe.kw)
        run_steal()
        torch.cuda.synchronize()
        steal_ms = timed_steps(torch, run_steal, 3, flush) / 3
        # the traced form: the same call with its event log, offsets, and the trace rebuilt from the log
        state = {}

        def run_steal_logged():
            state["sim"] = hos.hos_online_simulate_steal(*pipe.args(), pipe.out["pk"]["assign"], pipe.lam,
                                                         hos.HOS_QUEUE_SORTED, keep_events=True, ws=pipe.ws_on,
                                                         **pipe.kw)
            state["off"] = hos.hos_trace_offsets(state["sim"]["cres"])

        run_steal_logged()
        n_steal_iters = int(state["off"][-1].item())
        steal_trace = pipe.trace if n_steal_iters <= pipe.trace.shape[0] else \
            torch.empty((n_steal_iters, 16), dtype=torch.uint8, device=dev)
        run_steal_fill = lambda: hos.hos_trace_fill(*pipe.args(), len(w.lambdas_q16), state["sim"], steal_trace,
                                                    state["off"], **pipe.kw)
        run_steal_fill()
        torch.cuda.synchronize()
        steal_log_ms = timed_steps(torch, run_steal_logged, 3, flush) / 3
        steal_fill_ms = timed_steps(torch, run_steal_fill, 3, flush) / 3
        del steal_trace
        pipe.step()                                   # the plain simulator's log is back in the workspace

    e2e_trace = None
    if rank == 0 and not args.skip_e2e and not args.skip_e2e_trace:
        pipe.e2e_run(1, host_out, flush, with_trace=True)
        n_t = max(2, min(args.steps, 5))
        ms_t, h2d_t, d2h_t = pipe.e2e_run(n_t, host_out, flush, with_trace=True)
        e2e_trace = {"value": w.n_inst * n_t / (ms_t * 1e-3), "unit": UNIT, "steps": n_t, "n_gpus": 1,
                     "h2d_bytes_per_step": h2d_t, "d2h_bytes_per_step": d2h_t,
                     "note": "as e2e, with the full iteration trace delivered to pinned host memory every step"}
        pipe.step()
    study = sweep = gap = None
    if rank == 0 and not args.skip_reports:
        if len(w.lambdas_q16) == 1 and w.n_inst >= 8 and (args.study or w.name in ("c2", "c2e", "paper")):
            study = study_report(hos, pipe, w)
        if len(w.lambdas_q16) > 1 and w.ls_rounds > 0:
            sweep = sweep_report(torch, hos, pipe, w, flush)
        gap = packing_gap_report(torch, hos, pipe, w, flush)
        pipe.step()

    st = pipe.out
    bad = int((st["pk"]["status"] != 0).sum().item()) + int((st["sim"]["status"] != 0).sum().item())
    if bad:
        raise SystemExit(f"bench: {bad} units finished with a non-zero status")

    if rank == 0:
        prof = kernel_profile(torch, hos, pipe, max(2, min(args.steps, 5)), flush)
        peak, peak_kind = measured_peak()
        counters, counters_shape, counters_note = ncu_counters()
        shape = {"n_req": w.n_req, "n_clients": w.n_clients, "batch_cap": w.batch_cap}
        props = torch.cuda.get_device_properties(dev)
        mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
        alu_peak = props.multi_processor_count * 128 * mhz * 1e6 / 1e12       # T int32 op/s
        issue_peak = props.multi_processor_count * 4 * mhz * 1e6 / 1e9        # G warp instructions/s
        units = {"request": w.n_inst * w.n_req, "iteration": pipe.n_iters,
                 "round": executed_rounds(w, pipe)}

        def scaled(name, field):
            """Counter of the capture scaled to this launch by the units it processes."""
            c = counters.get(name)
            if not c:
                return None
            # instructions per unit depend on the lists' lengths and the batch size: only for the captured shape
            if field == "warp_inst_per_unit" and counters_shape != shape:
                return None
            n = units[c["unit"]]
            if c["unit"] == "request" and len(w.lambdas_q16) > 1 and name in ("k_simulate", "k_ls_lists"):
                n *= len(w.lambdas_q16)                  # one pass over the requests per multiplier value
            return c[field] * n

        rows = {}
        for name, r in prof.items():
            sec = r["ms_per_launch"] * 1e-3
            by = algorithmic_bytes(w, name, pipe)
            row = dict(r, ms_per_step=r["ms_per_launch"] * r["launches_per_step"], bound=BOUND.get(name, "hbm"),
                       algorithmic_bytes=by, traffic=scaled(name, "dram_bytes_per_unit"))
            if row["bound"] == "hbm":
                row.update(achieved=by / sec / 1e9, peak=peak, unit="GB/s", peak_source=f"of {peak_kind}")
            elif row["bound"] == "alu":
                row.update(achieved=INT_OPS_PER_ITERATION * pipe.n_iters / sec / 1e12, peak=alu_peak,
                           unit="Tint32op/s", peak_source="SMs x 128 int32 lanes x max SM clock",
                           ops_per_iteration=INT_OPS_PER_ITERATION)
            else:
                inst = scaled(name, "warp_inst_per_unit")
                row.update(achieved=None if inst is None else inst / sec / 1e9, peak=issue_peak,
                           unit="Gwarp-inst/s", peak_source="SMs x 4 schedulers x max SM clock",
                           warp_inst_per_launch=inst)
                row["effective_gbs"] = by / sec / 1e9     # what a streaming form of the step would have to sustain
            row["frac"] = None if row["achieved"] is None else row["achieved"] / row["peak"]
            rows[name] = row
        if "k_local_search" in rows and units["round"]:
            r, n_ctas = rows["k_local_search"], w.n_inst * (len(w.lambdas_q16) if len(w.lambdas_q16) > 1 else 1)
            inst = r.get("warp_inst_per_launch")
            # rounds run side by side, one CTA per (instance, copy): a CTA's rounds follow each other
            r["round"] = {"executed_rounds": units["round"], "rounds_per_cta": units["round"] / n_ctas,
                          "us_per_round_per_cta": r["ms_per_launch"] * 1e3 / (units["round"] / n_ctas),
                          "cycles_per_round_per_cta": r["ms_per_launch"] * 1e-3 * mhz * 1e6 / (units["round"] / n_ctas),
                          "warp_inst_per_round": None if inst is None else inst / units["round"],
                          "min_cycles_dependent_phases": LS_ROUND_MIN_CYCLES}
        top = max(rows, key=lambda n: rows[n]["ms_per_step"])
        t = rows[top]
        roofline = {"kernel": top, "bound": "alu" if t["bound"] == "issue" else t["bound"],
                    "model": {"hbm": "algorithmic bytes", "alu": "int32 operations of the method",
                              "issue": "warp instructions issued"}[t["bound"]],
                    "achieved": t["achieved"], "peak": t["peak"],
                    "unit": t["unit"], "frac": t["frac"], "traffic": t["traffic"], "peak_source": t["peak_source"],
                    "ms_per_launch": t["ms_per_launch"], "counters": counters_note}
        if t["bound"] == "issue":
            roofline["note"] = ("latency-bound chain on data resident on chip: warp instructions issued (ncu "
                                "count per unit of work x units of this launch) against the issue slots; "
                                "effective_gbs is what a streaming form re-reading the instance every round "
                                "would have to sustain, not a bandwidth this kernel reaches")
            roofline["effective_gbs"] = t["effective_gbs"]
            if "round" in t:
                roofline["round"] = t["round"]
        # the step as a whole against the HBM roofline: algorithmic bytes of every kernel, local search once
        step_bytes = sum(r["algorithmic_bytes"] for n, r in rows.items() if r["bound"] != "issue" or n == "k_lpt")
        step_bytes += 8.0 * w.n_inst * w.n_req if "k_local_search" in rows else 0.0
        step_roofline = {"algorithmic_bytes": step_bytes, "achieved_gbs": step_bytes / (ms / args.steps * 1e-3) / 1e9,
                         "frac_of_hbm": step_bytes / (ms / args.steps * 1e-3) / 1e9 / peak}
        launches = sum(r["launches_per_step"] for r in prof.values())
        n_s, reps = 0, 1
        if args.skip_cpu_baseline:
            cpu_inst, cpu_iters, cpu_dt = None, None, 0.0
        else:
            n_s = sample_size(w)
            if n_s == w.n_inst:                         # a small workload: over and over, for about 12 s in all
                t1 = time.perf_counter()
                oracle_sample(w, n_s)
                reps = max(1, int(12.0 / max(time.perf_counter() - t1, 1e-3)))
            cpu_inst, cpu_iters, cpu_dt = oracle_sample(w, n_s, reps)
        total_inst = w.n_inst * world
        line = {
            "metric": METRIC, "value": total_inst * args.steps / (ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE,
            "data": "synthetic",
            "config": {"workload": describe(w), "instances_per_gpu": w.n_inst,
                       "l2": ("inputs larger than L2" if flush is None else "L2 flushed between steps")},
            "sim_iterations_per_step": pipe.n_iters * world,
            "sim_iterations_per_s": pipe.n_iters * world * args.steps / (ms * 1e-3),
            "clocks": clocks,
            "e2e": {"value": None if args.skip_e2e else total_inst * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "note": "every step uploads its tables from pinned host memory and downloads its results "
                            "(assignment, loads, bounds, client and simulation results; the iteration trace stays "
                            "on the device); two sets of device tables, so step k+1's upload and step k-1's "
                            "download run beside step k's kernels; timed from the first upload to the last "
                            "download" + ("" if flush is None else ", L2 flushes included")},
            "e2e_with_trace": e2e_trace,
            "gpu_launches": int(round(launches * args.steps)),
            "requests_per_step": w.n_inst * w.n_req, "shape": shape,
            "ls_rounds_executed_per_step": units["round"],
            "input_sha256": input_sha256(pipe),
            "roofline": roofline,
            "step_roofline": step_roofline,
            "study": study, "sweep_local_search": sweep, "packing_gap": gap,
            "kernels": rows,
            "request_stealing": None if steal_ms is None else {
                "call": "hos_online_simulate_steal", "ms_per_call": steal_ms,
                "ms_per_call_with_event_log_and_offsets": steal_log_ms,
                "trace_fill_ms": steal_fill_ms, "trace_iterations": n_steal_iters,
                "trace_fill_gbs": 16.0 * n_steal_iters / (steal_fill_ms * 1e-3) / 1e9,
                "simulations_per_s": w.n_inst * len(w.lambdas_q16) / (steal_ms * 1e-3),
                "plain_simulate_ms": rows.get("k_simulate", {}).get("ms_per_launch")},
            "cpu_baseline": {"value": cpu_inst, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": f"first {n_s} instance(s) of the workload x {reps}, whole path, {cpu_dt:.1f} s",
                             "sim_iterations_per_s": cpu_iters},
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_reference(args):
    """The CPU oracle as it stands, one thread, on a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload(args.workload)
    n_s = max(1, sample_size(w, 3.0))        # per step: about three seconds of oracle work
    for _ in range(args.warmup):
        oracle_sample(w, 1)
    t0 = time.perf_counter()
    iters_per_s = 0.0
    for _ in range(args.steps):
        _, it, _ = oracle_sample(w, n_s)
        iters_per_s += it / args.steps
    dt = time.perf_counter() - t0
    value = n_s * args.steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3 / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": describe(w), "sample_instances_per_step": n_s},
        "sim_iterations_per_s": iters_per_s,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"first {n_s} instance(s) of the workload per step, whole path"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c4", choices=["c0", "c1", "c2", "c3", "c4", "paper", "c1e", "c2e"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--instances", type=int, default=0,
                    help="use only the first N instances of the workload (profiling captures)")
    ap.add_argument("--skip-steal", action="store_true",
                    help="do not time the request-stealing simulation (profiling captures)")
    ap.add_argument("--skip-e2e", action="store_true",
                    help="do not time the end-to-end step (profiling captures: one launch per kernel and step)")
    ap.add_argument("--skip-e2e-trace", action="store_true",
                    help="do not time the end-to-end step that also delivers the trace to the host")
    ap.add_argument("--skip-reports", action="store_true",
                    help="leave out the study / sweep / packing-gap reports (profiling captures)")
    ap.add_argument("--study", action="store_true",
                    help="hybrid-vs-baseline study on this workload too (default: c2, c2e, paper)")
    ap.add_argument("--skip-cpu-baseline", action="store_true",
                    help="do not time the CPU oracle (profiling captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
