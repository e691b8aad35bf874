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
# step alone must move once)
BYTES_PER_REQ = {"k_estimate_sort": 16, "k_lpt": 12, "k_lower_bound": 8, "k_queue_build": 16, "k_ls_lists": 15}
# what bounds each kernel (counters in profiles/): streaming kernels against the measured copy
# bandwidth, the two sequential recurrences against the integer issue rate
BOUND = {"k_simulate": "alu", "k_simulate_steal": "alu", "k_lpt": "latency (dependent chain)",
         "k_local_search": "latency / issue (instance resident on chip; bytes are those of a streaming round)"}
# integer operations of one simulated iteration as the method states it: duration (3), busy slot
# time (2), clock (1), waited decode time (2), sum of KV lengths (1), decision compare in Q16.16 (3),
# trace hash (9), counters (3)
INT_OPS_PER_ITERATION = 24
# DRAM bytes per request and launch measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum
# over 296 instances of c4's shape, see profiles/); None for a kernel changed since its capture
NCU_DRAM_BYTES_PER_REQ = {"k_estimate_sort": 8.68, "k_lower_bound": 8.05, "k_lpt": 12.69, "k_ls_lists": 18.09,
                          "k_local_search": 6.07, "k_queue_build": 15.77, "k_simulate": 20.75}
NCU_DRAM_BYTES_PER_ITERATION = {"k_trace_fill": 18.79}


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

    def e2e_run(self, steps, host_out, flush):
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
        main.wait_stream(self.down)
        main.wait_stream(self.up)
        end.record(main)
        torch.cuda.synchronize()
        h2d = sum(h.numel() * h.element_size() for h in host.values() if h is not None)
        d2h = sum(h.numel() * h.element_size() for h in host_out)
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
        extra = 64 * w.n_inst if name == "k_lower_bound" else 0
        return BYTES_PER_REQ[name] * n_req_total + extra
    if name == "k_local_search":
        src = pipe.out["ls"] if "ls" in pipe.out else pipe.out["pk"]
        applied = src["rounds_applied"].to("cpu").numpy().astype(np.int64)
        executed = np.minimum(applied + 1, w.ls_rounds).sum()          # the no-op round is evaluated too
        return float(executed) * (8 * w.n_req + 8 * w.n_clients)
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


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except (OSError, KeyError, ValueError):
            pass
    return 6650.0, "fallback"


def oracle_sample(w: Workload, n_sample: int):
    """Time the CPU oracle (one thread) on the first n_sample instances: the whole path."""
    from oracle import hos_oracle as ora
    sub = w.subset(0, n_sample)
    p, o = sub.lengths()
    est = sub.estimates()
    t0 = time.perf_counter()
    iters = 0
    for k in range(sub.n_inst):
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
    return sub.n_inst / dt, iters / dt, dt


def sample_size(w: Workload) -> int:
    # about 3 s of single-thread oracle work per instance at the largest size, milliseconds at the others
    per_inst = 3.0 if w.n_req >= 10000 else 0.025 * max(1, len(w.lambdas_q16)) + 0.03
    return max(1, min(w.n_inst, int(12.0 / per_inst)))


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

    st = pipe.out
    bad = int((st["pk"]["status"] != 0).sum().item()) + int((st["sim"]["status"] != 0).sum().item())
    if bad:
        raise SystemExit(f"bench: {bad} units finished with a non-zero status")

    if rank == 0:
        prof = kernel_profile(torch, hos, pipe, max(2, min(args.steps, 5)), flush)
        peak, peak_kind = measured_peak()
        rows = {}
        for name, r in prof.items():
            by = algorithmic_bytes(w, name, pipe)
            gbs = by / (r["ms_per_launch"] * 1e-3) / 1e9
            rows[name] = dict(r, algorithmic_bytes=by, achieved_gbs=gbs, frac=gbs / peak,
                              ms_per_step=r["ms_per_launch"] * r["launches_per_step"])
        for name in rows:
            rows[name]["bound"] = BOUND.get(name, "hbm")
        top = max(rows, key=lambda n: rows[n]["ms_per_step"])
        def dram_traffic(name):
            # scaled from the capture by the units a launch processes (requests of every instance or
            # simulation; iterations for the trace)
            if name in NCU_DRAM_BYTES_PER_ITERATION:
                return NCU_DRAM_BYTES_PER_ITERATION[name] * pipe.n_iters
            per_req = NCU_DRAM_BYTES_PER_REQ.get(name)
            if per_req is None:
                return None
            sims = len(w.lambdas_q16) if name in ("k_simulate", "k_local_search", "k_ls_lists") and len(w.lambdas_q16) > 1 else 1
            return per_req * w.n_inst * w.n_req * sims
        for name in rows:
            rows[name]["traffic"] = dram_traffic(name)
        traffic = dram_traffic(top)
        if BOUND.get(top) == "alu":
            # the iteration recurrence is integer arithmetic: operations of the method per second
            # against 128 int32 lanes per SM at the maximum SM clock
            props = torch.cuda.get_device_properties(dev)
            mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
            alu_peak = props.multi_processor_count * 128 * mhz * 1e6 / 1e12
            ach = INT_OPS_PER_ITERATION * pipe.n_iters / (rows[top]["ms_per_launch"] * 1e-3) / 1e12
            roofline = {"kernel": top, "bound": "alu", "achieved": ach, "peak": alu_peak, "unit": "Tint32op/s",
                        "frac": ach / alu_peak, "traffic": traffic,
                        "peak_source": "SMs x 128 int32 lanes x max SM clock",
                        "ops_per_iteration": INT_OPS_PER_ITERATION, "ms_per_launch": rows[top]["ms_per_launch"]}
        else:
            roofline = {"kernel": top, "bound": "hbm", "achieved": rows[top]["achieved_gbs"], "peak": peak,
                        "unit": "GB/s", "frac": rows[top]["frac"], "traffic": traffic,
                        "peak_source": f"of {peak_kind}", "ms_per_launch": rows[top]["ms_per_launch"]}
            if top == "k_local_search":
                roofline["note"] = ("effective: bytes a streaming implementation would re-read every executed "
                                    "round; this kernel reads the instance from HBM once")
        launches = sum(r["launches_per_step"] for r in prof.values())
        n_s = sample_size(w)
        if args.skip_cpu_baseline:
            cpu_inst, cpu_iters, cpu_dt = None, None, 0.0
        else:
            cpu_inst, cpu_iters, cpu_dt = oracle_sample(w, n_s)
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
            "gpu_launches": int(round(launches * args.steps)),
            "roofline": roofline,
            "kernels": rows,
            "request_stealing": None if steal_ms is None else {
                "call": "hos_online_simulate_steal", "ms_per_call": steal_ms,
                "simulations_per_s": w.n_inst * len(w.lambdas_q16) / (steal_ms * 1e-3),
                "plain_simulate_ms": rows.get("k_simulate", {}).get("ms_per_launch")},
            "cpu_baseline": {"value": cpu_inst, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": f"first {n_s} instance(s) of the workload, whole path, {cpu_dt:.1f} s",
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
    n_s = max(1, sample_size(w) // 4)        # per step; the default 50 steps then take about two minutes at c4
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
    ap.add_argument("--skip-cpu-baseline", action="store_true",
                    help="do not time the CPU oracle (profiling captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
