"""Runs the CUDA library and the CPU oracle on the same tables and compares them field by field."""
from __future__ import annotations

import numpy as np

from oracle import hos_oracle as ora


def to_dev(a, dtype=np.int32):
    import torch
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(a.astype(dtype, copy=False)).cuda()


def gpu_offline(hos, p, o, M, cap, kv, cm, ls_rounds, est=None, rsv=0, multifit_steps=0):
    ek = dict(o_est=None if est is None else to_dev(est), kv_reserve=rsv)
    r = hos.hos_offline_pack(to_dev(p), to_dev(o), M, cap, kv, cm, ls_rounds, want_log=True, want_lb=True,
                             multifit_steps=multifit_steps, **ek)
    import torch
    sep = hos.hos_lower_bound(to_dev(p), to_dev(o), M, cap, kv, cm, **ek)
    assert torch.equal(r["lb"], sep["lb"]), "bounds from hos_offline_pack differ from hos_lower_bound"
    out = {k: (v.cpu().numpy() if v is not None and k not in ("ls_log", "lb") else v) for k, v in r.items()}
    if r["ls_log"] is not None:
        from paper_2502_15763_b200.binding import view_struct
        out["ls_log"] = view_struct(r["ls_log"], hos.LS_MOVE_DTYPE)
    return out


def check_offline(hos, p, o, M, cap, kv, cm, ls_rounds, insts=None, est=None, rsv=0, multifit_steps=0):
    """GPU offline pack of the whole batch against the oracle on `insts` (default: all)."""
    g = gpu_offline(hos, p, o, M, cap, kv, cm, ls_rounds, est, rsv, multifit_steps)
    insts = range(p.shape[0]) if insts is None else insts
    for k in insts:
        e = ora.offline_pack(p[k], o[k] if est is None else est[k], M, cm, ls_rounds,
                             multifit_steps=multifit_steps)                             # packed on what is known
        assert g["status"][k] == 0
        if multifit_steps > 0:
            assert int(g["packer"][k]) == e["packer"], f"packer differs in instance {k}"
        assert np.array_equal(g["assign"][k], e["assign"]), f"assign differs in instance {k}"
        assert np.array_equal(g["load"][k], e["load"]), f"load differs in instance {k}"
        assert int(g["makespan_est"][k]) == e["makespan_est"]
        assert int(g["rounds_applied"][k]) == e["rounds_applied"]
        if ls_rounds > 0:
            gl, el = g["ls_log"][k], e["ls_log"]
            for f in ("i", "u", "k", "v"):
                assert np.array_equal(gl[f], el[f]), f"ls_log.{f} differs in instance {k}"
    return g


def check_lower_bound(hos, p, o, M, cap, kv, cm, insts=None, est=None, rsv=0):
    from paper_2502_15763_b200.binding import view_struct
    r = hos.hos_lower_bound(to_dev(p), to_dev(o), M, cap, kv, cm, o_est=None if est is None else to_dev(est),
                            kv_reserve=rsv)
    lb = view_struct(r["lb"], hos.LB_DTYPE)
    st = r["status"].cpu().numpy()
    insts = range(p.shape[0]) if insts is None else insts
    for k in insts:
        e = ora.lower_bound(p[k], o[k], M, cap, cm)
        if est is not None:          # the packing bounds are in units of the estimated times
            e.update({f: v for f, v in ora.lower_bound(p[k], est[k], M, cap, cm).items()
                      if f in ("lb_pack", "sum_T", "max_T", "pair_T")})
        assert st[k] == 0
        for f, v in e.items():
            assert int(lb[k][f]) == v, f"lower bound field {f} differs in instance {k}"
    return lb


def gpu_simulate(hos, p, o, M, cap, kv, cm, assign, lambdas, mode, max_iters=0x7FFFFFFF, want_trace=True,
                 trace_slots=None, est=None, rsv=0):
    """Counts (with the event log), offsets, then the trace twice: rebuilt from the event log by
    hos_trace_fill and written directly by a traced simulation; the two must be the same bytes.
    Returns host-side views."""
    import torch
    from paper_2502_15763_b200.binding import view_struct
    dp, do, da = to_dev(p), to_dev(o), to_dev(assign)
    dl = to_dev(np.asarray(lambdas, dtype=np.uint32))
    ek = dict(o_est=None if est is None else to_dev(est), kv_reserve=rsv)
    r = hos.hos_online_simulate(dp, do, M, cap, kv, cm, da, dl, mode, max_iters, keep_events=want_trace, **ek)
    out = dict(cres=view_struct(r["cres"], hos.CLIENT_RESULT_DTYPE),
               sres=view_struct(r["sres"], hos.SIM_RESULT_DTYPE), status=r["status"].cpu().numpy())
    if want_trace:
        if trace_slots is None:
            off = hos.hos_trace_offsets(r["cres"])
        else:
            n_units = p.shape[0] * len(lambdas) * M
            off = torch.arange(n_units + 1, dtype=torch.int64, device="cuda") * int(trace_slots)
        total = int(off[-1].item())
        trace = torch.zeros((max(total, 1), 16), dtype=torch.uint8, device="cuda")
        r2 = hos.hos_online_simulate(dp, do, M, cap, kv, cm, da, dl, mode, max_iters, trace=trace, trace_off=off,
                                     **ek)
        out2 = dict(cres=view_struct(r2["cres"], hos.CLIENT_RESULT_DTYPE),
                    sres=view_struct(r2["sres"], hos.SIM_RESULT_DTYPE), status=r2["status"].cpu().numpy())
        for f in out["cres"].dtype.names:
            assert np.array_equal(out["cres"][f], out2["cres"][f]), f"traced run changed cres.{f}"
        out["status_traced"] = out2["status"]
        filled = torch.zeros_like(trace)
        hos.hos_trace_fill(dp, do, M, cap, kv, cm, len(lambdas), r, filled, off, **ek)
        assert torch.equal(filled, trace), "trace rebuilt from the event log differs from the traced simulation"
        assert np.array_equal(r["status"].cpu().numpy(), out2["status"]), "status after hos_trace_fill differs"
        out["trace"] = view_struct(trace, hos.ITER_REC_DTYPE)
        out["trace_off"] = off.cpu().numpy()
    return out


def check_simulate(hos, p, o, M, cap, kv, cm, assign, lambdas, mode, insts=None, max_iters=0x7FFFFFFF,
                   want_trace=True, est=None, rsv=0):
    g = gpu_simulate(hos, p, o, M, cap, kv, cm, assign, lambdas, mode, max_iters, want_trace, est=est, rsv=rsv)
    insts = range(p.shape[0]) if insts is None else insts
    nl = len(lambdas)
    for k in insts:
        for li, lam in enumerate(lambdas):
            e = ora.simulate(assign[k], p[k], o[k], M, cm, cap, kv, int(lam), mode, max_iters, want_trace,
                             o_est=None if est is None else est[k], kv_reserve=rsv)
            s = g["sres"][k, li]
            assert int(s["makespan_us"]) == e.makespan_us, (k, li)
            assert int(s["busy_slot_us"]) == e.busy_slot_us
            assert abs(float(s["utilisation"]) - e.utilisation) <= 1e-9 * abs(e.utilisation)
            assert abs(float(s["tokens_per_s"]) - e.tokens_per_s) <= 1e-9 * abs(e.tokens_per_s)
            for j, ec in enumerate(e.clients):
                c = g["cres"][k, li, j]
                got = (int(c["makespan_us"]), int(c["busy_slot_us"]), int(c["n_prefill_iters"]),
                       int(c["n_decode_iters"]), int(c["trace_hash"]), int(g["status"][k, li, j]))
                want = (ec.makespan_us, ec.busy_slot_us, ec.n_prefill_iters, ec.n_decode_iters,
                        ec.trace_hash, ec.status)
                assert got == want, f"client result differs: inst {k} lambda {li} client {j}: {got} != {want}"
                assert abs(float(c["utilisation"]) - ec.utilisation) <= 1e-9 * abs(ec.utilisation)
                if want_trace:
                    x = (k * nl + li) * M + j
                    t0, t1 = int(g["trace_off"][x]), int(g["trace_off"][x + 1])
                    assert t1 - t0 == len(ec.trace)
                    gt = g["trace"][t0:t1]
                    for f in ("dur_us", "kind_n", "tokens", "aux"):
                        assert np.array_equal(gt[f], ec.trace[f]), f"trace.{f} differs: inst {k} lambda {li} client {j}"
    return g


def gpu_simulate_steal(hos, p, o, M, cap, kv, cm, assign, lambdas, mode, max_iters=0x7FFFFFFF, est=None, rsv=0):
    """hos_online_simulate_steal: counts (with the event log), offsets, then the trace twice: rebuilt
    from the event log by hos_trace_fill and written directly by a traced run with exact slots; the
    two must be the same bytes.  Host-side views."""
    import torch
    from paper_2502_15763_b200.binding import view_struct
    dp, do, da = to_dev(p), to_dev(o), to_dev(assign)
    dl = to_dev(np.asarray(lambdas, dtype=np.uint32))
    ek = dict(o_est=None if est is None else to_dev(est), kv_reserve=rsv)
    r = hos.hos_online_simulate_steal(dp, do, M, cap, kv, cm, da, dl, mode, max_iters, want_served_by=True,
                                      keep_events=True, **ek)
    off = hos.hos_trace_offsets(r["cres"])
    trace = torch.zeros((max(int(off[-1].item()), 1), 16), dtype=torch.uint8, device="cuda")
    r2 = hos.hos_online_simulate_steal(dp, do, M, cap, kv, cm, da, dl, mode, max_iters, trace=trace, trace_off=off,
                                       want_served_by=True, **ek)
    assert torch.equal(r["cres"][..., :32], r2["cres"][..., :32]) and torch.equal(r["served_by"], r2["served_by"])
    filled = torch.zeros_like(trace)
    hos.hos_trace_fill(dp, do, M, cap, kv, cm, len(lambdas), r, filled, off, **ek)
    assert torch.equal(filled, trace), "trace rebuilt from the stealing simulator's event log differs from the traced run"
    assert torch.equal(r["status"], r2["status"]), "status after hos_trace_fill differs"
    return dict(cres=view_struct(r2["cres"], hos.CLIENT_RESULT_DTYPE), sres=view_struct(r2["sres"], hos.SIM_RESULT_DTYPE),
                status=r2["status"].cpu().numpy(), served_by=r2["served_by"].cpu().numpy(),
                trace=view_struct(trace, hos.ITER_REC_DTYPE), trace_off=off.cpu().numpy())


def check_simulate_steal(hos, p, o, M, cap, kv, cm, assign, lambdas, mode, insts=None, max_iters=0x7FFFFFFF,
                         est=None, rsv=0):
    """hos_online_simulate_steal (counts, then a traced run with exact slots) against the oracle."""
    g = gpu_simulate_steal(hos, p, o, M, cap, kv, cm, assign, lambdas, mode, max_iters, est, rsv)
    cres, sres, st, served, tr, toff = g["cres"], g["sres"], g["status"], g["served_by"], g["trace"], g["trace_off"]
    insts = range(p.shape[0]) if insts is None else insts
    nl = len(lambdas)
    for k in insts:
        for li, lam in enumerate(lambdas):
            e, eserved = ora.simulate_steal(assign[k], p[k], o[k], M, cm, cap, kv, int(lam), mode, max_iters, True,
                                            o_est=None if est is None else est[k], kv_reserve=rsv)
            assert np.array_equal(served[k, li], eserved), f"served_by differs: inst {k} lambda {li}"
            s = sres[k, li]
            assert int(s["makespan_us"]) == e.makespan_us and int(s["busy_slot_us"]) == e.busy_slot_us
            assert abs(float(s["utilisation"]) - e.utilisation) <= 1e-9 * abs(e.utilisation)
            assert abs(float(s["tokens_per_s"]) - e.tokens_per_s) <= 1e-9 * abs(e.tokens_per_s)
            for j, ec in enumerate(e.clients):
                c = cres[k, li, j]
                got = (int(c["makespan_us"]), int(c["busy_slot_us"]), int(c["n_prefill_iters"]),
                       int(c["n_decode_iters"]), int(c["trace_hash"]), int(st[k, li, j]))
                want = (ec.makespan_us, ec.busy_slot_us, ec.n_prefill_iters, ec.n_decode_iters, ec.trace_hash,
                        ec.status)
                assert got == want, f"client result differs: inst {k} lambda {li} client {j}: {got} != {want}"
                x = (k * nl + li) * M + j
                gt = tr[int(toff[x]):int(toff[x + 1])]
                assert len(gt) == len(ec.trace)
                for f in ("dur_us", "kind_n", "tokens", "aux"):
                    assert np.array_equal(gt[f], ec.trace[f]), f"trace.{f} differs: inst {k} lambda {li} client {j}"
    return dict(cres=cres, sres=sres, status=st, served_by=served)
