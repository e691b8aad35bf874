"""CUDA path against the CPU oracle, element by element, through the C ABI (needs a GPU)."""
import numpy as np
import pytest

from oracle import hos_oracle as ora
from tests import gpu_harness as H
from workload import LAMBDA_NEVER_PREEMPT, LAMBDA_ONE, LAMBDA_PREFILL_FIRST, LengthDist, batch_lengths, workload

pytestmark = pytest.mark.gpu

LAMS = (LAMBDA_NEVER_PREEMPT, 20000, LAMBDA_ONE, 5 << 16, LAMBDA_PREFILL_FIRST)


@pytest.fixture(scope="module")
def hos():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2502_15763_b200 as m
    m.lib()
    return m


def full_pipeline(hos, w, ls_rounds, lambdas, insts=None, modes=(ora.QUEUE_SORTED, ora.QUEUE_FCFS)):
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    g = H.check_offline(hos, p, o, M, cap, kv, cm, ls_rounds, insts)
    H.check_lower_bound(hos, p, o, M, cap, kv, cm, insts)
    for mode in modes:
        H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], lambdas, mode, insts)
    return p, o, g


def test_config0(hos):
    full_pipeline(hos, workload("c0"), 10, LAMS)


def test_config1(hos):
    full_pipeline(hos, workload("c1"), 20, LAMS)


def test_config2_hybrid_and_baseline(hos):
    w = workload("c2")
    p, o, g = full_pipeline(hos, w, 0, (LAMBDA_ONE,), modes=(ora.QUEUE_SORTED,))
    rr = (np.arange(w.n_req, dtype=np.int32) % w.n_clients)[None, :].repeat(w.n_inst, 0)
    base = H.check_simulate(hos, p, o, w.n_clients, w.batch_cap, w.kv_budget, w.cost_model, rr,
                            (LAMBDA_PREFILL_FIRST, LAMBDA_NEVER_PREEMPT), ora.QUEUE_FCFS)
    hyb = H.gpu_simulate(hos, p, o, w.n_clients, w.batch_cap, w.kv_budget, w.cost_model, g["assign"],
                         (LAMBDA_ONE,), ora.QUEUE_SORTED, want_trace=False)
    gain = hyb["sres"]["utilisation"][:, 0] - base["sres"]["utilisation"][:, 0]
    assert gain.mean() > 0           # direction of the paper's 100-case study


def test_config3_sweep(hos):
    w = workload("c3")
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    g = H.check_offline(hos, p, o, M, cap, kv, cm, 0)
    H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], w.lambdas_q16, ora.QUEUE_SORTED,
                     insts=range(0, 100, 9), want_trace=False)
    H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], w.lambdas_q16[::13], ora.QUEUE_SORTED,
                     insts=(3, 50))
    # 20 local-search rounds on a private copy of the LPT assignment per (instance, multiplier)
    import torch
    from paper_2502_15763_b200.binding import view_struct
    nl = len(w.lambdas_q16)
    copies = torch.from_numpy(g["assign"]).cuda()[:, None, :].repeat(1, nl, 1).contiguous()
    r = hos.hos_local_search(H.to_dev(p), H.to_dev(o), M, cap, kv, cm, copies, w.ls_rounds, want_log=True)
    a, l = r["assign"].cpu().numpy(), r["load"].cpu().numpy()
    log = view_struct(r["ls_log"], hos.LS_MOVE_DTYPE)
    assert (r["status"].cpu().numpy() == 0).all()
    for k in range(w.n_inst):
        T = ora.estimate(p[k], o[k], cm)
        ea, el, applied, elog = ora.local_search(T, g["assign"][k], g["load"][k], w.ls_rounds)
        for c in range(nl):                                    # the copies agree bit for bit
            assert np.array_equal(a[k, c], ea) and np.array_equal(l[k, c], el)
            assert int(r["rounds_applied"][k, c]) == applied
            assert int(r["makespan_est"][k, c]) == int(el.max())
        for f in ("i", "u", "k", "v"):
            assert np.array_equal(log[k, 0][f], elog[f]) and np.array_equal(log[k, nl - 1][f], elog[f])


@pytest.mark.parametrize("n,M,cap", [(1, 1, 1), (2, 3, 1), (31, 4, 2), (33, 32, 16), (97, 33, 33),
                                     (257, 64, 64), (1000, 65, 100), (1301, 130, 128), (2050, 256, 200),
                                     (515, 7, 256), (64, 100, 5)])
def test_ragged_shapes(hos, n, M, cap):
    rng = np.random.default_rng(n * 1000 + M)
    n_inst = 3
    p = rng.integers(1, 300, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 120, size=(n_inst, n)).astype(np.uint32)
    o[:, ::7] = 1                                              # many ties and one-token outputs
    p[:, ::5] = p[:, :1]
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    kv = int((p.astype(np.int64) + o).max()) * int(rng.choice([1, 3, 1000]))
    g = H.check_offline(hos, p, o, M, cap, kv, cm, 6)
    H.check_lower_bound(hos, p, o, M, cap, kv, cm)
    rand_assign = rng.integers(0, M, size=(n_inst, n)).astype(np.int32)
    for assign in (g["assign"], rand_assign):
        for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
            H.check_simulate(hos, p, o, M, cap, kv, cm, assign, LAMS, mode)


def test_local_search_from_bad_assignments(hos):
    import torch
    from paper_2502_15763_b200.binding import view_struct
    rng = np.random.default_rng(77)
    n_inst, n, M, rounds = 4, 700, 9, 40
    p = rng.integers(1, 50, size=(n_inst, n)).astype(np.uint32)      # few distinct T: many ties
    o = rng.integers(1, 6, size=(n_inst, n)).astype(np.uint32)
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    assign = rng.integers(0, M, size=(n_inst, 2, n)).astype(np.int32)
    assign[:, 1, :] = 0                                              # everything on one client
    r = hos.hos_local_search(H.to_dev(p), H.to_dev(o), M, 8, 10 ** 6, cm, torch.from_numpy(assign).cuda(),
                             rounds, want_log=True)
    log = view_struct(r["ls_log"], hos.LS_MOVE_DTYPE)
    for k in range(n_inst):
        T = ora.estimate(p[k], o[k], cm)
        for c in range(2):
            l0 = np.array([int(T[assign[k, c] == j].sum()) for j in range(M)], dtype=np.int64)
            ea, el, applied, elog = ora.local_search(T, assign[k, c], l0, rounds)
            assert np.array_equal(r["assign"][k, c].cpu().numpy(), ea)
            assert np.array_equal(r["load"][k, c].cpu().numpy(), el)
            assert int(r["rounds_applied"][k, c]) == applied
            for f in ("i", "u", "k", "v"):
                assert np.array_equal(log[k, c][f], elog[f])


@pytest.mark.parametrize("n,M,scale", [(1530, 3, 1), (1024, 2, 1), (900, 5, 1), (600, 4, 10000),
                                       (1000, 3, 1), (1200, 4, 1)])
def test_local_search_short_list_and_general_forms(hos, n, M, scale):
    # member lists around the length up to which the critical client's list is evaluated from
    # on-chip memory (511), loads above 2^31 (scale), which take the 64-bit form, and list lengths
    # for which a thread runs two, three and four searches side by side
    rng = np.random.default_rng(n + M)
    n_inst = 2
    p = rng.integers(1, 3000, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 800, size=(n_inst, n)).astype(np.uint32)
    p[:, ::9] = p[:, 1:2]                                            # runs of equal T
    o[:, ::9] = o[:, 1:2]
    cm = (20000, 40, 15000, 300 * scale, 16, 40 * scale, 350 * scale)
    H.check_offline(hos, p, o, M, 16, 10 ** 7, cm, 60)


def test_wide_estimates_take_the_64bit_packing_path(hos):
    # T_i up to ~2^31: the packed 32-bit load keys cannot be used
    rng = np.random.default_rng(5)
    n_inst, n, M = 2, 400, 5
    p = rng.integers(1, 2000, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 2000, size=(n_inst, n)).astype(np.uint32)
    cm = (20000, 40, 15000, 300, 16, 500000, 500000)
    H.check_offline(hos, p, o, M, 8, 10 ** 6, cm, 5)
    H.check_lower_bound(hos, p, o, M, 8, 10 ** 6, cm)


def test_long_requests_use_the_wide_heap_entries(hos):
    # p + o >= 2^16 in instance 1 only: the two simulator instantiations split the batch between them
    rng = np.random.default_rng(11)
    n_inst, n, M, cap = 3, 300, 5, 12
    p = rng.integers(1, 3000, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 60, size=(n_inst, n)).astype(np.uint32)
    p[1, ::9] = rng.integers(65000, 90000, size=p[1, ::9].shape)
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    kv = 300000
    g = H.check_offline(hos, p, o, M, cap, kv, cm, 4)
    for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
        H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], LAMS, mode)
    # a divisor that is not a power of two takes the division path
    H.check_simulate(hos, p, o, M, cap, kv, (20000, 40, 15000, 300, 7, 40, 350), g["assign"], LAMS, ora.QUEUE_SORTED)


@pytest.mark.parametrize("n,M,cap", [(3, 2, 1), (40, 1, 4), (97, 5, 3), (300, 8, 16), (515, 33, 7), (1000, 64, 40),
                                     (700, 100, 128)])
def test_request_stealing(hos, n, M, cap):
    rng = np.random.default_rng(n * 7 + M)
    n_inst = 3
    p = rng.integers(1, 300, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 90, size=(n_inst, n)).astype(np.uint32)
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    kv = int((p.astype(np.int64) + o).max()) * int(rng.choice([1, 4, 1000]))
    g = H.gpu_offline(hos, p, o, M, cap, kv, cm, 0)
    lopsided = np.zeros((n_inst, n), dtype=np.int32)               # everything queued on client 0
    lopsided[1] = rng.integers(0, max(1, M // 2), size=n)
    for assign in (g["assign"], lopsided):
        for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
            H.check_simulate_steal(hos, p, o, M, cap, kv, cm, assign, LAMS, mode)
    H.check_simulate_steal(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED, max_iters=25)


def test_request_stealing_event_log_edges(hos):
    import torch
    # one slot per client: every request is a prefill and a retiring decode of its own, so the log is
    # as long as it can get (two entries per request) and nearly all of it sits with the clients that
    # took the requests from client 0's queue
    rng = np.random.default_rng(77)
    n_inst, n, M, cap = 3, 257, 7, 1
    p = rng.integers(1, 300, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 40, size=(n_inst, n)).astype(np.uint32)
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    assign = np.zeros((n_inst, n), dtype=np.int32)
    r = H.check_simulate_steal(hos, p, o, M, cap, 10 ** 6, cm, assign, (LAMBDA_ONE, LAMBDA_PREFILL_FIRST), ora.QUEUE_SORTED)
    assert int(r["cres"]["n_prefill_iters"].sum()) == 2 * n_inst * n          # one prefill per request and multiplier
    assert (r["cres"]["n_prefill_iters"][:, :, 1:] > 0).all()                   # the others served stolen requests
    # an invalid instance beside valid ones: no log entries, no trace records, neighbours untouched
    o2 = o.copy(); o2[1, 9] = 0
    dp, do, da = H.to_dev(p), H.to_dev(o2), H.to_dev(assign)
    dl = H.to_dev(np.asarray([LAMBDA_ONE], np.uint32))
    s = hos.hos_online_simulate_steal(dp, do, M, cap, 10 ** 6, cm, da, dl, ora.QUEUE_SORTED, keep_events=True)
    off = hos.hos_trace_offsets(s["cres"])
    offs = off.cpu().numpy()
    assert offs[M] == offs[2 * M]                                               # instance 1 has no iterations
    filled = torch.zeros((int(offs[-1]), 16), dtype=torch.uint8, device="cuda")
    hos.hos_trace_fill(dp, do, M, cap, 10 ** 6, cm, 1, s, filled, off)
    direct = torch.zeros_like(filled)
    hos.hos_online_simulate_steal(dp, do, M, cap, 10 ** 6, cm, da, dl, ora.QUEUE_SORTED, trace=direct, trace_off=off)
    assert torch.equal(filled, direct)
    st = s["status"].cpu().numpy()
    assert (st[1] == hos.HOS_ST_INVALID).all() and (st[0] == 0).all() and (st[2] == 0).all()
    # too few trace slots: the records that fit are the first ones, the status bit is set
    small = torch.arange(n_inst * M + 1, dtype=torch.int64, device="cuda") * 5
    part = torch.zeros((n_inst * M * 5, 16), dtype=torch.uint8, device="cuda")
    s = hos.hos_online_simulate_steal(dp, H.to_dev(o), M, cap, 10 ** 6, cm, da, dl, ora.QUEUE_SORTED, keep_events=True)
    hos.hos_trace_fill(dp, H.to_dev(o), M, cap, 10 ** 6, cm, 1, s, part, small)
    assert (s["status"].cpu().numpy() == hos.HOS_ST_TRACE).all()
    full_off = hos.hos_trace_offsets(s["cres"]).cpu().numpy()
    full = torch.zeros((int(full_off[-1]), 16), dtype=torch.uint8, device="cuda")
    hos.hos_online_simulate_steal(dp, H.to_dev(o), M, cap, 10 ** 6, cm, da, dl, ora.QUEUE_SORTED, trace=full,
                                  trace_off=H.to_dev(full_off, np.int64))
    for x in range(n_inst * M):
        assert torch.equal(part[5 * x:5 * x + 5], full[int(full_off[x]):int(full_off[x]) + 5])
    # the same workspace used by the plain simulator afterwards: the log's form follows the last call
    ws = s["ws"]
    s3 = hos.hos_online_simulate(dp, H.to_dev(o), M, cap, 10 ** 6, cm, da, dl, ora.QUEUE_SORTED, keep_events=True, ws=ws)
    off3 = hos.hos_trace_offsets(s3["cres"])
    f3 = torch.zeros((int(off3[-1].item()), 16), dtype=torch.uint8, device="cuda")
    hos.hos_trace_fill(dp, H.to_dev(o), M, cap, 10 ** 6, cm, 1, s3, f3, off3)
    d3 = torch.zeros_like(f3)
    hos.hos_online_simulate(dp, H.to_dev(o), M, cap, 10 ** 6, cm, da, dl, ora.QUEUE_SORTED, trace=d3, trace_off=off3)
    assert torch.equal(f3, d3)


def test_request_stealing_config1_and_wide(hos):
    w = workload("c1")
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    g = H.gpu_offline(hos, p, o, M, cap, kv, cm, 0)
    H.check_simulate_steal(hos, p, o, M, cap, kv, cm, g["assign"], LAMS, ora.QUEUE_SORTED)
    rr = (np.arange(w.n_req, dtype=np.int32) % M)[None, :]
    r = H.check_simulate_steal(hos, p, o, M, cap, kv, cm, rr, (LAMBDA_PREFILL_FIRST,), ora.QUEUE_FCFS)
    plain = H.gpu_simulate(hos, p, o, M, cap, kv, cm, rr, (LAMBDA_PREFILL_FIRST,), ora.QUEUE_FCFS, want_trace=False)
    assert r["sres"]["makespan_us"][0, 0] <= plain["sres"]["makespan_us"][0, 0]
    # long requests: the 64-bit heap entries
    p2 = p.copy(); p2[0, ::50] = 70000
    H.check_simulate_steal(hos, p2, o, M, cap, 300000, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED)


def test_prefill_levels(hos):
    # stepped prefill cost (Eq. 5-7) in the simulators and the bounds
    rng = np.random.default_rng(21)
    n_inst, n, M, cap = 3, 400, 4, 24
    p = rng.integers(1, 300, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 60, size=(n_inst, n)).astype(np.uint32)
    for levels in ([(300, 30000)], [(400, 20000), (900, 41000), (2500, 90000)]):
        cm = (5, 5, 15000, 300, 16, 40, 350, levels)
        g = H.check_offline(hos, p, o, M, cap, 10 ** 6, cm, 3)
        lb = H.check_lower_bound(hos, p, o, M, cap, 10 ** 6, cm)
        assert (lb["tp_paper_us"] > 0).all()
        for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
            H.check_simulate(hos, p, o, M, cap, 10 ** 6, cm, g["assign"], LAMS, mode)
            H.check_simulate_steal(hos, p, o, M, cap, 10 ** 6, cm, g["assign"], (LAMBDA_NEVER_PREEMPT, LAMBDA_ONE), mode)
    # a prompt longer than the largest level can never be prefilled: the instance is invalid
    p2 = p.copy(); p2[2, 7] = 301
    cm = (5, 5, 15000, 300, 16, 40, 350, [(300, 30000)])
    g2 = H.gpu_simulate(hos, p2, o, M, cap, 10 ** 6, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED, want_trace=False)
    assert (g2["status"][2] == hos.HOS_ST_INVALID).all() and (g2["status"][:2] == 0).all()
    with pytest.raises(hos.HosError):                        # caps must ascend
        hos.hos_lower_bound(H.to_dev(p), H.to_dev(o), M, cap, 10 ** 6, (5, 5, 15000, 300, 16, 40, 350, [(300, 1), (300, 2)]))


def test_paper_shaped_workload(hos):
    from workload import paper_shaped
    w = paper_shaped(n_inst=6)
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    g = H.check_offline(hos, p, o, M, cap, kv, cm, 0)
    lb = H.check_lower_bound(hos, p, o, M, cap, kv, cm)
    hyb = H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED)
    base = H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_PREFILL_FIRST,), ora.QUEUE_FCFS)
    assert (lb["lb_sim_us"] <= hyb["sres"]["makespan_us"][:, 0]).all()
    assert (hyb["sres"]["utilisation"][:, 0] > base["sres"]["utilisation"][:, 0]).mean() >= 0.5


def test_estimated_output_lengths(hos):
    """Packing, queues and queued-token counts on estimates, simulation on the true lengths, a fixed
    reservation per request: batch of the c2e workload, plus small ragged cases with tight budgets."""
    w = workload("c2e").subset(0, 12)
    p, o = w.lengths()
    est = w.estimates()
    M, cap, kv, cm, R = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model, w.kv_reserve
    g = H.check_offline(hos, p, o, M, cap, kv, cm, 10, est=est, rsv=R)
    H.check_lower_bound(hos, p, o, M, cap, kv, cm, est=est, rsv=R)
    for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
        H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], LAMS, mode, insts=range(0, 12, 3), est=est, rsv=R)
    H.check_simulate_steal(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE, 20000), ora.QUEUE_SORTED,
                           insts=range(0, 12, 4), est=est, rsv=R)
    rng = np.random.default_rng(77)
    for n, M, cap, R, kv in ((37, 3, 5, 700, 2500), (130, 5, 4, 640, 640), (64, 2, 9, 900, 5000)):
        p = rng.integers(1, 300, (3, n)).astype(np.uint32)
        o = rng.integers(1, 300, (3, n)).astype(np.uint32)
        est = np.clip(np.rint(o * np.exp(0.6 * rng.standard_normal((3, n)))), 1, 400).astype(np.uint32)
        g = H.check_offline(hos, p, o, M, cap, kv, cm, 6, est=est, rsv=R)
        H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], LAMS, ora.QUEUE_SORTED, est=est, rsv=R)
        H.check_simulate_steal(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED, est=est, rsv=R)
    # estimates without a reservation, a reservation above the budget: refused on the host;
    # a request longer than the reservation: the instance is marked invalid on the device
    with pytest.raises(hos.HosError):
        hos.hos_offline_pack(H.to_dev(p), H.to_dev(o), M, cap, kv, cm, 0, o_est=H.to_dev(est))
    with pytest.raises(hos.HosError):
        hos.hos_offline_pack(H.to_dev(p), H.to_dev(o), M, cap, 500, cm, 0, kv_reserve=600)
    o2 = o.copy()
    o2[1, 5] = 900
    r = hos.hos_offline_pack(H.to_dev(p), H.to_dev(o2), M, cap, kv, cm, 0, o_est=H.to_dev(est), kv_reserve=R)
    assert r["status"].cpu().tolist() == [0, hos.HOS_ST_INVALID, 0]


def test_maximum_request_count(hos):
    """The largest instance the library takes (24,384 requests, 256 clients of 256 slots): the
    shared-memory sort is at its size limit and the lists span every client; one more request is
    refused on the host."""
    rng = np.random.default_rng(24576)
    n, M, cap = 24384, 256, 256
    p = rng.integers(1, 2000, size=(2, n)).astype(np.uint32)
    o = rng.integers(1, 150, size=(2, n)).astype(np.uint32)
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    kv = 1 << 20
    g = H.check_offline(hos, p, o, M, cap, kv, cm, 4, insts=[1])
    H.check_lower_bound(hos, p, o, M, cap, kv, cm)
    H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE, LAMBDA_PREFILL_FIRST), ora.QUEUE_SORTED,
                     insts=[0])
    H.check_simulate_steal(hos, p, o, 64, 64, kv, cm, g["assign"] % 64, (LAMBDA_ONE,), ora.QUEUE_SORTED, insts=[1])
    with pytest.raises(hos.HosError):
        hos.hos_offline_pack(H.to_dev(np.ones((1, n + 1), np.uint32)), H.to_dev(np.ones((1, n + 1), np.uint32)),
                             M, cap, kv, cm)


def test_limits_and_bad_data(hos):
    w = workload("c0")
    p, o = w.lengths()
    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    g = H.gpu_offline(hos, p, o, M, cap, kv, cm, 0)
    # iteration limit: truncated exactly like the oracle
    H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED, max_iters=37)
    # trace slots too small: records dropped, hash and counts intact, status bit set
    full = H.gpu_simulate(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED)
    small = H.gpu_simulate(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE,), ora.QUEUE_SORTED, trace_slots=40)
    assert (small["status_traced"] == hos.HOS_ST_TRACE).all()
    assert np.array_equal(small["cres"]["trace_hash"], full["cres"]["trace_hash"])
    for j in range(M):
        t0 = int(full["trace_off"][j])
        assert np.array_equal(small["trace"][40 * j:40 * j + 40], full["trace"][t0:t0 + 40])
    # a zero-length output marks the instance invalid without touching the others
    p2 = np.concatenate([p, p]); o2 = np.concatenate([o, o]).copy(); o2[1, 5] = 0
    g2 = H.gpu_offline(hos, p2, o2, M, cap, kv, cm, 3)
    assert g2["status"].tolist() == [0, hos.HOS_ST_INVALID]
    assert np.array_equal(g2["assign"][0], ora.offline_pack(p[0], o[0], M, cm, 3)["assign"])
    assert (g2["assign"][1] == -1).all() and g2["makespan_est"][1] == 0
    s2 = H.gpu_simulate(hos, p2, o2, M, cap, kv, cm, np.concatenate([g["assign"], g["assign"]]),
                        (LAMBDA_ONE,), ora.QUEUE_SORTED, want_trace=False)
    assert (s2["status"][1] == hos.HOS_ST_INVALID).all() and (s2["status"][0] == 0).all()
    assert s2["sres"]["makespan_us"][1, 0] == 0 and s2["sres"]["makespan_us"][0, 0] == full["sres"]["makespan_us"][0, 0]
    # host-side rejections
    with pytest.raises(hos.HosError):
        hos.hos_offline_pack(H.to_dev(p), H.to_dev(o), 0, cap, kv, cm)
    with pytest.raises(hos.HosError):
        hos.hos_offline_pack(H.to_dev(p), H.to_dev(o), 300, cap, kv, cm)


def test_values_beyond_the_arithmetic_range_are_flagged(hos):
    from paper_2502_15763_b200.binding import view_struct
    # (1) an estimated output length so long that the queue's sort key p + o_est does not fit beside
    #     the client number in 32 bits: that instance is invalid, its neighbours are unaffected
    rng = np.random.default_rng(31)
    n_inst, n, M, cap, kv, rsv = 3, 60, 4, 8, 10 ** 6, 400
    p = rng.integers(1, 200, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 100, size=(n_inst, n)).astype(np.uint32)
    est = o.copy()
    est[1, 7] = 0x7FFFFFF0
    cm = (20000, 40, 15000, 300, 16, 1, 1)                     # est_per_output_token = 1: T_i still fits 32 bits
    assign = rng.integers(0, M, size=(n_inst, n)).astype(np.int32)
    for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
        s = H.gpu_simulate(hos, p, o, M, cap, kv, cm, assign, (LAMBDA_ONE,), mode, want_trace=False, est=est, rsv=rsv)
        if mode == ora.QUEUE_SORTED:
            assert (s["status"][1] == hos.HOS_ST_INVALID).all() and s["sres"]["makespan_us"][1, 0] == 0
        ok = (0, 2) if mode == ora.QUEUE_SORTED else (0, 1, 2)      # FCFS does not sort by the estimate
        for k in ok:
            e = ora.simulate(assign[k], p[k], o[k], M, cm, cap, kv, LAMBDA_ONE, mode, o_est=est[k], kv_reserve=rsv)
            assert int(s["sres"]["makespan_us"][k, 0]) == e.makespan_us and (s["status"][k] == 0).all()
    r = hos.hos_online_simulate_steal(H.to_dev(p), H.to_dev(o), M, cap, kv, cm, H.to_dev(assign),
                                      H.to_dev(np.asarray([LAMBDA_ONE], np.uint32)), ora.QUEUE_SORTED,
                                      o_est=H.to_dev(est), kv_reserve=rsv)
    st = r["status"].cpu().numpy()
    assert (st[1] == hos.HOS_ST_INVALID).all() and (st[0] == 0).all() and (st[2] == 0).all()
    # (2) coefficients and token sums that are each inside their limits but whose product in the
    #     decode bound passes 64 bits: the bounds of that instance are zeroed and flagged
    n = 24000
    p = np.ones((2, n), dtype=np.uint32)
    o = np.ones((2, n), dtype=np.uint32)
    o[0] = 1000
    cm = (20000, 40, 1, 1 << 30, 1 << 10, 40, 350)
    r = hos.hos_lower_bound(H.to_dev(p), H.to_dev(o), 2, 1, 10 ** 6, cm)
    lb = view_struct(r["lb"], hos.LB_DTYPE)
    assert r["status"].cpu().tolist() == [hos.HOS_ST_RANGE, 0]
    assert all(int(lb[0][f]) == 0 for f in lb.dtype.names)
    e = ora.lower_bound(p[1], o[1], 2, 1, cm)
    assert all(int(lb[1][f]) == v for f, v in e.items())
    pk = hos.hos_offline_pack(H.to_dev(p), H.to_dev(o), 2, 1, 10 ** 6, cm, 0, want_lb=True)
    assert pk["status"].cpu().tolist() == [hos.HOS_ST_RANGE, 0] and (pk["assign"][0] >= 0).all()
    with pytest.raises(hos.HosError):                          # the sums themselves could pass 64 bits
        hos.hos_lower_bound(H.to_dev(p), H.to_dev(o), 2, 1, (1 << 31) - 1, cm)


@pytest.mark.parametrize("n,M,hi,scale,steps", [(7, 3, 6, 1, 64), (1, 1, 50, 1, 64), (40, 64, 300, 1, 64),
                                                 (97, 5, 20, 1, 64), (300, 8, 2000, 1, 64), (300, 8, 2000, 1, 1),
                                                 (300, 8, 2000, 1, 5), (1000, 33, 900, 1, 64), (700, 100, 400, 1, 7),
                                                 (2050, 256, 3000, 1, 64), (500, 4, 3000, 1000, 64),
                                                 (1300, 130, 60, 1, 64)])
def test_multifit_packing(hos, n, M, hi, scale, steps):
    """hos_offline_pack_multifit against the oracle's MULTIFIT: which packing is kept, the packing,
    and the local search that starts from it; step limits, ties, 64-bit loads (scale)."""
    rng = np.random.default_rng(n * 31 + M + steps)
    n_inst = 4
    p = rng.integers(1, hi + 1, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, hi // 3 + 2, size=(n_inst, n)).astype(np.uint32)
    p[1, ::3] = p[1, 0]                                            # runs of equal T
    o[1, ::3] = o[1, 0]
    cm = (20000, 40, 15000, 300, 16, 40 * scale, 350 * scale)
    g = H.check_offline(hos, p, o, M, 16, 10 ** 7, cm, 8, multifit_steps=steps)
    lb = H.check_lower_bound(hos, p, o, M, 16, 10 ** 7, cm)
    assert (lb["lb_pack"] <= g["makespan_est"]).all()
    plain = H.gpu_offline(hos, p, o, M, 16, 10 ** 7, cm, 0)
    mf = H.gpu_offline(hos, p, o, M, 16, 10 ** 7, cm, 0, multifit_steps=steps)
    assert (mf["makespan_est"] <= plain["makespan_est"]).all()
    assert ((mf["makespan_est"] < plain["makespan_est"]) == (mf["packer"] == 1)).all()


def test_multifit_on_the_configs(hos):
    for name, count in (("c0", 1), ("c1", 1), ("c2", 100), ("c4", 6)):
        w = workload(name).subset(0, count)
        p, o = w.lengths()
        H.check_offline(hos, p, o, w.n_clients, w.batch_cap, w.kv_budget, w.cost_model, min(w.ls_rounds, 30) or 10,
                        multifit_steps=64)
    # an invalid instance keeps its zeros and does not disturb its neighbour
    w = workload("c0")
    p, o = w.lengths()
    p2 = np.concatenate([p, p]); o2 = np.concatenate([o, o]).copy(); o2[0, 3] = 0
    g = H.gpu_offline(hos, p2, o2, w.n_clients, w.batch_cap, w.kv_budget, w.cost_model, 5, multifit_steps=64)
    e = ora.offline_pack(p[0], o[0], w.n_clients, w.cost_model, 5, multifit_steps=64)
    assert g["status"].tolist() == [hos.HOS_ST_INVALID, 0] and g["packer"][0] == 0
    assert np.array_equal(g["assign"][1], e["assign"]) and (g["assign"][0] == -1).all()


@pytest.mark.parametrize("kind", ["all_equal", "two_values", "wide_keys", "wide_keys_short", "one_heavy_bucket"])
def test_sort_falls_back_on_bunched_or_wide_keys(hos, kind):
    """Instances whose keys bunch into a few buckets, or are too wide for a bucket entry, take the
    radix sort instead of the bucket sort -- next to ordinary instances in the same batch."""
    rng = np.random.default_rng(len(kind))
    n_inst, n, M, cap = 3, 6000, 12, 24
    p = rng.integers(16, 3000, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(8, 900, size=(n_inst, n)).astype(np.uint32)
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    if kind == "all_equal":
        p[1] = 77; o[1] = 13
    elif kind == "two_values":
        p[1] = np.where(rng.random(n) < 0.5, 100, 101); o[1] = 50
    elif kind == "wide_keys":                      # T up to ~2^31: rest of the key + id pass 32 bits at this size
        n = 12000
        p = rng.integers(16, 3000, size=(n_inst, n)).astype(np.uint32)
        o = rng.integers(8, 900, size=(n_inst, n)).astype(np.uint32)
        cm = (20000, 40, 15000, 300, 16, 500000, 500000)
    elif kind == "wide_keys_short":                # the same keys still fit beside a 9-bit id
        n = 500
        p, o = p[:, :n].copy(), o[:, :n].copy()
        cm = (20000, 40, 15000, 300, 16, 500000, 500000)
    elif kind == "one_heavy_bucket":
        p[2, : n // 2] = 500; o[2, : n // 2] = rng.integers(100, 102, size=n // 2)
    kv = 10 ** 6
    g = H.check_offline(hos, p, o, M, cap, kv, cm, 3)
    H.check_lower_bound(hos, p, o, M, cap, kv, cm)
    for mode in (ora.QUEUE_SORTED, ora.QUEUE_FCFS):
        H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], (LAMBDA_ONE,), mode)


@pytest.mark.parametrize("n_inst", [600, 1300])
def test_multifit_on_large_batches(hos, n_inst):
    """Batches large enough that the packing kernel resolves two levels, or one level, of the
    bisection per round instead of three (the probe sequence must not depend on that)."""
    rng = np.random.default_rng(n_inst)
    n, M = 90, 7
    p = rng.integers(1, 900, size=(n_inst, n)).astype(np.uint32)
    o = rng.integers(1, 300, size=(n_inst, n)).astype(np.uint32)
    cm = (20000, 40, 15000, 300, 16, 40, 350)
    H.check_offline(hos, p, o, M, 8, 10 ** 6, cm, 4, multifit_steps=64)
