"""The benchmark's end-to-end stream of batches (pinned host tables in, pinned host results out, two sets
of device tables) against results that the oracle has checked (needs a GPU)."""
import numpy as np
import pytest

from oracle import hos_oracle as ora
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hos():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2502_15763_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("name,steps", [("c2", 1), ("c2", 2), ("c2", 5), ("c2e", 4)])
def test_stream_of_batches(hos, name, steps):
    """The device tables are created from one seed and the host tables then replaced by another seed's, so
    a step that read tables which its own upload had not (yet) written gives other results; `steps` ends
    on the first set of tables (odd) or on the second (even)."""
    import torch
    import bench
    from paper_2502_15763_b200.binding import view_struct
    w0 = bench.rank_workload(name, 0)
    w = bench.rank_workload(name, 1)
    pipe = bench.Pipeline(w0, torch.device("cuda", 0))
    pipe.prepare()
    p, o = w.lengths()
    est = w.estimates()
    assert not np.array_equal(p, w0.lengths()[0])
    pipe.p_host.copy_(torch.from_numpy(p.view(np.int32)))
    pipe.o_host.copy_(torch.from_numpy(o.view(np.int32)))
    if est is not None:
        pipe.est_host.copy_(torch.from_numpy(est.view(np.int32)))
    host_out = []
    ms, h2d, d2h = pipe.e2e_run(steps, host_out, None)
    assert ms > 0
    assert h2d == p.nbytes + o.nbytes + 4 * len(w.lambdas_q16) + (0 if est is None else est.nbytes)
    assert d2h == sum(t.numel() * t.element_size() for t in host_out)
    assign, load, mk, st, lb_raw, cres_raw, sres_raw, sim_st = host_out

    M, cap, kv, cm = w.n_clients, w.batch_cap, w.kv_budget, w.cost_model
    ek = dict(est=est, rsv=w.kv_reserve)
    g = H.check_offline(hos, p, o, M, cap, kv, cm, w.ls_rounds, **ek)
    lb = H.check_lower_bound(hos, p, o, M, cap, kv, cm, **ek)
    s = H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], w.lambdas_q16, ora.QUEUE_SORTED,
                         want_trace=False, **ek)
    assert np.array_equal(assign.numpy(), g["assign"])
    assert np.array_equal(load.numpy(), g["load"])
    assert np.array_equal(mk.numpy(), g["makespan_est"])
    assert np.array_equal(st.numpy(), g["status"])
    assert np.array_equal(view_struct(lb_raw, hos.LB_DTYPE), lb)
    assert np.array_equal(view_struct(cres_raw, hos.CLIENT_RESULT_DTYPE), s["cres"])
    assert np.array_equal(view_struct(sres_raw, hos.SIM_RESULT_DTYPE), s["sres"])
    assert np.array_equal(sim_st.numpy(), s["status"])
