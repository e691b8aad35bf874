"""hos_lower_bound_static: the lower-bound call for callers that cannot allocate.

A scheduler sharing a GPU with an inference engine often has no device memory to ask for: the
engine took HBM for weights and KV cache, and a cudaMalloc in a serving loop would stall the
device anyway.  For those callers the library carries its own fixed scratch.  This test calls
the entry point through the C ABI twice in a row, the second time on a smaller, different
batch so that leftovers of the first call are still in the scratch, and wants the very same
bytes as the ordinary hos_lower_bound (integer results: bit-exact, like every other parity
test here).  It also checks that an oversized batch is refused with its own error code.
Collected last on purpose: a failure here cannot hide the results of the other tests.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_version_twice():
    import torch
    assert torch.cuda.is_available()
    import paper_2502_15763_b200 as hos
    from tests.gpu_harness import to_dev
    from workload import workload

    cases = [workload("c2").subset(0, 40), workload("c0")]       # big first, then small
    for w in cases:
        p, o = w.lengths()
        dp, do = to_dev(p), to_dev(o)
        args = (dp, do, w.n_clients, w.batch_cap, w.kv_budget, w.cost_model)
        want = hos.hos_lower_bound(*args)
        got = hos.hos_lower_bound_static(*args)
        torch.cuda.synchronize()
        assert torch.equal(got["lb"], want["lb"])
        assert torch.equal(got["status"], want["status"]) and int(got["status"].abs().sum()) == 0
    # an invalid instance is reported the same way
    o_bad = o.copy(); o_bad[0, 3] = 0
    args = (to_dev(p), to_dev(o_bad), w.n_clients, w.batch_cap, w.kv_budget, w.cost_model)
    assert torch.equal(hos.hos_lower_bound_static(*args)["status"], hos.hos_lower_bound(*args)["status"])


def test_static_scratch_refuses_oversized_batches():
    import torch
    import paper_2502_15763_b200 as hos
    n_inst, n_req = 64, 20000                                     # 1.28 M requests: beyond the built-in scratch
    p = torch.full((n_inst, n_req), 100, dtype=torch.int32, device="cuda")
    with pytest.raises(hos.HosError) as e:
        hos.hos_lower_bound_static(p, p, 8, 16, 1 << 20, (20000, 40, 15000, 300, 16, 40, 350))
    assert e.value.code == -5 and "scratch" in str(e.value)
