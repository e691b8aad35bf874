"""Seeded random shapes and option mixes through the C ABI against the CPU oracle (needs a GPU).

Every case draws a shape (requests, clients, slots, instances), length ranges with many ties, a KV
budget between "one request at a time" and "no limit", a KV divisor that is or is not a power of two,
optionally a stepped prefill cost, optionally estimated output lengths with a fixed reservation, a
few multiplier values and a queue order, and compares the packing, the local search (from the packing
and from a random assignment), the bounds, both simulators and the traces element by element."""
import numpy as np
import pytest

from oracle import hos_oracle as ora
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

LAMS_ALL = (0, 1000, 20000, 65536, 3 << 16, 1 << 20, 0xFFFFFFFF)


@pytest.fixture(scope="module")
def hos():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2502_15763_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("seed", range(4))
def test_random_cases(hos, seed):
    import torch
    rng = np.random.default_rng(1000 + seed)
    for _ in range(12):
        n, M, cap = int(rng.integers(1, 600)), int(rng.integers(1, 70)), int(rng.integers(1, 40))
        ninst = int(rng.integers(1, 4))
        pmax, omax = int(rng.choice([8, 300, 3000])), int(rng.choice([3, 120, 700]))
        p = rng.integers(1, pmax + 1, (ninst, n)).astype(np.uint32)
        o = rng.integers(1, omax + 1, (ninst, n)).astype(np.uint32)
        if rng.random() < 0.3:
            o[:, ::3] = 1
        if rng.random() < 0.3:
            p[:, ::4] = p[:, :1]
        need = int((p.astype(np.int64) + o).max())
        est, rsv, kv = None, 0, need * int(rng.choice([1, 2, 5, 1000]))
        if rng.random() < 0.3:
            est = np.clip(np.rint(o * np.exp(0.5 * rng.standard_normal(o.shape))), 1, 2 * omax).astype(np.uint32)
            rsv = need + int(rng.integers(0, 50))
            kv = rsv * int(rng.integers(1, 30))
        cm = [20000, 40, 15000, 300, int(rng.choice([16, 7, 1, 1 << 20])), 40, 350]
        if rng.random() < 0.25:
            top = int(p.max()) * int(rng.integers(1, 6))
            cm.append(tuple((top * (l + 1) // 3, 20000 + 100 * top * (l + 1) // 3) for l in range(3)))
        cm = tuple(cm)
        rounds = int(rng.choice([0, 1, 7, 30]))
        lams = tuple(int(x) for x in rng.choice(LAMS_ALL, size=int(rng.integers(1, 4)), replace=False))
        mode = int(rng.integers(0, 2))
        g = H.check_offline(hos, p, o, M, cap, kv, cm, rounds, est=est, rsv=rsv)
        H.check_lower_bound(hos, p, o, M, cap, kv, cm, est=est, rsv=rsv)
        H.check_simulate(hos, p, o, M, cap, kv, cm, g["assign"], lams, mode, est=est, rsv=rsv)
        if M * 32 * cap * 4 < 150000:          # the stealing simulator keeps one simulation's heaps in one CTA
            H.check_simulate_steal(hos, p, o, M, cap, kv, cm, g["assign"], lams[:1], mode, est=est, rsv=rsv)
        ra = rng.integers(0, M, (ninst, n)).astype(np.int32)
        r = hos.hos_local_search(H.to_dev(p), H.to_dev(o), M, cap, kv, cm, torch.from_numpy(ra[:, None, :].copy()).cuda(),
                                 max(rounds, 1), o_est=None if est is None else H.to_dev(est), kv_reserve=rsv)
        for k in range(ninst):
            T = ora.estimate(p[k], o[k] if est is None else est[k], cm)
            l0 = np.bincount(ra[k], weights=T.astype(np.float64), minlength=M).astype(np.int64)
            ea, el, _, _ = ora.local_search(T, ra[k], l0, max(rounds, 1))
            assert np.array_equal(r["assign"][k, 0].cpu().numpy(), ea)
            assert np.array_equal(r["load"][k, 0].cpu().numpy(), el)
