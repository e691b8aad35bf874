"""Input generators: Philox known answers, determinism, distribution shape, sharding."""
import numpy as np

from workload import LengthDist, instance_lengths, philox4x32_10, shard, workload


def test_philox_known_answers():
    # known-answer vectors published with the Random123 library for philox4x32-10
    out = philox4x32_10(np.array([0], dtype=np.uint64), 0, 0)
    assert [int(w[0]) for w in out] == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]


def test_lengths_deterministic_and_clipped():
    w = workload("c4")
    p1, o1 = instance_lengths(1000, 5000, w.dist_p, w.dist_o)
    p2, o2 = instance_lengths(1000, 5000, w.dist_p, w.dist_o)
    assert p1.dtype == np.uint32 and np.array_equal(p1, p2) and np.array_equal(o1, o2)
    assert p1.min() >= 16 and p1.max() <= 4096 and o1.min() >= 8 and o1.max() <= 2048
    # prefix property: instance tables do not depend on n_req
    p3, _ = instance_lengths(1000, 100, w.dist_p, w.dist_o)
    assert np.array_equal(p3, p1[:100])
    # different seeds give different tables
    p4, _ = instance_lengths(1001, 5000, w.dist_p, w.dist_o)
    assert not np.array_equal(p1, p4)


def test_lognormal_moments():
    d = LengthDist(120.0, 0.4, 1, 10 ** 6)
    p, _ = instance_lengths(7, 200000, d, d)
    lp = np.log(p.astype(np.float64))
    assert abs(lp.mean() - np.log(120.0)) < 0.01
    assert abs(lp.std() - 0.4) < 0.01


def test_config_shapes():
    for name, n_inst, n_req, M in (("c0", 1, 200, 4), ("c1", 1, 1300, 8), ("c2", 100, 1300, 8),
                                   ("c3", 100, 1300, 8), ("c4", 1024, 20000, 64)):
        w = workload(name)
        assert (w.n_inst, w.n_req, w.n_clients) == (n_inst, n_req, M)
    w3 = workload("c3")
    assert len(w3.lambdas_q16) == 64 and w3.lambdas_q16[15] == 65536 and w3.ls_rounds == 20
    assert workload("c4").ls_rounds == 100
    p, o = workload("c2").subset(3, 2).lengths()
    assert p.shape == (2, 1300)


def test_shard_partitions():
    for n in (0, 1, 7, 100, 1024):
        for ws in (1, 2, 3, 8):
            spans = [shard(n, ws, r) for r in range(ws)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == n
            for (f0, c0), (f1, _) in zip(spans, spans[1:]):
                assert f0 + c0 == f1
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1
