"""Host-side multi-rank logic on CPU: two gloo ranks shard instances without overlap, agree on the
max-over-ranks time, and use no data-path collective."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import hos_oracle as ora
    from workload import shard, workload
    # strong split of one workload: contiguous, disjoint, complete
    w = workload("c2")
    first, count = shard(w.n_inst, world, rank)
    spans = [None] * world
    dist.all_gather_object(spans, (first, count))
    # weak scaling as bench.py does it: same count per rank, disjoint seeds
    wr = bench.rank_workload("c2", rank, instances=3)
    seeds = [None] * world
    dist.all_gather_object(seeds, wr.seeds)
    # each rank evaluates its own instances with no exchange; results are just concatenated
    p, o = wr.lengths()
    mk = [ora.offline_pack(p[k], o[k], wr.n_clients, wr.cost_model)["makespan_est"] for k in range(wr.n_inst)]
    allmk = [None] * world
    dist.all_gather_object(allmk, mk)
    # timing reduction: max over ranks
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        out.put(dict(spans=spans, seeds=seeds, mk=allmk, t=float(t.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_without_overlap():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res["spans"] == [(0, 50), (50, 50)]
    assert res["seeds"][0] == (100, 101, 102) and res["seeds"][1] == (103, 104, 105)
    assert res["t"] == 11.0
    # the gathered results equal a single-process evaluation of the same seeds
    from oracle import hos_oracle as ora
    from workload import Workload, workload
    w = workload("c2")
    for r in range(2):
        wr = Workload(w.name, res["seeds"][r], w.n_req, w.n_clients, w.batch_cap, w.kv_budget, w.dist_p, w.dist_o)
        p, o = wr.lengths()
        assert res["mk"][r] == [ora.offline_pack(p[k], o[k], w.n_clients, w.cost_model)["makespan_est"]
                                for k in range(3)]
