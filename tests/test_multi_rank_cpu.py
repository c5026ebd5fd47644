"""The multi-rank host logic of bench.py on CPU (gloo, world size 2).

The planning path does not shard: N GPUs run N independent replicas on their own seeded batches
and there is no collective on the data path.  What the ranks do share is the measurement protocol:
disjoint seeded inputs per rank, a barrier, the maximum over ranks of the device time, and one
aggregate throughput.  This test runs exactly those helpers in two gloo processes.
"""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    import oracle as orc
    import workloads as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.CONFIGS["tiny"]
    ids = wl.make_topk_ids(w, seed=wl.BASE_SEED, plan_base=bench.rank_plan_base(rank, 0))
    again = wl.make_topk_ids(w, seed=wl.BASE_SEED, plan_base=bench.rank_plan_base(rank, 0))
    assert np.array_equal(ids, again)                       # deterministic per rank
    # every rank plans its own batch; the plans differ across ranks (independent replicas)
    cfg = orc.OracleConfig(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                           w.token_bytes, w.expert_bytes, main_rank=w.main_rank())
    omega = torch.from_numpy(orc.plan(cfg, ids, want_tokens=False).omega.astype(np.int64))
    gathered = [torch.zeros_like(omega) for _ in range(world)]
    dist.all_gather(gathered, omega)
    assert not torch.equal(gathered[0], gathered[1])
    # the slowest rank sets the time; the job's throughput counts every rank's assignments
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, torch.device("cpu"))
    assert ms == 10.0 * world
    value = bench.job_throughput(world, w.assignments, 4, ms)
    assert value == world * w.assignments * 4 / (ms * 1e-3)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, float(value)))


def test_two_rank_protocol_on_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    got = sorted(out.get(timeout=5) for _ in range(2))
    assert got[0][1] == got[1][1]                           # every rank reports the same job value


def _sharded_worker(rank, world, port, out):
    """Sharded deployment on the host: a process that owns a window of source ranks contributes
    only those rows of the routing matrix; after the all-gather every process solves the same
    matrix with the same deterministic rules and must hold the same plan, with no coordinator."""
    sys.path.insert(0, ROOT)
    import oracle as orc
    import workloads as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.CONFIGS["tiny"].replace(slots_per_rank=2)
    cfg = orc.OracleConfig(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                           w.token_bytes, w.expert_bytes, main_rank=w.main_rank())
    ids = wl.make_topk_ids(w, seed=5)[0]                    # [R][T][k]; each process reads its rows
    per = w.ranks // world
    mine = ids[rank * per:(rank + 1) * per]
    rows = torch.from_numpy(np.stack([np.bincount(r.ravel(), minlength=w.experts) for r in mine]))
    gathered = [torch.zeros_like(rows) for _ in range(world)]
    dist.all_gather(gathered, rows)
    omega = torch.cat(gathered).numpy()
    res = orc.solve(cfg, omega)
    whole = orc.plan(cfg, ids[None], want_tokens=True)
    assert np.array_equal(omega, whole.omega[0])
    assert np.array_equal(res.slotmap, whole.replica_map[0])
    digest = torch.from_numpy(np.concatenate([res.slotmap.ravel(), res.q.ravel(), res.L]).astype(np.int64))
    theirs = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(theirs, digest)
    assert all(torch.equal(t, digest) for t in theirs)      # bitwise-identical plans on all ranks
    # each process deals its own tokens from the shared plan: the union is the single-process result
    tr = orc.assign_tokens(cfg, res, ids)[rank * per:(rank + 1) * per]
    assert np.array_equal(tr, whole.token_replica[0][rank * per:(rank + 1) * per])
    dist.barrier()
    dist.destroy_process_group()
    out.put(rank)


def test_sharded_ranks_hold_identical_plans_on_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_sharded_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert sorted(out.get(timeout=5) for _ in range(2)) == [0, 1]


def test_plan_bases_are_disjoint():
    sys.path.insert(0, ROOT)
    import bench
    seen = set()
    for rank in range(8):
        for i in range(32):
            base = bench.rank_plan_base(rank, i)
            span = set(range(base, base + 232))
            assert not (seen & span)
            seen |= span
