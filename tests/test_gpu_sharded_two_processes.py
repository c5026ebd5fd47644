"""The sharded deployment form with TWO processes through the CUDA path (needs a B200).

Paper, "GPU-Native Load Balancer": every rank gathers the routing information of the EP group
and derives the same plan, no coordinator.  Here two processes share the one GPU of the test box,
each owning half of the source ranks, and talk over a gloo group (the gathered rows go through
host memory; no peer memory, no NCCL, nothing that needs a second GPU).  Each calls
Planner.plan_sharded: own histogram rows -> all-gather -> row permutation -> the whole group's plan
from the same matrix -> per-token assignment of its own ids.  Both must hold the oracle's plan bit
for bit, and their per-token outputs together must be the oracle's.  The kernels of the two
processes never wait on one another: each process runs its own complete launches.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = [
    ("mid", dict(slots_per_rank=3), 2),                         # both solver stages act
    ("dsv3", dict(tokens_per_rank=2051), 1),                    # ragged tile, every slot taken
    ("tiny", dict(slots_per_rank=2, tokens_per_rank=777), 3),   # refinement only
]


def _worker(rank, world, port, case, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import torch.distributed as dist
    import oracle as orc
    import workloads as wl
    from gpu_common import make_planner, oracle_config
    from paper_2609_35481_b200 import binding as B
    name, over, batch = case
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=33, batch=batch)               # the same seeded buffer everywhere
    ref = orc.plan(oracle_config(w), ids)
    cnt = w.ranks // world
    mine = np.ascontiguousarray(ids[:, rank * cnt:(rank + 1) * cnt])
    pl = make_planner(w, max_batch=batch)
    for rep in range(2):                                          # twice: nothing stale carries over
        res = pl.plan_sharded(torch.from_numpy(mine).to(pl.device))
        torch.cuda.synchronize()
        for field in ("replica_map", "dispatch_counts", "dispatch_offsets", "instance_counts"):
            got = getattr(res, field).cpu().numpy()
            assert np.array_equal(got, getattr(ref, field)), (rank, rep, field)
        got = res.token_replica.cpu().numpy()
        assert got.shape == mine.shape
        assert np.array_equal(got, ref.token_replica[:, rank * cnt:(rank + 1) * cnt]), (rank, rep)
        assert np.array_equal(pl.debug_tensor(B.T_Q, batch).numpy(), ref.q_instances)
        assert pl.status() == ref.flags
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, int(res.token_replica.shape[1])))


@pytest.mark.parametrize("case", CASES, ids=lambda c: c[0])
def test_plan_sharded_with_two_processes_on_one_gpu(case):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, case, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=300)
        assert p.exitcode == 0
    got = sorted(out.get(timeout=5) for _ in range(2))
    import workloads as wl
    ranks = wl.CONFIGS[case[0]].replace(**case[1]).ranks
    assert got == [(0, ranks // 2), (1, ranks // 2)]             # the two windows cover every rank
