"""Parity cases run against the bounds-checked build of the CUDA library (a script, not a test
module: tests/test_gpu_checked_build.py runs it in a process of its own with
TOPOEP_CHECKED_BUILD=1, because a process loads one build of the library).

In that build every index that is derived from data is checked; an index out of range would set
TOPOEP_FLAG_INTERNAL and be clamped.  The cases are the small, ragged and degenerate shapes where
an indexing mistake would show first.  Exit code 0: every case matched the oracle bit for bit and
no check fired.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))


def main():
    assert os.environ.get("TOPOEP_CHECKED_BUILD") == "1"
    import torch
    import oracle as orc
    import workloads as wl
    from gpu_common import assert_same, make_planner, oracle_config, run_gpu
    from paper_2609_35481_b200 import binding as B, build
    B.lib()
    assert os.path.exists(build.CHECKED_LIB)
    cases = [
        ("tiny", dict(), 2), ("tiny", dict(slots_per_rank=3), 2), ("tiny", dict(slots_per_rank=0), 1),
        ("tiny", dict(tokens_per_rank=1, top_k=1), 1), ("tiny", dict(tokens_per_rank=7, top_k=3), 2),
        ("tiny", dict(tokens_per_rank=1025, top_k=2, slots_per_rank=2), 2),
        ("tiny", dict(tokens_per_rank=4097, top_k=1, slots_per_rank=2), 1),
        ("mid", dict(tokens_per_rank=777, top_k=5, slots_per_rank=3), 2),
        ("mid", dict(nodes=1, gpus_per_node=8, experts=64, slots_per_rank=2, tokens_per_rank=1000), 1),
        ("tiny", dict(nodes=8, gpus_per_node=1, tokens_per_rank=3000), 1),
        ("tiny", dict(nodes=40, gpus_per_node=1, experts=80, slots_per_rank=2, top_k=4,
                      tokens_per_rank=700, zipf_s=0.9, ffn=2), 1),
        ("tiny", dict(nodes=3, gpus_per_node=4, experts=600, slots_per_rank=24, top_k=8,
                      tokens_per_rank=2048, zipf_s=0.3, ffn=1, hidden=32), 1),
        ("dsv3", dict(tokens_per_rank=2051), 1),
        ("scaleout", dict(tokens_per_rank=512), 1),
    ]
    n = 0
    for name, over, batch in cases:
        w = wl.CONFIGS[name].replace(**over)
        ids = wl.make_topk_ids(w, seed=17, batch=batch).copy()
        ids[0, 0, :1, :] = -1                     # some padding
        ref = orc.plan(oracle_config(w), ids)
        for chain, packed in ((1, 1), (1, 2), (2, 0), (3, 0)):
            pl = make_planner(w, max_batch=batch)
            pl.set_tuning(B.KNOB_CHAIN, chain)
            pl.set_tuning(B.KNOB_PACKED_IDS, packed)   # 2: the one-byte id copy and the multi-tile reroute kernel
            pl.set_tuning(B.KNOB_REROUTE_TILES, 3)
            for rep in range(2):
                gpu = run_gpu(pl, ids)
                assert_same(gpu, ref)
                assert gpu["flags"] == ref.flags == 0, (name, over, chain, packed, gpu["flags"])
            # the dispatch permutation and the replica copies on the same plan
            out = pl.plan(torch.from_numpy(ids).to(pl.device))
            send, recv, off = pl.dispatch_positions(out.token_replica)
            cfg = oracle_config(w)
            s_ref, r_ref, o_ref = orc.dispatch_positions(cfg, ref.token_replica[0])
            assert np.array_equal(send[0].cpu().numpy(), s_ref)
            assert np.array_equal(recv[0].cpu().numpy(), r_ref)
            assert pl.status() == 0
            pl.close()
            n += 1
    print("checked build: %d planner runs, no index check fired" % n)


if __name__ == "__main__":
    main()
