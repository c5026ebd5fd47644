"""The allocation-free histogram entry point against the regular one (needs a B200).

topoep_histogram_static serves callers that may not allocate device memory where they run (inside
someone else's capture region, with a frozen memory pool, ...): its per-tile scratch is a fixed
array inside the library.  Collected last on purpose, so that a run that stops at the first
failure has already run every other test.  It depends on nothing the other tests leave behind:
it passes alone in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import workloads as wl
from paper_2609_35481_b200 import Planner, binding as B

pytestmark = pytest.mark.gpu


def _regular(w, ids):
    pl = Planner(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k, w.tokens_per_rank,
                 max_batch=ids.shape[0], token_bytes=w.token_bytes, expert_bytes=w.expert_bytes,
                 main_rank=w.main_rank())
    omega = pl.histogram(torch.from_numpy(ids).cuda())
    torch.cuda.synchronize()
    flags = pl.status()
    pl.close()
    return omega, flags


def test_static_histogram_matches_regular_entry_point_twice_in_a_row():
    # first call: the DeepSeek-V3-shaped layer (16 tiles per rank); second call right after it: a
    # smaller, ragged shape, so anything stale in the shared scratch array would show up
    w1 = wl.CONFIGS["dsv3"]
    w2 = wl.CONFIGS["mid"].replace(tokens_per_rank=1023, top_k=3, nodes=2, gpus_per_node=3,
                                   experts=60)
    ids1 = wl.make_topk_ids(w1, seed=71)
    ids2 = wl.make_topk_ids(w2, seed=72, batch=2).copy()
    ids2[1, 4, 17, 2] = w2.experts + 5          # an out-of-range id: ignored and flagged
    ids2[0, 0, :9, :] = -1                      # padding: ignored silently
    flags = torch.full((1,), 123, dtype=torch.int32, device="cuda")   # must be cleared by the call
    for w, ids in ((w1, ids1), (w2, ids2)):
        want, want_flags = _regular(w, ids)
        dev = torch.from_numpy(ids).cuda()
        got = torch.full_like(want, -1)
        rc = B.topoep_histogram_static(dev, ids.shape[0], w.ranks, w.tokens_per_rank, w.top_k,
                                       w.experts, got, flags,
                                       torch.cuda.current_stream().cuda_stream)
        assert rc == B.OK, B.topoep_strerror(rc)
        torch.cuda.synchronize()
        assert torch.equal(got, want)           # integer counts: exact
        assert int(flags.item()) == want_flags
        for b in range(ids.shape[0]):
            for s in range(w.ranks):
                row = ids[b, s].ravel()
                row = row[(row >= 0) & (row < w.experts)]
                assert np.array_equal(got[b, s].cpu().numpy(), np.bincount(row, minlength=w.experts))


def test_static_histogram_rejects_what_does_not_fit_its_array():
    w = wl.CONFIGS["scaleout"]                  # 128 ranks x 32 tiles x 512 experts x 4 B = 8 MiB + 256
    out = torch.empty((1, w.ranks, w.experts), dtype=torch.int32, device="cuda")
    ids = torch.zeros((1, w.ranks, 8, w.top_k), dtype=torch.int32, device="cuda")
    rc = B.topoep_histogram_static(ids, 1, w.ranks, w.tokens_per_rank, w.top_k, w.experts, out, None, 0)
    assert rc == -11 and "scratch" in B.topoep_strerror(rc)
    assert B.topoep_histogram_static(ids, 1, w.ranks, 8, w.top_k, w.experts, None, None, 0) == -1
    assert B.topoep_histogram_static(ids, 0, w.ranks, 8, w.top_k, w.experts, out, None, 0) == 0
    # the same shape with few tokens fits and works
    rc = B.topoep_histogram_static(ids, 1, w.ranks, 8, w.top_k, w.experts, out, None, 0)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(out[0, :, 0].sum()) == w.ranks * 8 * w.top_k and int(out[0, :, 1:].sum()) == 0
