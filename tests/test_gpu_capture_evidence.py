"""Evidence that a plan is enqueue-only (needs a B200): what a timeline tool would show.

The target statement asks for a plan that is "CUDA-graph-capturable with zero D2H copies or host
syncs".  No timeline profiler is installed here, so the claim is checked three ways:
  * stream capture around topoep_plan succeeds (a synchronisation, a pageable copy or an
    allocation inside would fail it) -- tests/test_gpu_parity.py;
  * the captured graph is taken apart: every node must be a kernel node, and there must be as
    many as the library says a plan has kernels;
  * an activity trace of graph replays is read back: only this library's kernels may appear on
    the device, no copy of any kind, and no synchronisation call on the host between the replays.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import workloads as wl
from gpu_common import make_planner, oracle_config
from paper_2609_35481_b200 import binding as B

pytestmark = pytest.mark.gpu


def _cudart():
    try:
        from cuda.bindings import runtime as rt
    except Exception:   # older cuda-python layout
        from cuda import cudart as rt
    return rt


def _check(res):
    err = res[0]
    assert int(err) == 0, "CUDA runtime call failed: %s" % (err,)
    return res[1:] if len(res) > 2 else (res[1] if len(res) == 2 else None)


@pytest.mark.parametrize("name,chain,batch", [("dsv3", 0, 1), ("dsv3", 1, 1), ("tiny", 2, 2),
                                              ("scaleout", 0, 1), ("mid", 3, 2), ("dsv3", 11, 2)])
def test_captured_plan_is_kernel_nodes_only(name, chain, batch):
    # chain 11: five kernels with the one-byte copy of the ids (histogram writes, reroute reads it)
    packed = chain == 11
    chain = 1 if packed else chain
    rt = _cudart()
    w = wl.CONFIGS[name]
    ids = wl.make_topk_ids(w, seed=5, batch=batch)
    pl = make_planner(w, max_batch=batch)
    pl.set_tuning(B.KNOB_CHAIN, chain)
    if packed:
        pl.set_tuning(B.KNOB_PACKED_IDS, 2)
        assert B.topoep_plan_byte_copy(pl.handle, w.tokens_per_rank, batch) == 1
    dev_ids = torch.from_numpy(ids).to(pl.device)
    out = pl.alloc_outputs(batch, w.tokens_per_rank)
    pl.plan(dev_ids, out)                        # first call outside capture
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    _check(rt.cudaStreamBeginCapture(stream.cuda_stream,
                                     rt.cudaStreamCaptureMode.cudaStreamCaptureModeThreadLocal))
    pl.plan(dev_ids, out, stream=stream)
    graph = _check(rt.cudaStreamEndCapture(stream.cuda_stream))
    _, n = _check(rt.cudaGraphGetNodes(graph, 0))
    nodes, n = _check(rt.cudaGraphGetNodes(graph, n))
    kinds = [_check(rt.cudaGraphNodeGetType(node)) for node in nodes[:n]]
    kernel = rt.cudaGraphNodeType.cudaGraphNodeTypeKernel
    assert all(k == kernel for k in kinds), kinds     # no memcpy, memset, host or event node
    assert n == B.topoep_plan_kernels(pl.handle, w.tokens_per_rank, batch)
    # by size: two kernels for a small plan, four for a single 128-rank plan; forced otherwise
    assert n == {("dsv3", 0): 2, ("dsv3", 1): 5, ("tiny", 2): 2, ("scaleout", 0): 4, ("mid", 3): 4}[(name, chain)]
    if packed:   # the captured launches are the byte-copy pair, not the plain kernels
        from torch.profiler import ProfilerActivity, profile
        with profile(activities=[ProfilerActivity.CUDA]) as prof:
            pl.plan(dev_ids, out)
            torch.cuda.synchronize()
        launched = [e.name for e in prof.events() if str(e.device_type).endswith("CUDA")]
        assert any("reroute_rows_kernel" in k for k in launched), launched
    # the graph still does the work: instantiate, replay, compare with the oracle
    exe = _check(rt.cudaGraphInstantiate(graph, 0))
    out.token_replica.fill_(-7)
    torch.cuda.synchronize()
    for _ in range(2):
        _check(rt.cudaGraphLaunch(exe, stream.cuda_stream))
    stream.synchronize()
    ref = orc.plan(oracle_config(w), ids)
    assert np.array_equal(out.token_replica.cpu().numpy(), ref.token_replica)
    assert np.array_equal(out.dispatch_offsets.cpu().numpy(), ref.dispatch_offsets)
    assert pl.status() == 0
    _check(rt.cudaGraphExecDestroy(exe))
    _check(rt.cudaGraphDestroy(graph))


@pytest.mark.parametrize("name,chain", [("dsv3", 0), ("mid", 1)])
def test_activity_trace_of_replays_has_no_copy_and_no_host_sync(name, chain):
    from torch.profiler import ProfilerActivity, profile
    w = wl.CONFIGS[name]
    ids = wl.make_topk_ids(w, seed=6)
    pl = make_planner(w)
    pl.set_tuning(B.KNOB_CHAIN, chain)
    dev_ids = torch.from_numpy(ids).to(pl.device)
    out = pl.alloc_outputs(1, w.tokens_per_rank)
    pl.plan(dev_ids, out)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            pl.plan(dev_ids, out, stream=stream)
        graph.replay()
    torch.cuda.synchronize()
    replays = 20
    with profile(activities=[ProfilerActivity.CPU, ProfilerActivity.CUDA]) as prof:
        with torch.cuda.stream(stream):
            for _ in range(replays):
                graph.replay()
            done = torch.cuda.Event()
            done.record(stream)
        # the trace is closed by waiting on an event OUTSIDE the replay loop
        while not done.query():
            pass
    events = list(prof.events())
    names = [e.name for e in events]
    device = [e.name for e in events if str(e.device_type).endswith("CUDA")]
    lowered = [n.lower() for n in names]
    assert not any("memcpy" in n for n in lowered), [n for n in names if "emcpy" in n]
    assert not any("memset" in n for n in lowered), [n for n in names if "emset" in n]
    # host synchronisation: none from the first replay's launch to the last one's (the profiler
    # itself synchronises the device when it stops, after the window)
    launches = [e for e in events if e.name == "cudaGraphLaunch"]
    assert len(launches) == replays
    t0 = min(e.time_range.start for e in launches)
    t1 = max(e.time_range.end for e in launches)
    inside = [e.name for e in events
              if "synchronize" in e.name.lower() and t0 <= e.time_range.start <= t1]
    assert not inside, inside
    ours = [n for n in device if "topoep" in n]
    kernels = B.topoep_plan_kernels(pl.handle, w.tokens_per_rank, 1)
    assert len(device) > 0 and len(ours) == len(device), set(device) - set(ours)
    assert len(ours) == replays * kernels, (len(ours), replays, kernels)
    assert pl.status() == 0
