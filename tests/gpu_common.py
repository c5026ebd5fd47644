"""Shared helpers of the GPU parity tests: run the CUDA library through its C boundary and the
CPU oracle on the same seeded buffer, compare every output bit for bit."""
from __future__ import annotations

import numpy as np
import torch

import oracle as orc
import workloads as wl
from paper_2609_35481_b200 import Planner, binding as B


def oracle_config(w: wl.Workload, **over) -> orc.OracleConfig:
    kw = dict(nodes=w.nodes, gpus_per_node=w.gpus_per_node, experts=w.experts,
              slots_per_rank=w.slots_per_rank, top_k=w.top_k, token_bytes=w.token_bytes,
              expert_bytes=w.expert_bytes, c_intra=w.c_intra, c_inter=w.c_inter, t_ffn=w.t_ffn)
    kw.update(over)
    if "main_rank" not in kw:
        kw["main_rank"] = w.main_rank()
    return orc.OracleConfig(**kw)


def make_planner(w: wl.Workload, max_batch=None, max_tokens=None, **over) -> Planner:
    kw = dict(nodes=w.nodes, gpus_per_node=w.gpus_per_node, experts=w.experts,
              slots_per_rank=w.slots_per_rank, top_k=w.top_k,
              max_tokens_per_rank=max_tokens or max(w.tokens_per_rank, 1),
              max_batch=max_batch or w.batch, token_bytes=w.token_bytes,
              expert_bytes=w.expert_bytes, c_intra=w.c_intra, c_inter=w.c_inter, t_ffn=w.t_ffn)
    kw.update(over)
    if "main_rank" not in kw:
        kw["main_rank"] = w.main_rank()
    return Planner(**kw)


def run_gpu(pl: Planner, ids: np.ndarray):
    """Plan ids [B][R][T][k] on the GPU; returns dict of numpy outputs + intermediates."""
    dev = torch.from_numpy(np.ascontiguousarray(ids)).to(pl.device)
    out = pl.plan(dev)
    Bn = ids.shape[0]
    res = dict(replica_map=out.replica_map.cpu().numpy(),
               token_replica=out.token_replica.cpu().numpy(),
               dispatch_counts=out.dispatch_counts.cpu().numpy(),
               dispatch_offsets=out.dispatch_offsets.cpu().numpy(),
               instance_counts=out.instance_counts.cpu().numpy())
    res["omega"] = pl.debug_tensor(B.T_OMEGA, Bn).numpy()
    res["q_instances"] = pl.debug_tensor(B.T_Q, Bn).numpy()
    res["rank_load"] = pl.debug_tensor(B.T_RANK_LOAD, Bn).numpy()
    res["refine_iters"] = pl.debug_tensor(B.T_REFINE_ITERS, Bn).numpy()
    res["demand"] = pl.debug_tensor(B.T_D, Bn).numpy()
    res["inst_load"] = pl.debug_tensor(B.T_U, Bn).numpy()
    res["dims"] = (pl.M, pl.G)
    res["summaries"] = pl.summary(Bn)
    res["flags"] = pl.status()
    return res


FIELDS = ("omega", "replica_map", "q_instances", "rank_load", "refine_iters", "instance_counts",
          "dispatch_counts", "dispatch_offsets", "token_replica")


def assert_same(gpu: dict, ref: orc.PlanResult, plans=None):
    """Bit-exact comparison of every integer output; summaries field by field."""
    for name in FIELDS:
        g = gpu[name]
        r = getattr(ref, name)
        if plans is not None:
            g = g[plans]
        assert g.shape == r.shape, (name, g.shape, r.shape)
        if not np.array_equal(g, r):
            bad = np.argwhere(g != r)
            raise AssertionError("%s differs at %d places, first %s: gpu %s oracle %s"
                                 % (name, len(bad), bad[0].tolist(), g[tuple(bad[0])], r[tuple(bad[0])]))
    # the two remaining intermediates: domain demand D = the routing matrix summed over the ranks
    # of a domain (the solver reads it when it runs inter-node placement), per-instance load U
    M, G = gpu["dims"]
    D, U = gpu["demand"], gpu["inst_load"]
    if plans is not None:
        D, U = D[plans], U[plans]
    om = ref.omega.astype(np.int64)
    assert np.array_equal(D, om.reshape(om.shape[0], M, G, -1).sum(axis=2)), "demand"
    assert np.array_equal(U, ref.instance_counts), "instance load"
    gs = gpu["summaries"] if plans is None else gpu["summaries"][plans]
    for name in orc.SUMMARY_INT_FIELDS:
        assert np.array_equal(gs[name], ref.summaries[name]), name
    for name in orc.SUMMARY_FLOAT_FIELDS:
        np.testing.assert_allclose(gs[name], ref.summaries[name], rtol=1e-6, atol=0)


def parity(w: wl.Workload, seed: int, batch=None, ids=None, planner=None, **cfg_over):
    """Full-path parity of one workload; returns (gpu dict, oracle result, ids)."""
    if ids is None:
        ids = wl.make_topk_ids(w, seed=seed, batch=batch)
    pl = planner or make_planner(w, max_batch=max(ids.shape[0], 1), **cfg_over)
    gpu = run_gpu(pl, ids)
    ref = orc.plan(oracle_config(w, **cfg_over), ids)
    assert_same(gpu, ref)
    assert gpu["flags"] == ref.flags
    return gpu, ref, ids
