"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here touches CUDA.  Each test pins one part of oracle/topoep_oracle.c
to something other than itself: the paper's two worked examples, fixtures
derived by hand from the solver's prose, library routines (bincount, cumsum),
closed forms, the constraints C1-C5, per-iteration half-gap invariants, and the
exact optimum of the paper's MILP on tiny instances.
"""
import json
import os

import numpy as np
import pytest

import oracle as orc
import workloads as wl
from plan_checks import check_plan, dispatch_positions_by_sorting, objective

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MiB = 1 << 20


def _load(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return json.load(f)


def _cfg(d, **over):
    kw = dict(d)
    kw.update(over)
    mr = kw.pop("main_rank", None)
    return orc.OracleConfig(main_rank=None if mr is None else np.array(mr, np.int32), **kw)


def _omega(cfg, sparse):
    om = np.zeros((cfg.ranks, cfg.experts), np.int64)
    for s, e, v in sparse:
        om[s, e] = v
    return om


def _cross(cfg, q):
    dom = np.arange(cfg.ranks) // cfg.gpus_per_node
    return int(q.sum(axis=1)[dom[:, None] != dom[None, :]].sum())


def _q_dense(cfg, sparse):
    q = np.zeros((cfg.ranks, cfg.experts, cfg.ranks), np.int64)
    for s, e, r, v in sparse:
        q[s, e, r] = v
    return q


# ----------------------------------------------------------------------------------------------
# Worked example 1: "Topology-Dependent Cost" (64 MiB of token traffic vs 18 + 9 MiB).
# ----------------------------------------------------------------------------------------------
def test_cost_example_matches_paper_bytes():
    g = _load("cost_example.json")
    pv = g["paper_values"]
    s_tok = pv["hidden"] * pv["activation_bytes_per_element"]
    W = pv["expert_bytes_MiB"] * MiB
    assert g["config"]["token_bytes"] == s_tok and g["config"]["expert_bytes"] == W
    om = np.array(g["omega"], np.int64)

    # placement (a): the one replica sits on node 1 next to the main instance (what refinement
    # alone does: rank 2's 8192 are halved onto rank 3); node 0's 4096 assignments cross nodes
    cfg_a = _cfg(g["config"], stages=2)
    ra = orc.solve(cfg_a, om)
    sa = orc.summary(cfg_a, ra)
    assert sa["cross_assignments"] == pv["tokens_per_node"]
    # exposed half = 2*D*S_tok; forward+backward total = twice that = the paper's 64 MiB
    assert 2 * sa["cross_token_bytes"] == pv["token_traffic_fwd_bwd_MiB"] * MiB
    assert sa["t_token"] == sa["cross_token_bytes"]          # c_inter = 1, c_intra = 0
    assert sa["t_replica"] == 0 and sa["replicas_inter"] == 0 and sa["replicas_intra"] == 1
    assert ra.slotmap.tolist() == [[-1], [-1], [-1], [0]]

    # placement (b): what inter-node placement does (b = 32 MiB - 9 MiB > 0)
    cfg_b = _cfg(g["config"], stages=1)
    rb = orc.solve(cfg_b, om)
    sb = orc.summary(cfg_b, rb)
    assert rb.slotmap.tolist() == [[0], [-1], [-1], [-1]]
    assert sb["cross_assignments"] == 0 and sb["cross_token_bytes"] == 0
    assert sb["l_max"] == pv["tokens_per_node"] == sa["l_max"]   # same L_max in both placements
    assert sb["replicas_inter"] == 1
    assert sb["t_replica"] == W                                  # one forward parameter transfer
    # two fetches (buffers are reused across layers) + one gradient push
    assert 2 * sb["t_replica"] == pv["parameter_traffic_MiB"] * MiB
    assert 3 * sb["t_replica"] == (pv["parameter_traffic_MiB"] + pv["replica_gradient_traffic_MiB"]) * MiB
    ratio = (2 * sa["cross_token_bytes"]) / (3 * sb["t_replica"])
    assert round(ratio, 1) == pv["reduction_factor_approx"]


def test_c4_is_strict_at_the_threshold():
    # 2*D*S_tok == W exactly: the paper's criterion is a strict inequality, so no replica.
    cfg = orc.OracleConfig(2, 1, 2, 1, 1, token_bytes=4, expert_bytes=80)
    om = np.array([[0, 10], [0, 0]], np.int64)       # D[0][1] = 10 -> 2*10*4 = 80 = W
    assert orc.solve(cfg, om).slotmap.tolist() == [[-1], [-1]]
    om[0, 1] = 11
    assert orc.solve(cfg, om).slotmap.tolist() == [[1], [-1]]


# ----------------------------------------------------------------------------------------------
# Worked example 2: the two-stage figure (loads 14/6 -> 10/10, 4 assignments moved).
# ----------------------------------------------------------------------------------------------
def test_two_stage_example_matches_paper():
    g = _load("two_stage_example.json")
    pv = g["paper_values"]
    cfg = _cfg(g["config"])
    om = _omega(cfg, g["omega_sparse"])
    assert om[0, 4] == pv["assignments_gpu0_to_E4"] and cfg.main_rank[4] == pv["main_of_E4"]

    r0 = orc.solve(_cfg(g["config"], stages=0), om)
    assert r0.L.tolist() == g["expect_no_placement"]["L"]
    assert orc.summary(cfg, r0)["replica_served"] == 0        # every assignment on a main instance
    assert _cross(cfg, r0.q) == g["expect_no_placement"]["cross"] == pv["assignments_gpu0_to_E4"]

    r1 = orc.solve(_cfg(g["config"], stages=1), om)
    assert r1.slotmap.tolist() == g["expect_stage1"]["slotmap"]
    assert r1.L.tolist() == g["expect_stage1"]["L"]
    assert r1.L[:2].tolist() == pv["loads_gpu0_gpu1_after_inter_node"]
    assert _cross(cfg, r1.q) == 0
    # the eight assignments now execute on the replica E4' (GPU 0)
    assert orc.summary(cfg, r1)["replica_served"] == pv["E4_assignments_on_replicas"]

    r = orc.solve(cfg, om, trace_cap=8)
    ex = g["expect_final"]
    assert r.slotmap.tolist() == ex["slotmap"] and r.L.tolist() == ex["L"]
    assert r.L[:2].tolist() == pv["loads_after_refinement"]
    assert r.iters.tolist() == ex["iters"]
    assert len(r.trace) == 1
    row = dict(zip(orc.TRACE_FIELDS, r.trace[0].tolist()))
    for key, val in ex["trace"][0].items():
        assert row[key] == val
    assert row["delta"] == pv["moved_by_refinement"]
    assert _cross(cfg, r.q) == pv["new_cross_domain_routes"]
    # four stay on E4', four moved to E4'': all eight are executed by replicas, none by GPU 2
    sm = orc.summary(cfg, r)
    assert sm["replica_served"] == pv["E4_assignments_on_replicas"]
    assert sm["replica_fraction"] == pv["E4_assignments_on_replicas"] / om.sum()
    assert r.q[0, 4].tolist() == [4, 4, 0, 0]


@pytest.mark.parametrize("variant", ["variant_cost_tiebreak", "variant_cost_uses_main_rank"])
def test_two_stage_example_cost_tiebreak_variant(variant):
    g = _load("two_stage_example.json")
    v = g[variant]
    cfg = _cfg(g["config"])
    r = orc.solve(cfg, _omega(cfg, v["omega_sparse"]), trace_cap=8)
    assert r.slotmap.tolist() == v["expect_final"]["slotmap"]
    assert r.L.tolist() == v["expect_final"]["L"]
    assert r.iters.tolist() == v["expect_final"]["iters"] and len(r.trace) == 1
    row = dict(zip(orc.TRACE_FIELDS, r.trace[0].tolist()))
    for key, val in v["expect_final"]["trace"][0].items():
        assert row[key] == val


# ----------------------------------------------------------------------------------------------
# Hand-derived fixtures: one per ordering / tie-break / remainder rule.
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("case", _load("hand_derived.json")["cases"], ids=lambda c: c["name"])
def test_hand_derived_fixture(case):
    cfg = _cfg(case["config"], stages=case["stages"])
    om = _omega(cfg, case["omega_sparse"])
    r = orc.solve(cfg, om, trace_cap=32)
    ex = case["expect"]
    assert r.slotmap.tolist() == ex["slotmap"]
    assert (r.q == _q_dense(cfg, ex["q_sparse"])).all()
    assert r.iters.tolist() == ex["iters"]
    if "L" in ex:
        assert r.L.tolist() == ex["L"]
    if "cross" in ex:
        assert _cross(cfg, r.q) == ex["cross"]
    if "replica_served" in ex:
        # executed by a replica = on a rank other than main(e), whatever its domain
        summ = orc.summary(cfg, r)
        assert summ["replica_served"] == ex["replica_served"]
        assert summ["replica_fraction"] == ex["replica_served"] / om.sum()
    if "trace" in ex:
        assert len(r.trace) == len(ex["trace"])
        for got, want in zip(r.trace, ex["trace"]):
            row = dict(zip(orc.TRACE_FIELDS, got.tolist()))
            for key, val in want.items():
                assert row[key] == val, (key, row, want)


# ----------------------------------------------------------------------------------------------
# Library routines and closed forms.
# ----------------------------------------------------------------------------------------------
def _wl_cfg(w, **over):
    kw = dict(nodes=w.nodes, gpus_per_node=w.gpus_per_node, experts=w.experts,
              slots_per_rank=w.slots_per_rank, top_k=w.top_k, token_bytes=w.token_bytes,
              expert_bytes=w.expert_bytes, c_intra=w.c_intra, c_inter=w.c_inter, t_ffn=w.t_ffn,
              main_rank=w.main_rank())
    kw.update(over)
    return orc.OracleConfig(**kw)


def test_histogram_is_bincount_and_flags_bad_ids():
    w = wl.CONFIGS["tiny"]
    ids = wl.make_topk_ids(w, seed=7)[0].copy()
    ids[0, 0, 0] = -1          # padding: ignored, no flag
    cfg = _wl_cfg(w)
    om, flags = orc.histogram(cfg, ids)
    for s in range(w.ranks):
        row = ids[s].ravel()
        assert (om[s] == np.bincount(row[row >= 0], minlength=w.experts)).all()
    assert flags == 0
    ids[1, 5, 1] = w.experts   # out of range: ignored and flagged
    ids[2, 9, 0] = -7
    om2, flags2 = orc.histogram(cfg, ids)
    assert flags2 == orc.FLAG_BAD_ID
    assert om2.sum() == om.sum() - 2


def test_layout_is_cumsum_of_counts():
    w = wl.CONFIGS["tiny"]
    ids = wl.make_topk_ids(w, seed=11)
    cfg = _wl_cfg(w)
    p = orc.plan(cfg, ids)
    c = p.dispatch_counts[0].astype(np.int64)
    assert (p.dispatch_offsets[0, 0, :, 1:] == np.cumsum(c, axis=1)).all()
    assert (p.dispatch_offsets[0, 1, :, 1:] == np.cumsum(c.T, axis=1)).all()
    assert (p.dispatch_offsets[0, :, :, 0] == 0).all()
    assert (p.dispatch_offsets[0, 1, :, -1] == p.rank_load[0]).all()


@pytest.mark.parametrize("M,G", [(2, 2), (4, 2), (2, 4)])
def test_identity_plan_and_inter_node_fraction_closed_form(M, G):
    # No slots: every assignment goes to its main rank; with equal demand from every source to
    # every expert and mains spread evenly, the inter-node fraction is exactly (M-1)/M (the
    # 50.0% / 75.0% the paper reports for static placement over 2 / 4 nodes).
    R = M * G
    E = 2 * R
    cfg = orc.OracleConfig(M, G, E, 0, 1, token_bytes=1, expert_bytes=1)
    om = np.full((R, E), 5, np.int64)
    r = orc.solve(cfg, om)
    assert (r.x.sum(axis=1) == 1).all()
    for e in range(E):
        assert (r.q[:, e, cfg.main_rank[e]] == 5).all()
    s = orc.summary(cfg, r)
    assert s["cross_assignments"] * M == s["assignments"] * (M - 1)
    assert s["cross_fraction"] == pytest.approx((M - 1) / M, rel=1e-12)
    assert s["replica_served"] == 0 and s["imbalance"] == 1.0


def test_huge_expert_and_balanced_load_is_identity():
    cfg = orc.OracleConfig(2, 2, 8, 2, 1, token_bytes=2, expert_bytes=1 << 50)
    om = np.full((4, 8), 3, np.int64)
    r = orc.solve(cfg, om)
    assert (r.slotmap == -1).all() and r.iters.sum() == 0
    assert (r.L == r.L[0]).all()


def test_single_domain_skips_inter_node_placement():
    # One NVLink domain: nothing to evaluate in stage 1, the plan is refinement only.
    w = wl.CONFIGS["tiny"].replace(nodes=1, gpus_per_node=8)
    ids = wl.make_topk_ids(w, seed=3)
    a = orc.plan(_wl_cfg(w), ids)
    b = orc.plan(_wl_cfg(w, stages=2), ids)
    assert (a.replica_map == b.replica_map).all() and (a.token_replica == b.token_replica).all()
    assert a.summaries[0]["replicas_inter"] == 0 and a.summaries[0]["cross_assignments"] == 0


def test_uniform_routing_leaves_stage_one_idle():
    w = wl.CONFIGS["mid"].replace(uniform=True, tokens_per_rank=512)
    ids = wl.make_topk_ids(w, seed=5)
    p = orc.plan(_wl_cfg(w, stages=1), ids)
    assert (p.replica_map == -1).all()


# ----------------------------------------------------------------------------------------------
# Constraints C1-C5 and structural properties on every kind of plan.
# ----------------------------------------------------------------------------------------------
SHAPES = [
    ("tiny", {}),
    ("tiny", {"slots_per_rank": 3}),
    ("mid", {"tokens_per_rank": 512, "slots_per_rank": 3}),
    ("dsv3", {"tokens_per_rank": 1024, "slots_per_rank": 4}),
    ("mid", {"tokens_per_rank": 300, "nodes": 1, "gpus_per_node": 8, "experts": 64}),
    ("scaleout", {"tokens_per_rank": 256}),
]


@pytest.mark.parametrize("name,over", SHAPES)
def test_constraints_hold_on_synthetic_plans(name, over):
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=101, batch=2)
    cfg = _wl_cfg(w)
    p = orc.plan(cfg, ids)
    for b in range(2):
        info = check_plan(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                          cfg.main_rank, w.token_bytes, w.expert_bytes, ids[b], p.replica_map[b],
                          p.token_replica[b], p.dispatch_counts[b], p.dispatch_offsets[b],
                          p.instance_counts[b], p.rank_load[b])
        assert (info["omega"] == p.omega[b]).all()
        # q(s, instance) rows sum to omega per expert (C1) and are zero on unused instances (C2)
        qi = p.q_instances[b].astype(np.int64)
        ie = info["inst_expert"]
        assert (qi[:, ie < 0] == 0).all()
        for s in range(w.ranks):
            per_e = np.bincount(ie[ie >= 0], weights=qi[s][ie >= 0], minlength=w.experts)
            assert (per_e.astype(np.int64) == p.omega[b, s]).all()
        assert (qi.sum(axis=0) == p.instance_counts[b]).all()


def _random_instance(rng, M, G, E, N):
    R = M * G
    main = rng.integers(0, R, size=E).astype(np.int32) if rng.random() < 0.5 else None
    if main is None and E % R:
        main = (np.arange(E) % R).astype(np.int32)
    s_tok = int(rng.integers(1, 4))
    W = int(rng.integers(1, 40))
    cfg = orc.OracleConfig(M, G, E, N, 1, token_bytes=s_tok, expert_bytes=W,
                           c_intra=int(rng.integers(0, 3)), c_inter=int(rng.integers(1, 9)),
                           t_ffn=int(rng.integers(0, 50)), main_rank=main)
    om = rng.integers(0, 30, size=(R, E)) * (rng.random((R, E)) < 0.5)
    return cfg, om.astype(np.int64)


def test_solver_invariants_and_half_gap_on_random_instances():
    rng = np.random.default_rng(20260935)
    for trial in range(300):
        M, G = int(rng.integers(1, 4)), int(rng.integers(1, 5))
        E, N = int(rng.integers(1, 13)), int(rng.integers(0, 4))
        cfg, om = _random_instance(rng, M, G, E, N)
        R = cfg.ranks
        r = orc.solve(cfg, om, trace_cap=4096)
        stage1 = orc.solve(orc.OracleConfig(**{**cfg.__dict__, "stages": 1}), om)
        dom = np.arange(R) // G
        # C1, C2, C3, C5
        assert (r.q.sum(axis=2) == om).all()
        assert (r.q.transpose(1, 2, 0) <= om.T[:, None, :] * r.x[:, :, None]).all()
        assert (r.x[np.arange(E), cfg.main_rank] == 1).all()
        nonmain = r.x.copy()
        nonmain[np.arange(E), cfg.main_rank] = 0
        assert (nonmain.sum(axis=0) <= N).all()
        # slot map and x agree
        for rr in range(R):
            assert sorted(e for e in r.slotmap[rr] if e >= 0) == np.nonzero(nonmain[:, rr])[0].tolist()
        # C4 for every cross-domain instance
        for e, rr in zip(*np.nonzero(nonmain)):
            if dom[rr] != dom[cfg.main_rank[e]]:
                assert 2 * r.D[dom[rr], e] * cfg.token_bytes > cfg.expert_bytes
        # loads
        assert (r.U == r.q.sum(axis=0)).all() and (r.L == r.U.sum(axis=0)).all()
        # refinement never puts an expert into a domain that lacked it after stage 1, never adds
        # cross-domain assignments, and never raises a domain's maximum load
        host1 = np.array([[stage1.x[e, dom == d].any() for d in range(M)] for e in range(E)])
        host2 = np.array([[r.x[e, dom == d].any() for d in range(M)] for e in range(E)])
        assert (host1 == host2).all()
        assert _cross(cfg, r.q) == _cross(cfg, stage1.q)
        for d in range(M):
            assert r.L[dom == d].max() <= stage1.L[dom == d].max()
            assert r.L[dom == d].sum() == stage1.L[dom == d].sum()
        # every commit obeys the half-gap bound: order of source and target is not reversed
        assert len(r.trace) == r.iters.sum()
        for row in r.trace:
            t = dict(zip(orc.TRACE_FIELDS, row.tolist()))
            assert t["delta"] >= 1 and dom[t["r_b"]] == dom[t["r_t"]] == t["d"]
            assert t["L_b"] - t["delta"] >= t["L_t"] + t["delta"]
        # termination: no rank pair of a domain is left with a feasible move
        assert r.flags == 0


def test_refinement_cap_is_an_input_and_is_flagged():
    cfg = orc.OracleConfig(1, 4, 4, 2, 1, token_bytes=1, expert_bytes=1, max_refine_iters=2)
    om = np.zeros((4, 4), np.int64)
    om[0, 0] = 100
    r = orc.solve(cfg, om)
    assert r.iters.tolist() == [2] and r.flags == orc.FLAG_REFINE_CAP
    free = orc.solve(orc.OracleConfig(1, 4, 4, 2, 1, token_bytes=1, expert_bytes=1), om)
    assert free.flags == 0 and free.iters[0] > 2
    assert free.L.max() - free.L.min() <= 1


# ----------------------------------------------------------------------------------------------
# Per-token assignment (O7) against brute-force counting.
# ----------------------------------------------------------------------------------------------
def test_token_assignment_brute_force():
    rng = np.random.default_rng(5)
    for trial in range(20):
        M, G, E, N, k, T = 2, 2, 6, 2, 2, 40
        main = (np.arange(E) % (M * G)).astype(np.int32)
        cfg = orc.OracleConfig(M, G, E, N, k, token_bytes=1, expert_bytes=int(rng.integers(1, 30)),
                               main_rank=main)
        ids = rng.integers(-1, E, size=(M * G, T, k)).astype(np.int32)   # duplicates and padding
        om, _ = orc.histogram(cfg, ids)
        r = orc.solve(cfg, om)
        out = orc.assign_tokens(cfg, r, ids)
        s_phys = cfg.s_phys
        # brute force: list each (s,e) group's assignments in flat order and cut it by quota
        for s in range(M * G):
            flat = ids[s].ravel()
            for e in range(E):
                pos = [f for f in range(flat.size) if flat[f] == e]
                cursor = 0
                for rr in range(M * G):
                    n = int(r.q[s, e, rr])
                    for f in pos[cursor:cursor + n]:
                        p = out[s].ravel()[f]
                        assert p // s_phys == rr
                    cursor += n
                assert cursor == len(pos)
            assert (out[s].ravel()[flat < 0] == -1).all()


def test_dispatch_positions_are_the_sorted_order():
    # O10 against numpy.lexsort: the send buffer is the assignments of a source sorted by
    # (instance, flat index), the receive buffer those of a rank sorted by (instance, source, flat)
    for name, over in (("tiny", dict(slots_per_rank=2)), ("mid", dict(tokens_per_rank=300, slots_per_rank=3))):
        w = wl.CONFIGS[name].replace(**over)
        ids = wl.make_topk_ids(w, seed=17).copy()
        ids[0, 1, 5:9, :] = -1
        cfg = _wl_cfg(w)
        p = orc.plan(cfg, ids)
        send, recv, off = orc.dispatch_positions(cfg, p.token_replica[0])
        s2, r2, o2 = dispatch_positions_by_sorting(w.ranks, cfg.s_phys, p.token_replica[0])
        assert (send.reshape(w.ranks, -1) == s2).all()
        assert (recv.reshape(w.ranks, -1) == r2).all()
        assert (off == o2).all()
        # the offsets are the exclusive scan of the instance counts, the last one is L_r
        U = p.instance_counts[0].reshape(w.ranks, cfg.s_phys)
        assert (off[:, 1:] == np.cumsum(U, axis=1)).all() and (off[:, -1] == p.rank_load[0]).all()
        # a source's block for destination rank r starts at its send offset
        tr = p.token_replica[0].reshape(w.ranks, -1)
        for s in range(w.ranks):
            for r in range(w.ranks):
                sel = (tr[s] >= 0) & (tr[s] // cfg.s_phys == r)
                if sel.any():
                    assert send.reshape(w.ranks, -1)[s][sel].min() == p.dispatch_offsets[0, 0, s, r]


# ----------------------------------------------------------------------------------------------
# The MILP of the paper's formulation, solved exactly on tiny instances.
# ----------------------------------------------------------------------------------------------
def _milp_optimum(cfg, om):
    from scipy.optimize import milp, LinearConstraint, Bounds
    M, G, E, N = cfg.nodes, cfg.gpus_per_node, cfg.experts, cfg.slots_per_rank
    R = M * G
    dom = np.arange(R) // G
    C = np.where(dom[:, None] == dom[None, :], cfg.c_intra, cfg.c_inter).astype(float)
    np.fill_diagonal(C, 0)
    D = om.reshape(M, G, E).sum(axis=1)
    nx, nq = E * R, R * E * R
    xi = lambda e, r: e * R + r
    qi = lambda s, e, r: nx + (s * E + e) * R + r
    lm = nx + nq
    nvar = lm + 1
    cost = np.zeros(nvar)
    cost[lm] = cfg.t_ffn
    for s in range(R):
        for e in range(E):
            for r in range(R):
                cost[qi(s, e, r)] = 2 * cfg.token_bytes * C[s, r]
    lb, ub = np.zeros(nvar), np.full(nvar, np.inf)
    for e in range(E):
        for r in range(R):
            ub[xi(e, r)] = 1
            m = cfg.main_rank[e]
            if r == m:
                lb[xi(e, r)] = 1                                     # C5
            else:
                cost[xi(e, r)] = C[m, r] * cfg.expert_bytes
                if dom[r] != dom[m] and not (cfg.expert_bytes < 2 * D[dom[r], e] * cfg.token_bytes):
                    ub[xi(e, r)] = 0                                 # C4
    rows, lo, hi = [], [], []
    for s in range(R):
        for e in range(E):
            a = np.zeros(nvar)
            for r in range(R):
                a[qi(s, e, r)] = 1
            rows.append(a); lo.append(om[s, e]); hi.append(om[s, e])          # C1
            for r in range(R):
                a = np.zeros(nvar)
                a[qi(s, e, r)] = 1
                a[xi(e, r)] = -om[s, e]
                rows.append(a); lo.append(-np.inf); hi.append(0)              # C2
    for r in range(R):
        a = np.zeros(nvar)
        for e in range(E):
            if cfg.main_rank[e] != r:
                a[xi(e, r)] = 1
        rows.append(a); lo.append(-np.inf); hi.append(N)                      # C3
        a = np.zeros(nvar)
        for s in range(R):
            for e in range(E):
                a[qi(s, e, r)] = 1
        a[lm] = -1
        rows.append(a); lo.append(-np.inf); hi.append(0)                      # L_r <= L_max
    integrality = np.ones(nvar)
    integrality[lm] = 0
    res = milp(cost, constraints=LinearConstraint(np.array(rows), lo, hi), integrality=integrality,
               bounds=Bounds(lb, ub))
    assert res.status == 0, res.message
    return res.fun


def test_plans_are_feasible_and_bounded_by_the_milp_optimum():
    rng = np.random.default_rng(77)
    gaps = []
    for trial in range(25):
        M, G = (2, 2) if trial % 2 else (1, 3)
        E = int(rng.integers(2, 7))
        cfg, om = _random_instance(rng, M, G, E, int(rng.integers(0, 3)))
        r = orc.solve(cfg, om)
        tc, tt, trp = objective(M, G, cfg.main_rank, cfg.token_bytes, cfg.expert_bytes, cfg.c_intra,
                                cfg.c_inter, cfg.t_ffn, r.x, r.q)
        s = orc.summary(cfg, r)
        assert (tc, tt, trp) == (s["t_comp"], s["t_token"], s["t_replica"])
        opt = _milp_optimum(cfg, om)
        assert tc + tt + trp >= opt - 1e-6
        if opt > 0:
            gaps.append((tc + tt + trp) / opt)
    # the heuristic claims no optimum: the gap is reported, only its sign is asserted
    print("objective / MILP optimum: min %.3f median %.3f max %.3f over %d instances"
          % (min(gaps), float(np.median(gaps)), max(gaps), len(gaps)))
    assert min(gaps) >= 1 - 1e-9


def test_forced_optimum_is_reached():
    # One hot expert, one free slot, two ranks of one domain, compute dominating the objective:
    # the optimum splits the load in half through one replica, and so does refinement.
    cfg = orc.OracleConfig(1, 2, 2, 1, 1, token_bytes=1, expert_bytes=10, c_intra=1, c_inter=8,
                           t_ffn=1000)
    om = np.array([[10, 0], [0, 0]], np.int64)
    r = orc.solve(cfg, om)
    total = sum(objective(1, 2, cfg.main_rank, 1, 10, 1, 8, 1000, r.x, r.q))
    assert total == 1000 * 5 + 2 * 1 * 1 * 5 + 1 * 10
    assert total == pytest.approx(_milp_optimum(cfg, om))
    # and across two single-GPU domains with a demand that justifies the parameter transfer,
    # inter-node placement reaches the optimum of the communication terms (t_ffn = 0)
    cfg2 = orc.OracleConfig(2, 1, 2, 1, 1, token_bytes=4, expert_bytes=40, c_intra=1, c_inter=2,
                            t_ffn=0)
    om2 = np.array([[0, 9], [0, 0]], np.int64)
    r2 = orc.solve(cfg2, om2)
    assert sum(objective(2, 1, cfg2.main_rank, 4, 40, 1, 2, 0, r2.x, r2.q)) == \
        pytest.approx(_milp_optimum(cfg2, om2))


# ----------------------------------------------------------------------------------------------
# Qualitative agreement with the evaluation section.
# ----------------------------------------------------------------------------------------------
def test_one_slot_starves_refinement_more_slots_balance():
    # "With one slot the ratio remains [high] ... with two slots [it] drops": with one slot
    # stage 1 takes every slot; from two slots on refinement has room and imbalance does not rise.
    w = wl.CONFIGS["dsv3"].replace(tokens_per_rank=2048)
    ids = wl.make_topk_ids(w, seed=9)
    imb = []
    for n in (0, 1, 2, 3, 4):
        p = orc.plan(_wl_cfg(w, slots_per_rank=n), ids, want_tokens=False, want_q=False)
        imb.append(p.summaries[0]["imbalance"])
    assert imb[1] < imb[0]
    assert imb[2] <= imb[1] and imb[3] <= imb[2] + 1e-12 and imb[4] <= imb[3] + 1e-12
    assert imb[4] < 1.5


def test_summary_floats_are_the_integer_ratios():
    w = wl.CONFIGS["tiny"]
    ids = wl.make_topk_ids(w, seed=2)
    s = orc.plan(_wl_cfg(w), ids).summaries[0]
    assert s["assignments"] == w.assignments
    assert s["imbalance"] == s["l_max"] * w.ranks / s["assignments"]
    assert s["cross_fraction"] == s["cross_assignments"] / s["assignments"]
    assert s["replica_fraction"] == s["replica_served"] / s["assignments"]
    assert s["t_comp"] == w.t_ffn * s["l_max"]


# ---- O11 / O12: replica parameter pull and gradient return ---------------------------------------
def _transfer_cfg(fx):
    return orc.OracleConfig(fx["nodes"], fx["gpus_per_node"], fx["experts"], fx["slots_per_rank"], 1, 0, 0,
                            main_rank=np.array(fx["main_rank"], np.int32))


def test_replica_pull_and_grad_return_hand_written_bytes():
    fx = _load("replica_transfer.json")
    cfg = _transfer_cfg(fx)
    rmap = np.array(fx["replica_map"], np.int32)
    after = orc.replica_pull(cfg, rmap, np.array(fx["main_params"], np.uint8),
                             np.array(fx["replica_before"], np.uint8))
    assert np.array_equal(after, np.array(fx["replica_after_pull"], np.uint8))
    R, W = cfg.ranks, fx["param_bytes"]
    expect = np.zeros((R, R, cfg.e_loc, W), np.uint8)
    for m, s, l, b in fx["grad_acc_entries"]:
        expect[m, s, l] = b
    got = orc.replica_grad_return(cfg, rmap, np.array(fx["replica_grads"], np.uint8),
                                  np.zeros_like(expect))
    assert np.array_equal(got, expect)


@pytest.mark.parametrize("seed", range(4))
def test_replica_transfers_identity_code(seed):
    """Every byte of expert e's main block is e: a pulled slot must read back its own map entry,
    an empty slot its old bytes; returned gradients coded (source, slot) must land once each in
    the region [main(e)][source], and pull followed by return reproduces the main block there."""
    rng = np.random.default_rng(seed)
    M, G, E, N, W = 2, 3, 24, 3, 48
    R = M * G
    main_rank = rng.integers(0, R, E).astype(np.int32)
    cfg = orc.OracleConfig(M, G, E, N, 1, 0, 0, main_rank=main_rank)
    e_loc = cfg.e_loc
    mp = np.full((R, e_loc, W), 255, np.uint8)
    nxt = np.zeros(R, int)
    where = {}
    for e in range(E):
        mp[main_rank[e], nxt[main_rank[e]]] = e
        where[e] = (int(main_rank[e]), int(nxt[main_rank[e]]))
        nxt[main_rank[e]] += 1
    rmap = np.full((R, N), -1, np.int32)
    for r in range(R):
        others = [e for e in range(E) if main_rank[e] != r]
        n = int(rng.integers(0, N + 1))
        rmap[r, :n] = rng.choice(others, n, replace=False)
    before = np.full((R, N, W), 254, np.uint8)
    after = orc.replica_pull(cfg, rmap, mp, before)
    assert np.array_equal(after[:, :, 0], np.where(rmap >= 0, rmap, 254).astype(np.uint8))
    assert (after == after[:, :, :1]).all()
    # backward, bytes coded by (source rank, slot)
    grads = (np.arange(R)[:, None, None] * 16 + np.arange(N)[None, :, None]
             + np.zeros((1, 1, W), int)).astype(np.uint8)
    acc = orc.replica_grad_return(cfg, rmap, grads, np.full((R, R, e_loc, W), 253, np.uint8))
    written = 0
    for r in range(R):
        for j in range(N):
            if rmap[r, j] >= 0:
                m, l = where[int(rmap[r, j])]
                assert (acc[m, r, l] == r * 16 + j).all()
                written += 1
    assert (acc != 253).sum() == written * W          # nothing else was touched
    # pull then return: the main rank gets its own parameters back in the source's region
    acc2 = orc.replica_grad_return(cfg, rmap, after, np.full((R, R, e_loc, W), 253, np.uint8))
    for r in range(R):
        for j in range(N):
            if rmap[r, j] >= 0:
                m, l = where[int(rmap[r, j])]
                assert np.array_equal(acc2[m, r, l], mp[m, l])


# ---- policy variant: slots reserved for the refinement -------------------------------------------
def _skewed_case(seed, nodes=2, gpus=4, experts=32, slots=3, tokens=600, k=2):
    w = wl.CONFIGS["tiny"].replace(nodes=nodes, gpus_per_node=gpus, experts=experts,
                                   slots_per_rank=slots, tokens_per_rank=tokens, top_k=k,
                                   zipf_s=1.4, ffn=16)   # small experts: many candidates
    ids = wl.make_topk_ids(w, seed=seed)
    return w, ids


@pytest.mark.parametrize("seed", range(3))
def test_reserved_slots_stage1_takes_the_top_candidates_only(seed):
    """With r slots reserved, inter-node placement alone (stages = 1) must fill exactly the
    (N - r) * G best candidates of each domain, in the order (benefit down, expert id up), dealt
    round-robin over the ranks -- recomputed here with a plain sort."""
    w, ids = _skewed_case(seed)
    M, G, E, N = w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank
    mr = w.main_rank()
    for reserve in (0, 1, 2, 3):
        cfg = orc.OracleConfig(M, G, E, N, w.top_k, w.token_bytes, w.expert_bytes, main_rank=mr,
                               stages=1, reserve_slots=reserve)
        res = orc.plan(cfg, ids)
        omega = res.omega[0]
        D = omega.reshape(M, G, E).sum(axis=1)
        for d in range(M):
            b = 2 * D[d] * w.token_bytes - w.expert_bytes
            cands = [e for e in range(E) if mr[e] // G != d and b[e] > 0]
            cands.sort(key=lambda e: (-b[e], e))
            assert len(cands) > (N - 1) * G          # the capacity binds whenever reserve >= 1
            take = cands[:(N - reserve) * G]
            want = np.full((G, N), -1, np.int32)
            for i, e in enumerate(take):
                want[i % G, i // G] = e
            assert np.array_equal(res.replica_map[0, d * G:(d + 1) * G], want), (reserve, d)


@pytest.mark.parametrize("seed", range(3))
def test_reserving_every_slot_equals_refinement_only(seed):
    w, ids = _skewed_case(seed)
    kw = dict(main_rank=w.main_rank())
    a = orc.plan(orc.OracleConfig(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                                  w.token_bytes, w.expert_bytes, reserve_slots=w.slots_per_rank,
                                  **kw), ids)
    b = orc.plan(orc.OracleConfig(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                                  w.token_bytes, w.expert_bytes, stages=2, **kw), ids)
    for name in ("replica_map", "token_replica", "dispatch_counts", "instance_counts", "rank_load"):
        assert np.array_equal(getattr(a, name), getattr(b, name)), name
    assert a.refine_iters.sum() > 0


@pytest.mark.parametrize("reserve", [1, 2])
def test_reserved_slots_keep_every_constraint(reserve):
    w, ids = _skewed_case(7)
    cfg = orc.OracleConfig(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                           w.token_bytes, w.expert_bytes, main_rank=w.main_rank(),
                           reserve_slots=reserve)
    res = orc.plan(cfg, ids)
    check_plan(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k, w.main_rank(),
               w.token_bytes, w.expert_bytes, ids[0], res.replica_map[0], res.token_replica[0],
               res.dispatch_counts[0], res.dispatch_offsets[0], res.instance_counts[0],
               res.rank_load[0])


# ---- policy variant: stage-1 candidates to the least-loaded rank (LPT) ---------------------------
@pytest.mark.parametrize("seed", range(3))
def test_lpt_places_the_same_experts_on_the_least_loaded_ranks(seed):
    """With stage1_rank = 1 inter-node placement alone (stages = 1) must replicate exactly the
    experts the default policy replicates in each domain, but deal them greedily: the next
    candidate (benefit down, expert id up) to the rank with a free slot and the smallest estimated
    load -- main-instance demand plus the demand of replicas already there; ties to the lowest
    rank.  Re-derived here from the routing matrix with a sort and a loop."""
    w, ids = _skewed_case(seed, slots=2)
    M, G, E, N = w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank
    R = M * G
    mr = w.main_rank()
    kw = dict(main_rank=mr, stages=1)
    base = orc.plan(orc.OracleConfig(M, G, E, N, w.top_k, w.token_bytes, w.expert_bytes, **kw), ids)
    lpt = orc.plan(orc.OracleConfig(M, G, E, N, w.top_k, w.token_bytes, w.expert_bytes,
                                    stage1_rank=1, **kw), ids)
    omega = base.omega[0]
    D = omega.reshape(M, G, E).sum(axis=1)
    est = np.zeros(R, np.int64)
    for e in range(E):
        est[mr[e]] += D[:, e].sum()
    differs = False
    for d in range(M):
        b = 2 * D[d] * w.token_bytes - w.expert_bytes
        cands = sorted((e for e in range(E) if mr[e] // G != d and b[e] > 0), key=lambda e: (-b[e], e))
        want = np.full((G, N), -1, np.int32)
        used = np.zeros(G, int)
        for e in cands:
            free = [g for g in range(G) if used[g] < N]
            if not free:
                break
            g = min(free, key=lambda g: (est[d * G + g], g))
            want[g, used[g]] = e
            used[g] += 1
            est[d * G + g] += D[d, e]
        got = lpt.replica_map[0, d * G:(d + 1) * G]
        assert np.array_equal(got, want), d
        assert sorted(got[got >= 0].tolist()) == sorted(base.replica_map[0, d * G:(d + 1) * G][
            base.replica_map[0, d * G:(d + 1) * G] >= 0].tolist())
        differs |= not np.array_equal(got, base.replica_map[0, d * G:(d + 1) * G])
    assert differs          # the variant is not vacuous on this input


def test_lpt_keeps_every_constraint():
    w, ids = _skewed_case(5)
    cfg = orc.OracleConfig(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                           w.token_bytes, w.expert_bytes, main_rank=w.main_rank(), stage1_rank=1)
    res = orc.plan(cfg, ids)
    check_plan(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k, w.main_rank(),
               w.token_bytes, w.expert_bytes, ids[0], res.replica_map[0], res.token_replica[0],
               res.dispatch_counts[0], res.dispatch_offsets[0], res.instance_counts[0],
               res.rank_load[0])
