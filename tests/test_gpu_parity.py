"""CUDA library vs CPU oracle, element by element, through the C boundary (needs a B200)."""
import ctypes

import numpy as np
import pytest
import torch

import oracle as orc
import workloads as wl
from plan_checks import check_plan, dispatch_positions_by_sorting
from gpu_common import assert_same, make_planner, oracle_config, parity, run_gpu

pytestmark = pytest.mark.gpu

from paper_2609_35481_b200 import binding as B  # noqa: E402


# ---- the benchmark configurations at full size -----------------------------------------------
@pytest.mark.parametrize("name", ["tiny", "mid", "dsv3"])
@pytest.mark.parametrize("seed", [20260935, 1, 2])
def test_configs_1_to_3_full_size(name, seed):
    gpu, ref, _ = parity(wl.CONFIGS[name], seed)
    assert gpu["flags"] == 0


@pytest.mark.parametrize("name", ["scaleout", "scaleout_uniform"])
def test_config_5_full_size(name):
    w = wl.CONFIGS[name]
    gpu, ref, ids = parity(w, wl.BASE_SEED)
    assert gpu["flags"] == 0
    check_plan(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k, w.main_rank(),
               w.token_bytes, w.expert_bytes, ids[0], gpu["replica_map"][0], gpu["token_replica"][0],
               gpu["dispatch_counts"][0], gpu["dispatch_offsets"][0], gpu["instance_counts"][0],
               gpu["rank_load"][0])


def test_config_4_batched_full_size_every_plan():
    # 232 plans of the dsv3 shape in ONE call, as the bench launches it.  The oracle recomputes every
    # plan (they are independent; a quarter of the batch at a time keeps the host copies small);
    # structural properties are checked on two of them; omega of every plan is checked against
    # bincount.
    w = wl.CONFIGS["dsv3_batched"]
    ids = wl.make_topk_ids(w, seed=wl.BASE_SEED)
    pl = make_planner(w)
    gpu = run_gpu(pl, ids)
    assert gpu["flags"] == 0
    step = 58
    for b0 in range(0, w.batch, step):
        part = list(range(b0, min(b0 + step, w.batch)))
        ref = orc.plan(oracle_config(w), ids[part])
        assert ref.flags == 0
        assert_same(gpu, ref, plans=part)
    for b in (5, 200):
        check_plan(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k, w.main_rank(),
                   w.token_bytes, w.expert_bytes, ids[b], gpu["replica_map"][b],
                   gpu["token_replica"][b], gpu["dispatch_counts"][b], gpu["dispatch_offsets"][b],
                   gpu["instance_counts"][b], gpu["rank_load"][b])
    E = w.experts
    flat = ids.reshape(w.batch * w.ranks, -1).astype(np.int64)
    flat += (np.arange(flat.shape[0]) * E)[:, None]
    om = np.bincount(flat.ravel(), minlength=flat.shape[0] * E).reshape(w.batch, w.ranks, E)
    assert np.array_equal(om, gpu["omega"])


# ---- shapes where inter-node placement AND refinement both act ------------------------------
BOTH_STAGES = [
    ("dsv3", dict(slots_per_rank=3, tokens_per_rank=2048)),
    ("dsv3", dict(slots_per_rank=4, tokens_per_rank=2048)),
    ("dsv3", dict(slots_per_rank=8, tokens_per_rank=4096, zipf_s=0.8)),
    ("mid", dict(slots_per_rank=3)),
    ("scaleout", dict(slots_per_rank=4, tokens_per_rank=2048, zipf_s=1.0)),
    ("tiny", dict(slots_per_rank=3)),
]


@pytest.mark.parametrize("name,over", BOTH_STAGES)
def test_both_stages_active(name, over):
    w = wl.CONFIGS[name].replace(**over)
    gpu, ref, _ = parity(w, 77, batch=3)
    assert ref.refine_iters.sum() > 0
    if w.nodes > 1 and name != "tiny":
        assert ref.summaries["replicas_inter"].sum() > 0


# ---- degenerate and ragged shapes --------------------------------------------------------------
def test_single_domain():
    w = wl.CONFIGS["mid"].replace(nodes=1, gpus_per_node=8, experts=64, slots_per_rank=2,
                                  tokens_per_rank=1000)
    gpu, ref, _ = parity(w, 5, batch=2)
    assert ref.summaries["replicas_inter"].sum() == 0 and ref.refine_iters.sum() > 0


def test_one_gpu_per_node_and_no_slots():
    parity(wl.CONFIGS["tiny"].replace(nodes=8, gpus_per_node=1, tokens_per_rank=3000), 6)
    parity(wl.CONFIGS["tiny"].replace(slots_per_rank=0), 6)


@pytest.mark.parametrize("T,k", [(1, 1), (3, 1), (7, 3), (1023, 2), (1025, 2), (2049, 3), (4097, 1),
                                 (5000, 2), (777, 5)])
def test_ragged_token_counts(T, k):
    # T*k not a multiple of 4 (scalar loads), of the tile, or smaller than one warp
    w = wl.CONFIGS["tiny"].replace(tokens_per_rank=T, top_k=k, slots_per_rank=2)
    parity(w, 100 + T, batch=2)


def test_uneven_main_map_and_odd_topology():
    # 3 nodes x 3 GPUs, 20 experts placed by a seeded random map (some ranks get none)
    rng = np.random.default_rng(3)
    w = wl.CONFIGS["tiny"].replace(nodes=3, gpus_per_node=3, experts=20, slots_per_rank=2,
                                   top_k=3, tokens_per_rank=1500)
    main = rng.integers(0, 9, size=20).astype(np.int32)
    ids = wl.make_topk_ids(w, seed=9, batch=2)
    pl = make_planner(w, max_batch=2, main_rank=main)
    gpu = run_gpu(pl, ids)
    ref = orc.plan(oracle_config(w, main_rank=main), ids)
    assert_same(gpu, ref)


def test_many_domains_wide_nodes_and_many_candidates():
    # 40 single-GPU nodes (hosting masks beyond bit 31), a 32-GPU node (one refinement lane per
    # target), and a cheap expert (tiny ||W||) so that a domain has far more than 128 stage-1
    # candidates (slot-by-slot selection path) and many split experts per source (several passes
    # of the reroute ranking)
    w = wl.CONFIGS["tiny"].replace(nodes=40, gpus_per_node=1, experts=80, slots_per_rank=2, top_k=4,
                                   tokens_per_rank=700, zipf_s=0.9)
    parity(w, 21, batch=2, expert_bytes=4096)
    w = wl.CONFIGS["tiny"].replace(nodes=2, gpus_per_node=32, experts=128, slots_per_rank=2, top_k=4,
                                   tokens_per_rank=900, zipf_s=1.3)
    gpu, ref, _ = parity(w, 22, batch=2)
    assert ref.refine_iters.sum() > 0
    w = wl.CONFIGS["tiny"].replace(nodes=3, gpus_per_node=4, experts=600, slots_per_rank=24,
                                   top_k=8, tokens_per_rank=4096, zipf_s=0.3)
    gpu, ref, _ = parity(w, 23, batch=1, expert_bytes=64, token_bytes=64)
    assert ref.summaries["replicas_inter"][0] > 128


@pytest.mark.parametrize("nodes,gpus,experts,slots", [(32, 8, 768, 1), (16, 8, 1024, 2), (32, 8, 512, 2)])
def test_largest_shapes_the_library_accepts(nodes, gpus, experts, slots):
    """Shapes at the edge of what fits one SM's shared memory (the next larger ones are refused
    with TOPOEP_ERR_SMEM): 256 ranks, up to 1024 experts."""
    w = wl.CONFIGS["scaleout"].replace(nodes=nodes, gpus_per_node=gpus, experts=experts,
                                       slots_per_rank=slots, top_k=4, tokens_per_rank=1536)
    gpu, ref, _ = parity(w, 71)
    assert ref.summaries["replicas_inter"].sum() > 0
    cost = B.CostParams(w.token_bytes, w.expert_bytes, 1, 8, 0, 0, 0)
    rc, _ = B.topoep_create(nodes, gpus, 4 * experts, slots, 4, 64, 1, None, cost)
    assert rc == -9


def test_random_small_problems():
    rng = np.random.default_rng(11)
    for trial in range(40):
        M, G = int(rng.integers(1, 5)), int(rng.integers(1, 6))
        R = M * G
        E = int(rng.integers(1, 40))
        N = int(rng.integers(0, 4))
        k = int(rng.integers(1, min(E, 4) + 1))
        T = int(rng.integers(1, 400))
        main = rng.integers(0, R, size=E).astype(np.int32)
        tok, W = int(rng.integers(1, 64)), int(rng.integers(0, 4000))
        ids = rng.integers(0, E, size=(2, R, T, k)).astype(np.int32)   # duplicates inside a token
        w = wl.Workload("rnd", M, G, E, N, k, T)
        over = dict(main_rank=main, token_bytes=tok, expert_bytes=W,
                    c_intra=int(rng.integers(0, 3)), c_inter=int(rng.integers(0, 9)))
        pl = make_planner(w, max_batch=2, **over)
        gpu = run_gpu(pl, ids)
        ref = orc.plan(oracle_config(w, **over), ids)
        assert_same(gpu, ref)
        pl.close()


def test_random_problems_with_policies_tunings_and_skew():
    """Random topologies, UNEVEN random main maps, skewed and partly padded ids, random policy
    variants, tile sizes and launch protocols (a wider net of the same kind found a wrong load
    estimate for ranks with fewer main experts than E_loc under the least-loaded-rank policy)."""
    rng = np.random.default_rng(12)
    for trial in range(60):
        M, G = int(rng.integers(1, 7)), int(rng.integers(1, 9))
        R = M * G
        E = int(rng.integers(1, 120))
        N = int(rng.integers(0, 6))
        k = int(rng.integers(1, min(E, 6) + 1))
        T = int(rng.integers(1, 3000))
        Bn = int(rng.integers(1, 4))
        main = rng.integers(0, R, size=E).astype(np.int32)
        tok, W = int(rng.integers(1, 64)), int(rng.integers(0, 4000))
        skew = float(rng.uniform(0.5, 3.0))
        ids = np.minimum((rng.random((Bn, R, T, k)) ** skew * E).astype(np.int32), E - 1)
        if rng.random() < 0.2:
            ids[rng.random(ids.shape) < 0.05] = -1
        w = wl.Workload("rnd", M, G, E, N, k, T)
        reserve, lpt = int(rng.integers(0, N + 1)), int(rng.integers(0, 2))
        over = dict(main_rank=main, token_bytes=tok, expert_bytes=W,
                    c_intra=int(rng.integers(0, 3)), c_inter=int(rng.integers(0, 9)))
        pl = make_planner(w, max_batch=Bn, **over)
        pl.set_policy(B.POLICY_RESERVE_SLOTS, reserve)
        pl.set_policy(B.POLICY_STAGE1_RANK, lpt)
        pl.set_tuning(B.KNOB_TILE_IDS, int(rng.choice([1024, 2048, 4096, 8192])))
        pl.set_tuning(B.KNOB_PDL, int(rng.integers(0, 4)))
        pl.set_tuning(B.KNOB_CHAIN, int(rng.integers(0, 4)))
        pl.set_tuning(B.KNOB_PACKED_IDS, int(rng.integers(0, 3)))
        pl.set_tuning(B.KNOB_REROUTE_TILES, int(rng.integers(1, 6)))
        gpu = run_gpu(pl, ids)
        ref = orc.plan(oracle_config(w, reserve_slots=reserve, stage1_rank=lpt, **over), ids)
        try:
            assert_same(gpu, ref)
        except AssertionError as err:
            raise AssertionError("trial %d %s: %s" % (trial, (M, G, E, N, k, T, Bn, reserve, lpt), err))
        assert gpu["flags"] == ref.flags
        pl.close()


def test_random_many_domain_problems_through_the_combined_kernel():
    """Many domains and experts (M * E >= 4096): there the solver blocks of the combined kernel read
    the published inter-node placement instead of ranking every domain's demand again.  Random
    shapes, main maps, padding and slot reservations through the two- and four-kernel chains."""
    rng = np.random.default_rng(33)
    done = 0
    while done < 40:
        M, G = int(rng.integers(4, 33)), int(rng.integers(1, 9))
        R = M * G
        E = int(rng.integers(max(1, 4096 // M), 1200))
        N = int(rng.integers(0, 4))
        k = int(rng.integers(1, 9))
        T = int(rng.integers(1, 1500))
        Bn = int(rng.integers(1, 3))
        main = rng.integers(0, R, size=E).astype(np.int32)
        tok, W = int(rng.integers(1, 64)), int(rng.integers(0, 2000))
        skew = float(rng.uniform(0.5, 3.0))
        ids = np.minimum((rng.random((Bn, R, T, k)) ** skew * E).astype(np.int32), E - 1)
        if rng.random() < 0.3:
            ids[rng.random(ids.shape) < 0.02] = -1
        w = wl.Workload("rnd", M, G, E, N, k, T)
        reserve = int(rng.integers(0, N + 1))
        over = dict(main_rank=main, token_bytes=tok, expert_bytes=W,
                    c_intra=int(rng.integers(0, 3)), c_inter=int(rng.integers(0, 9)))
        try:
            pl = make_planner(w, max_batch=Bn, **over)
        except Exception:
            continue   # a shape the library refuses (tables beyond shared memory)
        pl.set_policy(B.POLICY_RESERVE_SLOTS, reserve)
        chain = int(rng.choice([0, 2, 3]))
        pl.set_tuning(B.KNOB_CHAIN, chain)
        ref = orc.plan(oracle_config(w, reserve_slots=reserve, **over), ids)
        for rep in range(2):
            gpu = run_gpu(pl, ids)
            try:
                assert_same(gpu, ref)
            except AssertionError as err:
                raise AssertionError("%s: %s" % ((M, G, E, N, k, T, Bn, chain, reserve), err))
            assert gpu["flags"] == ref.flags
        pl.close()
        done += 1


def test_invalid_and_padded_ids():
    w = wl.CONFIGS["tiny"].replace(slots_per_rank=2)
    ids = wl.make_topk_ids(w, seed=4, batch=2).copy()
    ids[0, 1, 100:300, :] = -1                      # padded rows: ignored, no flag
    gpu, ref, _ = parity(w, 4, ids=ids)
    assert gpu["flags"] == 0 and (gpu["token_replica"][0, 1, 100:300] == -1).all()
    ids[1, 2, 7, 0] = w.experts                     # out of range: ignored and flagged
    ids[1, 3, 9, 1] = -5
    gpu, ref, _ = parity(w, 4, ids=ids)
    assert gpu["flags"] == B.FLAG_BAD_ID == ref.flags
    assert gpu["token_replica"][1, 2, 7, 0] == -1 and gpu["token_replica"][1, 3, 9, 1] == -1


def test_refinement_cap_binds_identically():
    w = wl.CONFIGS["scaleout_uniform"].replace(tokens_per_rank=1024)
    gpu, ref, _ = parity(w, 8, max_refine_iters=3)
    assert gpu["flags"] == B.FLAG_REFINE_CAP and (gpu["refine_iters"] <= 3).all()
    gpu2, ref2, _ = parity(w, 8, min_delta=5)
    assert gpu2["flags"] == 0


def test_empty_batch_and_zero_tokens():
    w = wl.CONFIGS["tiny"]
    pl = make_planner(w, max_batch=2)
    out = pl.alloc_outputs(1, 0)
    ids = torch.empty((1, w.ranks, 0, w.top_k), dtype=torch.int32, device=pl.device)
    pl.plan(ids, out)
    torch.cuda.synchronize()
    assert (out.dispatch_counts == 0).all() and (out.replica_map == -1).all()
    assert (out.dispatch_offsets == 0).all() and (out.instance_counts == 0).all()
    rc = B.topoep_plan(pl.handle, None, 5, 0, None, None, None, None, None, 0)
    assert rc == B.OK                      # batch 0: nothing to do
    assert pl.status() == 0


# ---- the two kernel chains of topoep_plan ---------------------------------------------------
CHAIN_CASES = [
    ("tiny", dict(), 2),                                    # refinement acts: solver blocks + flags
    ("tiny", dict(slots_per_rank=3), 3),
    ("mid", dict(), 1),                                     # closed form: every slot taken
    ("mid", dict(slots_per_rank=3), 2),
    ("dsv3", dict(), 1),
    ("dsv3", dict(slots_per_rank=3, tokens_per_rank=2048), 2),
    ("dsv3", dict(tokens_per_rank=1027, top_k=3), 1),       # ragged tiles, scalar loads
    ("mid", dict(nodes=1, gpus_per_node=8, experts=64, slots_per_rank=2, tokens_per_rank=1000), 2),
    ("tiny", dict(slots_per_rank=0), 1),                    # no slots: closed form, no replicas
    ("tiny", dict(nodes=8, gpus_per_node=1, tokens_per_rank=3000), 1),
    ("tiny", dict(nodes=40, gpus_per_node=1, experts=80, slots_per_rank=2, top_k=4,
                  tokens_per_rank=700, zipf_s=0.9, ffn=2), 2),   # hosting masks beyond bit 31
    ("tiny", dict(nodes=3, gpus_per_node=4, experts=600, slots_per_rank=24, top_k=8,
                  tokens_per_rank=4096, zipf_s=0.3, ffn=1, hidden=32), 1),   # > 128 candidates
    ("scaleout", dict(tokens_per_rank=1024), 1),            # 128 ranks, 512 experts, 2 slots
]


@pytest.mark.parametrize("name,over,batch", CHAIN_CASES)
def test_kernel_chains_agree_with_one_another_and_the_oracle(name, over, batch):
    """topoep_plan has three kernel chains (TOPOEP_KNOB_CHAIN): five kernels; for small calls an
    accumulating histogram followed by one grid of placement, solver, rank and per-token blocks;
    for a single mid-size plan histogram, omega, the same grid with route blocks in place of the
    per-token blocks, and the reroute kernel.  All must give the oracle's plan bit for bit, call
    after call on one handle (the accumulators of the second chain alternate between two pairs and
    clean up after themselves; records and flags are told apart by the call's serial number), also
    when the chains alternate and when the batch size changes between calls."""
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=91, batch=batch)
    ref = orc.plan(oracle_config(w), ids)
    pl = make_planner(w, max_batch=batch)
    for chain in (2, 2, 1, 3, 2, 0, 3, 3, 2):
        pl.set_tuning(B.KNOB_CHAIN, chain)
        gpu = run_gpu(pl, ids)
        assert_same(gpu, ref)
        assert gpu["flags"] == ref.flags
    if batch > 1:   # a smaller batch in between leaves sums of the larger one behind: cleared?
        pl.set_tuning(B.KNOB_CHAIN, 2)
        one = orc.plan(oracle_config(w), ids[:1])
        for part, want in ((ids[:1], one), (ids, ref), (ids[:1], one), (ids[:1], one), (ids, ref)):
            assert_same(run_gpu(pl, part), want)
    # a stage call continues from stage calls, not from a plan of the two-kernel chain
    pl.set_tuning(B.KNOB_CHAIN, 2)
    dev = torch.from_numpy(ids).to(pl.device)
    out = pl.plan(dev)
    assert B.topoep_reroute(pl.handle, dev, w.tokens_per_rank, batch, out.token_replica, 0) == -6
    # but the solver stage may start from the routing matrix the plan left behind
    again = pl.solve(None, batch, tokens_per_rank=w.tokens_per_rank)
    torch.cuda.synchronize()
    assert np.array_equal(again.replica_map.cpu().numpy(), ref.replica_map)
    assert np.array_equal(again.dispatch_offsets.cpu().numpy()[:, 1], ref.dispatch_offsets[:, 1])
    assert pl.status() == 0


# ---- the one-byte copy of the ids (five-kernel chain, E <= 256) ---------------------------------
PACKED_CASES = [
    ("tiny", {}, 3, "clean"),
    ("mid", dict(slots_per_rank=3), 2, "padded"),
    ("dsv3", dict(tokens_per_rank=3000, slots_per_rank=2), 2, "invalid"),
    ("tiny", dict(tokens_per_rank=778, top_k=6, slots_per_rank=2), 2, "padded"),
    ("tiny", dict(experts=30, tokens_per_rank=2048, slots_per_rank=2), 2, "padded"),   # E % 4 != 0
    ("tiny", dict(tokens_per_rank=777, top_k=5), 2, "clean"),   # rows of 3885 ids: not whole groups of four
    ("dsv3", dict(experts=224, tokens_per_rank=1536), 2, "padded"),
    ("mid", dict(experts=512, nodes=2, tokens_per_rank=1024), 2, "clean"),   # E > 256: no copy exists
]


@pytest.mark.parametrize("name,over,batch,dirt", PACKED_CASES)
def test_one_byte_id_copy_matches_the_oracle(name, over, batch, dirt):
    """With at most 256 experts the histogram of a large topoep_plan call leaves a one-byte copy of
    the ids for the reroute kernel (TOPOEP_KNOB_PACKED_IDS; here forced on for small calls).  A
    tile with padding (-1) or an invalid id cannot be expressed in bytes and is read again in
    full; rows that are not whole groups of four ids and configs with more experts fall back to
    the plain kernels.  Every variant must give the oracle's plan, bit for bit."""
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=7, batch=batch).copy()
    if dirt in ("padded", "invalid"):
        ids[0, 1, -37:, :] = -1                                          # tail tokens of one rank
        ids[batch - 1, w.ranks - 1, w.tokens_per_rank // 2:, :] = -1     # half a rank
    if dirt == "invalid":
        ids[0, 2, 5, 0] = w.experts
        ids[1, 0, 100, 1] = 1 << 20
        ids[1, 3, 7, 2] = -7
    ref = orc.plan(oracle_config(w), ids)
    for tile, tiles_per_block in ((1024, 1), (1024, 3), (4096, 4), (8192, 2)):
        pl = make_planner(w, max_batch=batch)
        pl.set_tuning(B.KNOB_CHAIN, 1)
        pl.set_tuning(B.KNOB_PACKED_IDS, 2)
        pl.set_tuning(B.KNOB_TILE_IDS, tile)
        pl.set_tuning(B.KNOB_REROUTE_TILES, tiles_per_block)
        for rep in range(2):   # the second call finds the first one's copy and flags in the workspace
            gpu = run_gpu(pl, ids)
            assert_same(gpu, ref)
            assert gpu["flags"] == ref.flags
        pl.close()


# ---- determinism: reruns and launch configurations ----------------------------------------
def test_bitwise_identical_across_reruns_and_tunings():
    w = wl.CONFIGS["dsv3"].replace(slots_per_rank=3)
    ids = wl.make_topk_ids(w, seed=31, batch=2)
    pl = make_planner(w, max_batch=2)
    base = run_gpu(pl, ids)
    for tile in (1024, 2048, 4096, 8192):
        for mode in (0, 1):
            pl.set_tuning(B.KNOB_TILE_IDS, tile)
            pl.set_tuning(B.KNOB_HIST_MODE, mode)
            # launch protocol: plain order, automatic, never early, always early
            pl.set_tuning(B.KNOB_PDL, (tile // 1024 + mode) % 4)
            # kernel chain: by size, five kernels, two kernels, four kernels
            pl.set_tuning(B.KNOB_CHAIN, (tile // 1024 + mode) % 4)
            # one-byte id copy for the reroute kernel: by size, never, whenever possible; and the
            # tiles a block of that kernel walks
            pl.set_tuning(B.KNOB_PACKED_IDS, (tile // 2048 + mode) % 3)
            pl.set_tuning(B.KNOB_REROUTE_TILES, 1 + (tile // 1024 + 3 * mode) % 5)
            for rep in range(2):
                again = run_gpu(pl, ids)
                for key, val in base.items():
                    if key == "flags":
                        assert again[key] == val
                    elif key == "summaries":
                        assert again[key].tobytes() == val.tobytes()
                    else:
                        assert np.array_equal(again[key], val), (key, tile, mode)
    ref = orc.plan(oracle_config(w), ids)
    assert_same(base, ref)


def test_histogram_entry_point_matches_bincount():
    w = wl.CONFIGS["mid"]
    ids = wl.make_topk_ids(w, seed=12, batch=2)
    pl = make_planner(w, max_batch=2)
    om = pl.histogram(torch.from_numpy(ids).to(pl.device)).cpu().numpy()
    for b in range(2):
        for s in range(w.ranks):
            assert np.array_equal(om[b, s], np.bincount(ids[b, s].ravel(), minlength=w.experts))


@pytest.mark.parametrize("packed", [1, 2])
def test_stage_entry_points_equal_the_fused_plan(packed):
    """packed = 2: the histogram call leaves the one-byte copy of the ids and the reroute call, given
    the same buffer, reads it; given another buffer with the same ids it reads that one."""
    w = wl.CONFIGS["mid"].replace(slots_per_rank=3)
    ids = wl.make_topk_ids(w, seed=13, batch=2).copy()
    ids[1, 5, -100:, :] = -1
    pl = make_planner(w, max_batch=2)
    pl.set_tuning(B.KNOB_CHAIN, 1)
    pl.set_tuning(B.KNOB_PACKED_IDS, packed)
    dev = torch.from_numpy(ids).to(pl.device)
    fused = pl.plan(dev)
    out = pl.alloc_outputs(2, w.tokens_per_rank)
    for t in (out.replica_map, out.token_replica, out.dispatch_counts, out.dispatch_offsets,
              out.instance_counts):
        t.fill_(-9)
    omega = torch.empty((2, w.ranks, w.experts), dtype=torch.int32, device=pl.device)
    T = w.tokens_per_rank
    assert B.topoep_histogram(pl.handle, dev, T, 2, omega, 0) == 0
    # the solver accepts the routing matrix from anywhere (e.g. rows gathered from other ranks)
    assert B.topoep_solve(pl.handle, omega.clone(), 2, out.replica_map, out.dispatch_counts,
                          out.dispatch_offsets, out.instance_counts, 0) == 0
    assert B.topoep_reroute(pl.handle, dev, T - 1, 2, out.token_replica, 0) == -6
    assert B.topoep_reroute(pl.handle, dev, T, 2, out.token_replica, 0) == 0
    torch.cuda.synchronize()
    for name in ("replica_map", "token_replica", "dispatch_counts", "dispatch_offsets",
                 "instance_counts"):
        assert torch.equal(getattr(out, name), getattr(fused, name)), name
    out.token_replica.fill_(-9)
    assert B.topoep_reroute(pl.handle, dev.clone(), T, 2, out.token_replica, 0) == 0
    torch.cuda.synchronize()
    assert torch.equal(out.token_replica, fused.token_replica)
    assert pl.status() == 0


# ---- policy variant: slots reserved for the refinement ------------------------------------------
@pytest.mark.parametrize("name,over,reserve", [
    ("dsv3", dict(slots_per_rank=2, tokens_per_rank=2048), 1),
    ("dsv3", dict(slots_per_rank=4, tokens_per_rank=2048), 3),
    ("mid", dict(slots_per_rank=1), 1),                    # everything reserved: refinement only
    ("scaleout", dict(slots_per_rank=3, tokens_per_rank=2048, zipf_s=1.0), 2),
    ("tiny", dict(slots_per_rank=3, ffn=16), 1),           # many candidates, capacity binds
])
def test_reserved_slots_policy_matches_the_oracle(name, over, reserve):
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=41, batch=2)
    pl = make_planner(w, max_batch=2)
    pl.set_policy(B.POLICY_RESERVE_SLOTS, reserve)
    gpu = run_gpu(pl, ids)
    ref = orc.plan(oracle_config(w, reserve_slots=reserve), ids)
    assert_same(gpu, ref)
    assert ref.refine_iters.sum() > 0
    assert B.topoep_set_policy(pl.handle, B.POLICY_RESERVE_SLOTS, w.slots_per_rank + 1) == -10
    # back to the default: the paper's procedure again
    pl.set_policy(B.POLICY_RESERVE_SLOTS, 0)
    assert_same(run_gpu(pl, ids), orc.plan(oracle_config(w), ids))


@pytest.mark.parametrize("name,over,reserve", [
    ("dsv3", dict(slots_per_rank=2, tokens_per_rank=2048), 0),
    ("mid", dict(slots_per_rank=3), 1),
    ("scaleout", dict(slots_per_rank=3, tokens_per_rank=2048, zipf_s=1.0), 0),
    ("tiny", dict(slots_per_rank=3, ffn=16), 0),
    ("tiny", dict(slots_per_rank=5, ffn=1, experts=512, tokens_per_rank=4096, top_k=4), 0),  # > 128 candidates
])
def test_least_loaded_rank_policy_matches_the_oracle(name, over, reserve):
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=43, batch=2)
    pl = make_planner(w, max_batch=2)
    pl.set_policy(B.POLICY_STAGE1_RANK, 1)
    pl.set_policy(B.POLICY_RESERVE_SLOTS, reserve)
    ref = orc.plan(oracle_config(w, stage1_rank=1, reserve_slots=reserve), ids)
    assert_same(run_gpu(pl, ids), ref)
    assert ref.summaries["replicas_inter"].sum() > 0
    pl.set_policy(B.POLICY_STAGE1_RANK, 0)
    pl.set_policy(B.POLICY_RESERVE_SLOTS, 0)
    assert_same(run_gpu(pl, ids), orc.plan(oracle_config(w), ids))


# ---- sharded deployment: every rank plans from the gathered routing matrix -----------------------
@pytest.mark.parametrize("name,over,batch,window", [
    ("mid", dict(slots_per_rank=3), 2, 1),
    ("mid", dict(slots_per_rank=2, tokens_per_rank=777), 1, 3),   # ragged last window and tile
    ("dsv3", dict(tokens_per_rank=4099), 1, 8),                    # one process per node
    ("scaleout", dict(tokens_per_rank=1500), 1, 16),
])
def test_sharded_ranks_reach_the_same_plan_as_the_oracle(name, over, batch, window):
    """Each emulated process owns a window of source ranks: it histograms its own ids, the rows
    are gathered, every process solves the whole group from the gathered matrix and reroutes its
    own ids.  The processes run one after the other on this GPU, each with its own handle and
    workspace.  Every process must hold the same plan, bit for bit, and the union of their
    per-token outputs must equal the oracle's single-process result."""
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=21, batch=batch)
    ref = orc.plan(oracle_config(w), ids)
    R, T = w.ranks, w.tokens_per_rank
    windows = [(f, min(window, R - f)) for f in range(0, R, window)]
    procs = []
    for first, count in windows:
        pl = make_planner(w, max_batch=batch)
        pl.set_rank_window(first, count)
        procs.append((pl, torch.from_numpy(np.ascontiguousarray(ids[:, first:first + count])).to(pl.device)))
    rows = [pl.histogram(mine) for pl, mine in procs]
    for (first, count), r in zip(windows, rows):
        assert np.array_equal(r.cpu().numpy(), ref.omega[:, first:first + count])
    gathered = torch.cat(rows, dim=1).contiguous()          # the EP-group all-gather
    outs = [pl.solve(gathered, batch, tokens_per_rank=T) for pl, _ in procs]
    parts = [pl.reroute(mine) for pl, mine in procs]
    torch.cuda.synchronize()
    for (pl, _), out in zip(procs, outs):
        for field in ("replica_map", "dispatch_counts", "dispatch_offsets", "instance_counts"):
            assert np.array_equal(getattr(out, field).cpu().numpy(), getattr(ref, field)), field
        assert pl.status() == 0
        assert np.array_equal(pl.debug_tensor(B.T_Q, batch).numpy(), ref.q_instances)
    assert np.array_equal(torch.cat(parts, dim=1).cpu().numpy(), ref.token_replica)


def test_plan_sharded_over_a_one_process_nccl_group():
    """The NCCL form of the same step, in a group of one process (one GPU here): the all-gather,
    the row permutation and the window bookkeeping run as they would in a larger group."""
    import socket
    import torch.distributed as dist
    w = wl.CONFIGS["mid"].replace(slots_per_rank=2)
    ids = wl.make_topk_ids(w, seed=22, batch=2)
    ref = orc.plan(oracle_config(w), ids)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                            device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        pl = make_planner(w, max_batch=2)
        out = pl.plan_sharded(torch.from_numpy(ids).to(pl.device))
        torch.cuda.synchronize()
        for field in ("replica_map", "token_replica", "dispatch_counts", "dispatch_offsets",
                      "instance_counts"):
            assert np.array_equal(getattr(out, field).cpu().numpy(), getattr(ref, field)), field
        assert pl.status() == 0
    finally:
        dist.destroy_process_group()


def test_rank_window_argument_errors():
    w = wl.CONFIGS["tiny"]
    pl = make_planner(w)
    ids = torch.from_numpy(wl.make_topk_ids(w, seed=3)).to(pl.device)
    for first, count in ((-1, 1), (0, 0), (w.ranks, 1), (1, w.ranks)):
        assert B.topoep_set_rank_window(pl.handle, first, count) == -10
    pl.set_rank_window(1, 2)
    out = pl.alloc_outputs(1, w.tokens_per_rank)
    # a whole plan, the solver without a gathered matrix, and the dispatch permutation need all ranks
    assert B.topoep_plan(pl.handle, ids, w.tokens_per_rank, 1, out.replica_map, out.token_replica,
                         out.dispatch_counts, out.dispatch_offsets, out.instance_counts, 0) == -10
    assert B.topoep_solve(pl.handle, None, 1, out.replica_map, out.dispatch_counts,
                          out.dispatch_offsets, out.instance_counts, 0) == -1
    pl.set_rank_window(0, w.ranks)
    run = pl.plan(ids)
    assert pl.status() == 0 and run.token_replica.shape[1] == w.ranks


# ---- dispatch permutation (the step after the path) --------------------------------------------
@pytest.mark.parametrize("name,over,batch", [
    ("tiny", dict(slots_per_rank=2), 2),
    ("mid", dict(tokens_per_rank=777, slots_per_rank=3, top_k=5), 2),
    ("dsv3", dict(tokens_per_rank=1024), 1),
])
def test_dispatch_positions_match_the_oracle(name, over, batch):
    w = wl.CONFIGS[name].replace(**over)
    ids = wl.make_topk_ids(w, seed=41, batch=batch).copy()
    ids[0, 1, 3:20, :] = -1
    pl = make_planner(w, max_batch=batch)
    out = pl.plan(torch.from_numpy(ids).to(pl.device))
    send, recv, off = pl.dispatch_positions(out.token_replica)
    cfg = oracle_config(w)
    ref = orc.plan(cfg, ids)
    assert np.array_equal(out.token_replica.cpu().numpy(), ref.token_replica)
    for b in range(batch):
        s_ref, r_ref, o_ref = orc.dispatch_positions(cfg, ref.token_replica[b])
        assert np.array_equal(send[b].cpu().numpy(), s_ref)
        assert np.array_equal(recv[b].cpu().numpy(), r_ref)
        assert np.array_equal(off[b].cpu().numpy(), o_ref)
    assert pl.status() == 0


@pytest.mark.parametrize("name", ["dsv3", "scaleout"])
def test_dispatch_positions_full_size_are_the_sorted_order(name):
    # at full size the permutation is checked against its definition: a stable sort
    w = wl.CONFIGS[name]
    ids = wl.make_topk_ids(w, seed=43)
    pl = make_planner(w)
    out = pl.plan(torch.from_numpy(ids).to(pl.device))
    send, recv, off = pl.dispatch_positions(out.token_replica)
    tr = out.token_replica[0].cpu().numpy()
    s2, r2, o2 = dispatch_positions_by_sorting(w.ranks, pl.s_phys, tr)
    assert np.array_equal(send[0].cpu().numpy().reshape(w.ranks, -1), s2)
    assert np.array_equal(recv[0].cpu().numpy().reshape(w.ranks, -1), r2)
    assert np.array_equal(off[0].cpu().numpy(), o2)
    # a destination's block in a source's send buffer starts at the plan's send offset
    send_off = out.dispatch_offsets[0, 0].cpu().numpy()
    trf = tr.reshape(w.ranks, -1)
    for s in (0, w.ranks - 1):
        for r in (0, w.ranks // 2, w.ranks - 1):
            sel = (trf[s] // pl.s_phys == r) & (trf[s] >= 0)
            if sel.any():
                assert s2[s][sel].min() == send_off[s, r]


# ---- capture: the plan is enqueue-only ---------------------------------------------------------
def test_plan_is_capturable_in_a_cuda_graph_and_replays_identically():
    w = wl.CONFIGS["dsv3"]
    ids = wl.make_topk_ids(w, seed=21)
    pl = make_planner(w)
    dev_ids = torch.from_numpy(ids).to(pl.device)
    out = pl.alloc_outputs(1, w.tokens_per_rank)
    eager = pl.plan(dev_ids)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        # a host synchronisation, a device-to-host copy or an allocation inside would fail capture
        with torch.cuda.graph(graph, stream=stream):
            pl.plan(dev_ids, out, stream=stream)
    for _ in range(3):
        out.token_replica.fill_(-7)
        graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out.token_replica, eager.token_replica)
    assert torch.equal(out.replica_map, eager.replica_map)
    assert torch.equal(out.dispatch_offsets, eager.dispatch_offsets)
    ref = orc.plan(oracle_config(w), ids)
    assert np.array_equal(out.token_replica.cpu().numpy(), ref.token_replica)


def test_plan_dispatch_and_replica_copies_in_one_captured_graph():
    """What a training step would enqueue per layer -- plan, the two chunks' dispatch layouts, the
    parameter pull and the gradient return -- captured once (after a warm-up call of each entry
    point) and replayed: nothing in it may allocate, copy to the host or synchronise."""
    w = wl.CONFIGS["mid"].replace(slots_per_rank=2)
    cfg = oracle_config(w)
    ids = wl.make_topk_ids(w, seed=23)
    pl = make_planner(w)
    dev = pl.device
    R, T, k, N, S, Wb = w.ranks, w.tokens_per_rank, w.top_k, 2, pl.s_phys, 4096
    dev_ids = torch.from_numpy(ids).to(dev)
    out = pl.alloc_outputs(1, T)
    i32 = dict(dtype=torch.int32, device=dev)
    half = T // 2
    chunks = []
    for first, count in ((0, half), (half, T - half)):
        nb = B.topoep_dispatch_scratch_bytes(pl.handle, count, 1)
        chunks.append(dict(first=first, count=count, nb=nb,
                           scratch=torch.empty(nb + 256, dtype=torch.uint8, device=dev),
                           send=torch.empty((1, R, count, k), **i32), recv=torch.empty((1, R, count, k), **i32),
                           ioff=torch.empty((1, R, S + 1), **i32), counts=torch.empty((1, R, R), **i32),
                           offs=torch.empty((1, 2, R, R + 1), **i32)))
    main = torch.from_numpy(wl.make_param_bytes((R, pl.e_loc, Wb), 5)).to(dev)
    slots = torch.zeros((R, N, Wb), dtype=torch.uint8, device=dev)
    acc = torch.zeros((R, R, pl.e_loc, Wb), dtype=torch.uint8, device=dev)

    def step(st):
        pl.plan(dev_ids, out, stream=st)
        for c in chunks:
            ptr = (c["scratch"].data_ptr() + 255) // 256 * 256
            assert B.topoep_dispatch_window(pl.handle, out.token_replica, T, 1, c["first"], c["count"],
                                            c["send"], c["recv"], c["ioff"], c["counts"], c["offs"],
                                            ptr, c["nb"], st.cuda_stream) == 0
        assert B.topoep_replica_pull(pl.handle, out.replica_map[0], main, slots, Wb, st.cuda_stream) == 0
        assert B.topoep_replica_grad_return(pl.handle, out.replica_map[0], slots, acc, Wb,
                                            st.cuda_stream) == 0

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        step(stream)                                   # first calls set kernel attributes
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step(stream)
    slots.zero_()
    acc.zero_()
    for c in chunks:
        c["send"].fill_(-9)
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    ref = orc.plan(cfg, ids)
    assert np.array_equal(out.token_replica.cpu().numpy(), ref.token_replica)
    for c in chunks:
        part = np.ascontiguousarray(ref.token_replica[0][:, c["first"]:c["first"] + c["count"]])
        want_send, want_recv, want_ioff = orc.dispatch_positions(cfg, part)
        assert np.array_equal(c["send"][0].cpu().numpy(), want_send)
        assert np.array_equal(c["recv"][0].cpu().numpy(), want_recv)
        assert np.array_equal(c["ioff"][0].cpu().numpy(), want_ioff)
    want_slots = orc.replica_pull(cfg, ref.replica_map[0], main.cpu().numpy(), np.zeros((R, N, Wb), np.uint8))
    assert np.array_equal(slots.cpu().numpy(), want_slots)
    want_acc = orc.replica_grad_return(cfg, ref.replica_map[0], want_slots,
                                       np.zeros((R, R, pl.e_loc, Wb), np.uint8))
    assert np.array_equal(acc.cpu().numpy(), want_acc)
    assert pl.status() == 0


# ---- boundary errors that need a live workspace ---------------------------------------------
def test_size_and_pointer_errors():
    w = wl.CONFIGS["tiny"]
    pl = make_planner(w, max_batch=1)
    out = pl.alloc_outputs(1, w.tokens_per_rank)
    ids = torch.zeros((1, w.ranks, w.tokens_per_rank, w.top_k), dtype=torch.int32, device=pl.device)
    args = (out.replica_map, out.token_replica, out.dispatch_counts, out.dispatch_offsets,
            out.instance_counts, 0)
    assert B.topoep_plan(pl.handle, ids, w.tokens_per_rank + 1, 1, *args) == -6
    assert B.topoep_plan(pl.handle, ids, w.tokens_per_rank, 2, *args) == -6
    assert B.topoep_plan(pl.handle, None, w.tokens_per_rank, 1, *args) == -1
    assert B.topoep_plan(pl.handle, ids, w.tokens_per_rank, 1, None, *args[1:]) == -1
    assert B.topoep_plan(pl.handle, ids.data_ptr() + 2, w.tokens_per_rank, 1, *args) == -7
    assert B.topoep_set_workspace(pl.handle, pl._ws_ptr + 4, 1 << 30) == -5
    assert B.topoep_set_workspace(pl.handle, pl._ws_ptr, 16) == -5
    assert B.topoep_set_tuning(pl.handle, B.KNOB_TILE_IDS, 3000) == -10
    # a rejected set_workspace leaves the previous workspace in place
    assert B.topoep_plan(pl.handle, ids, w.tokens_per_rank, 1, *args) == 0
    torch.cuda.synchronize()


def test_imbalance_against_slot_count_on_the_slot_experiment_shape():
    """The shape of the paper's slot-count experiment (32 ranks, 640 experts, top-8; its routing
    trace is not public, so Zipf-skewed synthetic routing stands in): the max/mean rank load of the
    CUDA plan equals the oracle's for every slot count and policy, replicas never make it worse
    than no replicas, and holding one slot back for the refinement helps when slots are scarce."""
    base = wl.CONFIGS["dsv3"].replace(experts=640, tokens_per_rank=2048, zipf_s=1.2, bursts=0)
    ids = wl.make_topk_ids(base, seed=51)
    table = {}
    for slots in (0, 1, 2, 4):
        for reserve in (0, 1):
            if reserve > slots:
                continue
            w = base.replace(slots_per_rank=slots)
            pl = make_planner(w)
            pl.set_policy(B.POLICY_RESERVE_SLOTS, reserve)
            gpu = run_gpu(pl, ids)
            ref = orc.plan(oracle_config(w, reserve_slots=reserve), ids)
            assert_same(gpu, ref)
            table[(slots, reserve)] = float(gpu["summaries"]["imbalance"][0])
    print("imbalance (slots, reserve):", {k: round(v, 3) for k, v in table.items()})
    none = table[(0, 0)]
    assert all(v <= none + 1e-9 for v in table.values())
    assert table[(1, 1)] < table[(1, 0)]


# ---- two-chunk pipeline: dispatch layout of a window of tokens ----------------------------------
@pytest.mark.parametrize("name,over,batch,cut", [
    ("mid", dict(slots_per_rank=3), 2, 2048),                      # the even split of the paper
    ("tiny", dict(slots_per_rank=2), 1, 511),                      # odd cut: ragged, unaligned rows
    ("dsv3", dict(slots_per_rank=2, tokens_per_rank=1024), 1, 384),
    ("tiny", dict(slots_per_rank=1), 2, 0),                        # an empty first chunk
])
def test_two_chunk_dispatch_windows_match_the_oracle(name, over, batch, cut):
    """The routed tokens are cut into chunks c1 = tokens [0, cut) and c2 = [cut, T) of every source.
    Each chunk's send/receive positions and instance offsets must equal the oracle's dispatch
    permutation of that slice of token_replica; its counts are a bincount of the slice, its offsets
    their cumulative sums; the two chunks' counts add up to the plan's dispatch counts."""
    w = wl.CONFIGS[name].replace(**over)
    cfg = oracle_config(w)
    ids = wl.make_topk_ids(w, seed=61, batch=batch)
    pl = make_planner(w, max_batch=batch)
    out = pl.plan(torch.from_numpy(ids).to(pl.device))
    tr = out.token_replica.cpu().numpy()
    R, T, S = w.ranks, w.tokens_per_rank, pl.s_phys
    total = np.zeros((batch, R, R), np.int64)
    for first, count in ((0, cut), (cut, T - cut)):
        send, recv, ioff, counts, offsets = (t.cpu().numpy() for t in
                                             pl.dispatch_window(out.token_replica, first, count))
        for b in range(batch):
            part = np.ascontiguousarray(tr[b][:, first:first + count])
            want_send, want_recv, want_ioff = orc.dispatch_positions(cfg, part)
            assert np.array_equal(send[b], want_send) and np.array_equal(recv[b], want_recv)
            assert np.array_equal(ioff[b], want_ioff)
            flat = part.reshape(R, -1)
            want_counts = np.stack([np.bincount(flat[s][flat[s] >= 0] // S, minlength=R)
                                    for s in range(R)])
            assert np.array_equal(counts[b], want_counts)
            zero = np.zeros((R, 1), np.int64)
            assert np.array_equal(offsets[b, 0], np.concatenate([zero, np.cumsum(want_counts, 1)], 1))
            assert np.array_equal(offsets[b, 1], np.concatenate([zero, np.cumsum(want_counts.T, 1)], 1))
        total += counts
    assert np.array_equal(total, out.dispatch_counts.cpu().numpy())
    # window errors
    assert B.topoep_dispatch_window(pl.handle, out.token_replica, T, batch, T - 1, 2, None, None,
                                    None, None, None, 256, 0, 0) == -6


# ---- quota boundaries against tile boundaries ---------------------------------------------------
@pytest.mark.parametrize("T,pattern", [
    (4 * 4096, "one_expert"),          # every id the same expert: quotas are multiples of a tile
    (4 * 4096, "two_experts_blocks"),  # long runs: whole tiles of one expert, boundary mid-run
    (3 * 4096 + 17, "one_expert"),     # ragged last tile
    (8192, "alternate"),               # two experts interleaved id by id
])
def test_quota_boundaries_on_and_off_tile_edges(T, pattern):
    """A tile whose ids of a split expert fall inside one instance's quota takes that instance
    without ranking; a tile that straddles a boundary ranks.  These id patterns put the quota
    boundaries exactly on tile edges, inside long runs and in a ragged last tile."""
    w = wl.CONFIGS["tiny"].replace(top_k=1, tokens_per_rank=T, slots_per_rank=3, ffn=16)
    R, E = w.ranks, w.experts
    ids = np.empty((2, R, T, 1), np.int32)
    t = np.arange(T)
    for b in range(2):
        for s in range(R):
            hot, other = (3 * s + b) % E, (3 * s + b + 7) % E
            if pattern == "one_expert":
                row = np.full(T, hot)
            elif pattern == "two_experts_blocks":
                row = np.where((t // 6000) % 2 == 0, hot, other)
            else:
                row = np.where(t % 2 == 0, hot, other)
            ids[b, s, :, 0] = row
    gpu, ref, _ = parity(w, 0, ids=ids)
    # the case is only interesting if assignments really are split across instances
    assert ref.summaries["replica_served"].sum() > 0
    for tile_ids in (1024, 8192):
        pl = make_planner(w, max_batch=2)
        pl.set_tuning(B.KNOB_TILE_IDS, tile_ids)
        assert_same(run_gpu(pl, ids), ref)
