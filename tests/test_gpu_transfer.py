"""Replica parameter executor on the GPU against the CPU oracle, byte for byte (through the C
boundary).  The replica maps come from real plans of the CUDA path and from hand-made corner
cases; every buffer is pre-filled so that a byte written where none should be shows up."""
import numpy as np
import pytest
import torch

import oracle as orc
import workloads as wl
from gpu_common import make_planner, oracle_config
from paper_2609_35481_b200 import binding as B

pytestmark = pytest.mark.gpu


def _both_directions(pl, cfg, rmap, W, seed, mode):
    R, N, e_loc = cfg.ranks, cfg.slots_per_rank, cfg.e_loc
    pl.set_tuning(B.KNOB_TRANSFER_MODE, mode)
    main = wl.make_param_bytes((R, e_loc, W), seed)
    slots0 = wl.make_param_bytes((R, N, W), seed + 1)
    acc0 = wl.make_param_bytes((R, R, e_loc, W), seed + 2)
    d_map = torch.from_numpy(np.ascontiguousarray(rmap, np.int32)).to(pl.device)
    d_main = torch.from_numpy(main).to(pl.device)
    d_slots = torch.from_numpy(slots0).to(pl.device)
    d_acc = torch.from_numpy(acc0).to(pl.device)
    pl.replica_pull(d_map, d_main, d_slots)
    torch.cuda.synchronize()
    want_slots = orc.replica_pull(cfg, rmap, main, slots0)
    assert np.array_equal(d_slots.cpu().numpy(), want_slots), "parameter pull differs"
    assert np.array_equal(d_main.cpu().numpy(), main)
    # backward: the slots now carry gradients
    grads = wl.make_param_bytes((R, N, W), seed + 3)
    d_slots.copy_(torch.from_numpy(grads))
    pl.replica_grad_return(d_map, d_slots, d_acc)
    torch.cuda.synchronize()
    want_acc = orc.replica_grad_return(cfg, rmap, grads, acc0)
    assert np.array_equal(d_acc.cpu().numpy(), want_acc), "gradient return differs"
    assert pl.status() == 0


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("W", [16, 48, 16384, 16400, 100000, 5 * 16384 + 4096])
def test_transfers_follow_a_real_plan(W, mode):
    w = wl.CONFIGS["mid"].replace(slots_per_rank=3)
    pl = make_planner(w)
    ids = wl.make_topk_ids(w, seed=31)
    out = pl.plan(torch.from_numpy(ids).to(pl.device))
    rmap = out.replica_map[0].cpu().numpy()
    assert (rmap >= 0).any() and (rmap < 0).any()
    _both_directions(pl, oracle_config(w), rmap, W, 100 + W % 97, mode)


@pytest.mark.parametrize("mode", [0, 1])
def test_transfers_dsv3_shape_many_chunks_per_cta(mode):
    """32 ranks x 2 slots of 192 KiB + 16 bytes: more chunks than CTAs, a ragged last chunk."""
    w = wl.CONFIGS["dsv3"].replace(slots_per_rank=2, tokens_per_rank=2048)
    pl = make_planner(w)
    out = pl.plan(torch.from_numpy(wl.make_topk_ids(w, seed=32)).to(pl.device))
    rmap = out.replica_map[0].cpu().numpy()
    _both_directions(pl, oracle_config(w), rmap, 192 * 1024 + 16, 7, mode)


@pytest.mark.parametrize("mode", [0, 1])
def test_transfers_hand_made_maps_and_uneven_main_map(mode):
    rng = np.random.default_rng(4)
    w = wl.CONFIGS["tiny"].replace(slots_per_rank=4)
    R, E, N = w.ranks, w.experts, 4
    main_rank = rng.integers(0, R, E).astype(np.int32)
    main_rank[:R] = np.arange(R)                  # every rank owns something
    pl = make_planner(w, main_rank=main_rank)
    cfg = oracle_config(w, main_rank=main_rank)
    full = np.stack([rng.choice([e for e in range(E) if main_rank[e] != r], N, replace=False)
                     for r in range(R)]).astype(np.int32)
    empty = np.full((R, N), -1, np.int32)
    sparse = full.copy()
    sparse[rng.random((R, N)) < 0.7] = -1         # holes anywhere, not only at the end
    for i, rmap in enumerate((full, empty, sparse)):
        _both_directions(pl, cfg, rmap, 20000 * 16, 50 + i, mode)


def test_transfer_argument_errors_and_bad_entries():
    w = wl.CONFIGS["tiny"].replace(slots_per_rank=2)
    pl = make_planner(w)
    R, N, e_loc, W = w.ranks, 2, pl.e_loc, 64
    rmap = torch.full((R, N), -1, dtype=torch.int32, device=pl.device)
    main = torch.zeros((R, e_loc, W), dtype=torch.uint8, device=pl.device)
    slots = torch.full((R, N, W), 7, dtype=torch.uint8, device=pl.device)
    assert B.topoep_replica_pull(pl.handle, None, main, slots, W, 0) == -1
    assert B.topoep_replica_pull(pl.handle, rmap, main, slots, W - 8, 0) == -7
    assert B.topoep_replica_pull(pl.handle, rmap, main.data_ptr() + 4, slots, W, 0) == -7
    assert B.topoep_replica_pull(pl.handle, rmap, main, slots, 0, 0) == 0
    # an entry that is no expert id is skipped and flagged; the other slots are still served
    rmap[0, 0] = w.experts + 5
    e_ok = next(e for e in range(w.experts) if w.main_rank()[e] != 1)
    rmap[1, 1] = e_ok
    main.copy_(torch.from_numpy(wl.make_param_bytes((R, e_loc, W), 9)))
    assert B.topoep_replica_pull(pl.handle, rmap, main, slots, W, 0) == 0
    torch.cuda.synchronize()
    assert pl.status() == B.FLAG_BAD_ID
    got = slots.cpu().numpy()
    m = int(w.main_rank()[e_ok])
    l = int((w.main_rank()[:e_ok] == m).sum())
    assert np.array_equal(got[1, 1], main[m, l].cpu().numpy())
    got[1, 1] = 7
    assert (got == 7).all()


def test_bounded_wait_that_runs_out_flags_drains_and_returns():
    """The bulk engine waits on its ring's barriers with a poll limit.  The self-test knob makes
    block 0 wait for a copy it never issued: that wait runs out, the block must set
    TOPOEP_FLAG_INTERNAL, let its other copies land and return by itself (the context stays
    usable).  Every other block completes, so exactly block 0's chunks keep their old bytes."""
    w = wl.CONFIGS["mid"].replace(slots_per_rank=2)
    pl = make_planner(w)
    cfg = oracle_config(w)
    R, N, e_loc, W = w.ranks, 2, pl.e_loc, 96 * 1024
    rng = np.random.default_rng(8)
    rmap = np.stack([rng.choice([e for e in range(w.experts) if w.main_rank()[e] != r], N,
                                replace=False) for r in range(R)]).astype(np.int32)
    main = wl.make_param_bytes((R, e_loc, W), 3)
    slots0 = np.full((R, N, W), 0xEE, np.uint8)
    d_map = torch.from_numpy(rmap).to(pl.device)
    d_main = torch.from_numpy(main).to(pl.device)
    d_slots = torch.from_numpy(slots0).to(pl.device)
    pl.set_tuning(B.KNOB_TRANSFER_SELFTEST, 1)
    pl.replica_pull(d_map, d_main, d_slots)
    torch.cuda.synchronize()                      # returns: the kernel ended on its own
    assert pl.status() == B.FLAG_INTERNAL
    want = orc.replica_pull(cfg, rmap, main, slots0)
    got = d_slots.cpu().numpy()
    sms = torch.cuda.get_device_properties(pl.device).multi_processor_count
    chunk, grid = 32 * 1024, 2 * sms
    per_block = W // chunk
    skipped = np.zeros((R * N, per_block), bool)  # block 0 owns items 0, grid, 2*grid, ...
    skipped.ravel()[0::grid] = True
    g = got.reshape(R * N, per_block, chunk)
    wv = want.reshape(R * N, per_block, chunk)
    assert np.array_equal(g[~skipped], wv[~skipped])
    assert (g[skipped] == 0xEE).all()
    # switched off again: a normal transfer, no flag
    pl.set_tuning(B.KNOB_TRANSFER_SELFTEST, 0)
    pl.replica_pull(d_map, d_main, d_slots)
    torch.cuda.synchronize()
    assert pl.status() == 0
    assert np.array_equal(d_slots.cpu().numpy(), want)
