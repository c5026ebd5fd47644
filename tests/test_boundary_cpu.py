"""Host-side checks of the C boundary that need no GPU: the library loads, exports every
declared symbol, and rejects bad arguments with the documented codes."""
import os
import re

import numpy as np

from paper_2609_35481_b200 import binding as B
from paper_2609_35481_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "topoep.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(topoep_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    build_mod.build()
    L = B.lib()
    names = _declared()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(L, n) is not None


def test_strerror_is_total():
    for code in range(-11, 1):
        assert isinstance(B.topoep_strerror(code), str) and B.topoep_strerror(code)


def test_create_rejects_bad_arguments():
    c = B.CostParams(2048, 1 << 20, 1, 8, 0, 0, 0)
    good = dict(nodes=2, gpus_per_node=4, experts=32, slots_per_rank=1, top_k=2,
                max_tokens_per_rank=128, max_batch=1, main_rank_host=None, cost=c)

    def rc(**kw):
        a = dict(good)
        a.update(kw)
        code, h = B.topoep_create(**a)
        if h is not None:
            B.topoep_destroy(h)
        return code

    assert rc() == 0
    assert rc(nodes=0) == -2 and rc(nodes=65) == -2 and rc(gpus_per_node=33) == -2
    assert rc(experts=0) == -2 and rc(slots_per_rank=-1) == -2 and rc(top_k=0) == -2
    assert rc(max_tokens_per_rank=0) == -2 and rc(max_batch=0) == -2
    assert rc(experts=30) == -3                                   # 30 % 8 != 0 with no map
    assert rc(experts=30, main_rank_host=(np.arange(30) % 8).astype(np.int32)) == 0
    bad = (np.arange(32) % 8).astype(np.int32)
    bad[5] = 8
    assert rc(main_rank_host=bad) == -3
    assert rc(cost=B.CostParams(-1, 1, 1, 8, 0, 0, 0)) == -4
    assert rc(cost=B.CostParams(1, 1, -1, 8, 0, 0, 0)) == -4
    assert rc(cost=None) == -1
    assert rc(experts=1 << 14, main_rank_host=(np.arange(1 << 14) % 8).astype(np.int32)) == -9  # shared memory
    # every count of a plan (rank loads, receive offsets) is bounded by R * T * k: it must fit int32
    assert rc(nodes=64, gpus_per_node=32, experts=2048, top_k=1, max_tokens_per_rank=1 << 20) == -2
    assert rc(nodes=64, gpus_per_node=32, experts=2048, top_k=1, max_tokens_per_rank=(1 << 20) - 1) != -2


def test_static_histogram_size_rule_cannot_be_wrapped_around():
    # 4 * batch * ranks * tiles * experts = 2^66 here: the product wraps to 0 in 64 bits, the
    # stepwise check must still refuse it (the pointers are never dereferenced: nothing is enqueued)
    rc = B.topoep_histogram_static(256, 32768, 32768, 2**31 - 1, 1, 8192, 256, None, 0)
    assert rc == -11
    assert B.topoep_histogram_static(256, 1, 1, 2**31 - 1, 2, 8, 256, None, 0) == -2   # T*k >= 2^31


def test_calls_without_workspace_or_handle_fail_cleanly():
    c = B.CostParams(2048, 1 << 20, 1, 8, 0, 0, 0)
    code, h = B.topoep_create(2, 4, 32, 1, 2, 128, 1, None, c)
    assert code == 0
    assert B.topoep_workspace_bytes(h) % 256 == 0 and B.topoep_workspace_bytes(h) > 0
    assert B.topoep_get_layout(h) == (0, 4, 5, 40)
    assert B.topoep_plan(h, 256, 128, 1, 256, 256, 256, 256, None, 0) == -5
    assert B.topoep_histogram(h, 256, 128, 1, 256, 0) == -5
    assert B.topoep_summary(h, 1, 256, 0) == -5
    assert B.topoep_read_status(h)[0] == -5
    assert B.topoep_debug_tensor(h, 0)[0] == -5
    assert B.topoep_set_workspace(h, None, 1 << 20) == -1
    assert B.topoep_set_tuning(h, 99, 0) == -10
    assert B.topoep_set_tuning(h, B.KNOB_TILE_IDS, 2048) == 0
    assert B.topoep_set_tuning(h, B.KNOB_PACKED_IDS, 2) == 0
    assert B.topoep_set_tuning(h, B.KNOB_PACKED_IDS, 3) == -10
    assert B.topoep_set_tuning(h, B.KNOB_REROUTE_TILES, 64) == 0
    assert B.topoep_set_tuning(h, B.KNOB_REROUTE_TILES, 0) == -10
    B.topoep_destroy(h)
    assert B.topoep_workspace_bytes(None) == 0
    assert B.topoep_plan(None, 0, 0, 0, 0, 0, 0, 0, 0, 0) == -1
    B.topoep_destroy(None)
