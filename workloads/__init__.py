"""Seeded synthetic routing workloads (inputs only; none of the method's arithmetic).

The five shapes follow the benchmark configurations: a Zipf popularity over a
seeded permutation of the experts, shared by all source ranks of one
(layer, microbatch) plan -- the same structure as the paper's synthetic
routing (random logits plus a fixed expert-specific bias, "End-to-End
Performance") -- optionally with a few seeded "burst" experts whose weight is
multiplied.  Each token draws k distinct experts.

Both the CPU oracle's tests and the CUDA path's tests / bench read the buffers
made here; neither side's code is used to make them.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libwlgen.so")
_lib = None

BASE_SEED = 20260935


def build(force: bool = False) -> str:
    """Compile the generator with gcc (OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.wl_hash.restype = ctypes.c_uint64
        lib.wl_hash.argtypes = [ctypes.c_uint64] * 4
        lib.wl_gen_topk.restype = ctypes.c_int
        lib.wl_gen_topk.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                    ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                    ctypes.c_void_p]
        _lib = lib
    return _lib


@dataclasses.dataclass(frozen=True)
class Workload:
    """Topology, model and routing-skew description of one benchmark shape."""
    name: str
    nodes: int                 # M
    gpus_per_node: int         # G
    experts: int               # E
    slots_per_rank: int        # N_slot
    top_k: int
    tokens_per_rank: int       # T
    batch: int = 1             # B plans per call
    hidden: int = 1024
    ffn: int = 2048
    c_intra: int = 1
    c_inter: int = 8
    main_map: str = "blocked"  # "blocked": e // (E/R); "round_robin": e % R
    zipf_s: float = 1.0        # popularity exponent; None-like <0 means per-plan draw
    zipf_s_range: Optional[tuple] = None   # (lo, hi): s drawn per plan by hash
    bursts: int = 0            # experts per plan whose weight is multiplied
    burst_mult: float = 3.0
    uniform: bool = False      # control run: equal weights

    @property
    def ranks(self) -> int:
        return self.nodes * self.gpus_per_node

    @property
    def token_bytes(self) -> int:        # S_tok, bf16 activations
        return 2 * self.hidden

    @property
    def expert_bytes(self) -> int:       # ||W||, three bf16 FFN matrices
        return 3 * self.hidden * self.ffn * 2

    @property
    def t_ffn(self) -> int:              # reporting only; never changes a plan
        return (6 * self.hidden * self.ffn) // 1000

    @property
    def assignments(self) -> int:
        return self.batch * self.ranks * self.tokens_per_rank * self.top_k

    def main_rank(self) -> np.ndarray:
        e = np.arange(self.experts, dtype=np.int64)
        if self.main_map == "round_robin":
            return (e % self.ranks).astype(np.int32)
        if self.experts % self.ranks:
            raise ValueError("blocked main map needs E % R == 0")
        return (e // (self.experts // self.ranks)).astype(np.int32)

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    # 0: 2 x 4 ranks, 32 experts round-robin, top-2, 1024 tokens/rank, Zipf 1.2
    "tiny": Workload("tiny", 2, 4, 32, 1, 2, 1024, hidden=1024, ffn=2048,
                     main_map="round_robin", zipf_s=1.2),
    # 1: 4 x 8 ranks, 64 experts, top-6, 4096 tokens/rank, Zipf 1.0
    "mid": Workload("mid", 4, 8, 64, 1, 6, 4096, hidden=2048, ffn=1408, zipf_s=1.0),
    # 2: DeepSeek-V3-shaped layer: 256 experts, top-8, 8192 tokens/rank, Zipf 1.1 + bursts
    "dsv3": Workload("dsv3", 4, 8, 256, 1, 8, 8192, hidden=7168, ffn=2048, zipf_s=1.1,
                     bursts=4, burst_mult=3.0),
    # 3: 58 layers x 4 microbatches of the dsv3 shape, s ~ U[0.8, 1.4] per plan
    "dsv3_batched": Workload("dsv3_batched", 4, 8, 256, 1, 8, 8192, batch=58 * 4, hidden=7168,
                             ffn=2048, zipf_s_range=(0.8, 1.4), bursts=4, burst_mult=3.0),
    # 4: 16 x 8 ranks, 512 experts, 2 slots, top-8, 16384 tokens/rank, Zipf 1.5
    "scaleout": Workload("scaleout", 16, 8, 512, 2, 8, 16384, hidden=7168, ffn=2048,
                         zipf_s=1.5),
    "scaleout_uniform": Workload("scaleout_uniform", 16, 8, 512, 2, 8, 16384, hidden=7168,
                                 ffn=2048, uniform=True),
}


def _hash(seed: int, a: int, b: int, c: int) -> int:
    return int(_load().wl_hash(seed & (2**64 - 1), a & (2**64 - 1), b & (2**64 - 1),
                               c & (2**64 - 1)))


def plan_popularity(w: Workload, seed: int, plan: int) -> np.ndarray:
    """Per-expert sampling weights (float64, sum 1) of plan `plan`."""
    E = w.experts
    if w.uniform:
        return np.full(E, 1.0 / E)
    # Fisher-Yates permutation of the experts from the hash stream.
    perm = np.arange(E, dtype=np.int64)
    for i in range(E - 1, 0, -1):
        j = _hash(seed, plan, i, 0x7065726d) % (i + 1)
        perm[i], perm[j] = perm[j], perm[i]
    if w.zipf_s_range is not None:
        lo, hi = w.zipf_s_range
        s = lo + (hi - lo) * (_hash(seed, plan, 0, 0x7a697066) >> 11) / float(1 << 53)
    else:
        s = w.zipf_s
    weights = np.empty(E, dtype=np.float64)
    weights[perm] = (np.arange(E, dtype=np.float64) + 1.0) ** (-s)
    if w.bursts:
        chosen = []
        a = 0
        while len(chosen) < min(w.bursts, E):
            e = _hash(seed, plan, a, 0x6275727374) % E
            a += 1
            if e not in chosen:
                chosen.append(e)
        weights[np.array(chosen)] *= w.burst_mult
    return weights / weights.sum()


def _cdf63(weights: np.ndarray) -> np.ndarray:
    c = np.cumsum(weights) / weights.sum()
    cdf = np.minimum(np.floor(c * float(1 << 63)), float((1 << 63) - 1024)).astype(np.uint64)
    cdf[-1] = np.uint64(1 << 63)
    inc = np.diff(np.concatenate(([np.uint64(0)], cdf)).astype(np.float64))
    if not (inc > 0).all():
        raise ValueError("an expert has zero sampling width")
    return cdf


def make_topk_ids(w: Workload, seed: int = BASE_SEED, batch: Optional[int] = None,
                  plan_base: int = 0, out: Optional[np.ndarray] = None) -> np.ndarray:
    """int32 [B][R][T][k] top-k expert ids for plans plan_base .. plan_base+B-1."""
    B = w.batch if batch is None else batch
    R, T, k, E = w.ranks, w.tokens_per_rank, w.top_k, w.experts
    cdf = np.stack([_cdf63(plan_popularity(w, seed, plan_base + b)) for b in range(B)]) \
        if B else np.zeros((0, E), np.uint64)
    cdf = np.ascontiguousarray(cdf)
    if out is None:
        out = np.empty((B, R, T, k), dtype=np.int32)
    assert out.dtype == np.int32 and out.flags.c_contiguous and out.size == B * R * T * k
    if out.size:
        rc = _load().wl_gen_topk(seed, plan_base, B, R, T, k, E, cdf.ctypes.data, out.ctypes.data)
        if rc != 0:
            raise ValueError("wl_gen_topk rejected the shape (k > E or k > 64)")
    return out.reshape(B, R, T, k)


def make_param_bytes(shape, seed: int) -> np.ndarray:
    """Seeded stand-in for expert parameters or gradients: uniform random bytes of `shape`."""
    return np.random.default_rng(seed).integers(0, 256, size=shape, dtype=np.uint8)
