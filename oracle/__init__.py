"""CPU oracle of the TopoEP planning step (test infrastructure, not product code).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It wraps the plain-C implementation in ``topoep_oracle.c`` with
ctypes and numpy; it never touches CUDA and shares nothing with the CUDA path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "topoep_oracle.c")
_LIB = os.path.join(_HERE, "libtopoep_oracle.so")
_lib = None

FLAG_BAD_ID = 1
FLAG_REFINE_CAP = 2
TRACE_COLS = 9
TRACE_FIELDS = ("d", "it", "e", "r_b", "r_t", "delta", "L_b", "L_t", "created")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 (single-threaded, no intrinsics)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-Wall", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Config(ctypes.Structure):
    _fields_ = [("nodes", ctypes.c_int32), ("gpus_per_node", ctypes.c_int32),
                ("experts", ctypes.c_int32), ("slots_per_rank", ctypes.c_int32),
                ("top_k", ctypes.c_int32), ("c_intra", ctypes.c_int32),
                ("c_inter", ctypes.c_int32), ("max_refine_iters", ctypes.c_int32),
                ("min_delta", ctypes.c_int32), ("stages", ctypes.c_int32),
                ("reserve_slots", ctypes.c_int32), ("stage1_rank", ctypes.c_int32),
                ("token_bytes", ctypes.c_int64), ("expert_bytes", ctypes.c_int64),
                ("t_ffn", ctypes.c_int64)]


SUMMARY_INT_FIELDS = ("assignments", "l_max", "cross_assignments", "replica_served",
                      "replicas_inter", "replicas_intra", "t_comp", "t_token", "t_replica",
                      "cross_token_bytes", "refine_iters", "reserved")
SUMMARY_FLOAT_FIELDS = ("imbalance", "cross_fraction", "replica_fraction")
SUMMARY_DTYPE = np.dtype([(n, np.int64) for n in SUMMARY_INT_FIELDS] +
                         [(n, np.float64) for n in SUMMARY_FLOAT_FIELDS])


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp = ctypes.c_void_p
        lib.oracle_e_loc.restype = ctypes.c_int
        lib.oracle_e_loc.argtypes = [vp, vp]
        lib.oracle_histogram.restype = None
        lib.oracle_histogram.argtypes = [vp, vp, ctypes.c_int, vp, vp]
        lib.oracle_solve.restype = None
        lib.oracle_solve.argtypes = [vp] * 10 + [vp, vp, ctypes.c_int64, vp]
        lib.oracle_assign_tokens.restype = None
        lib.oracle_assign_tokens.argtypes = [vp, vp, vp, vp, ctypes.c_int, vp, vp]
        lib.oracle_layout.restype = None
        lib.oracle_layout.argtypes = [vp] * 8
        lib.oracle_summary_of.restype = None
        lib.oracle_summary_of.argtypes = [vp] * 7
        lib.oracle_dispatch_positions.restype = None
        lib.oracle_dispatch_positions.argtypes = [vp, vp, ctypes.c_int, vp, vp, vp, vp]
        lib.oracle_replica_pull.restype = None
        lib.oracle_replica_pull.argtypes = [vp, vp, vp, ctypes.c_int64, vp, vp]
        lib.oracle_replica_grad_return.restype = None
        lib.oracle_replica_grad_return.argtypes = [vp, vp, vp, ctypes.c_int64, vp, vp]
        lib.oracle_plan.restype = ctypes.c_int
        lib.oracle_plan.argtypes = [vp, vp, vp, ctypes.c_int, ctypes.c_int] + [vp] * 11
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


@dataclass
class OracleConfig:
    """Problem statement of the paper's "System Model"."""
    nodes: int
    gpus_per_node: int
    experts: int
    slots_per_rank: int
    top_k: int
    token_bytes: int
    expert_bytes: int
    c_intra: int = 1
    c_inter: int = 8
    t_ffn: int = 0
    max_refine_iters: int = 0
    min_delta: int = 0
    main_rank: Optional[np.ndarray] = None   # [E] int32; None = blocked e // (E/R)
    stages: int = 3                          # bit 0 inter-node placement, bit 1 refinement
    reserve_slots: int = 0                   # policy variant: slots stage 1 leaves to refinement
    stage1_rank: int = 0                     # policy variant: 1 = least estimated load (LPT)

    def __post_init__(self):
        R = self.ranks
        if self.main_rank is None:
            if self.experts % R:
                raise ValueError("blocked main map needs E % R == 0")
            self.main_rank = (np.arange(self.experts) // (self.experts // R)).astype(np.int32)
        self.main_rank = np.ascontiguousarray(self.main_rank, dtype=np.int32)
        assert self.main_rank.shape == (self.experts,)
        assert (self.main_rank >= 0).all() and (self.main_rank < R).all()

    @property
    def ranks(self) -> int:
        return self.nodes * self.gpus_per_node

    def c_struct(self) -> _Config:
        return _Config(self.nodes, self.gpus_per_node, self.experts, self.slots_per_rank,
                       self.top_k, self.c_intra, self.c_inter, self.max_refine_iters,
                       self.min_delta, self.stages, self.reserve_slots, self.stage1_rank, self.token_bytes,
                       self.expert_bytes, self.t_ffn)

    @property
    def e_loc(self) -> int:
        c = self.c_struct()
        return int(_load().oracle_e_loc(ctypes.addressof(c), _p(self.main_rank)))

    @property
    def s_phys(self) -> int:
        return self.e_loc + self.slots_per_rank

    @property
    def instances(self) -> int:
        return self.ranks * self.s_phys


@dataclass
class SolveResult:
    x: np.ndarray          # [E][R] int8
    slotmap: np.ndarray    # [R][N_slot] int32
    q: np.ndarray          # [R][E][R] int64
    U: np.ndarray          # [E][R] int64
    L: np.ndarray          # [R] int64
    D: np.ndarray          # [M][E] int64
    iters: np.ndarray      # [M] int32
    flags: int
    trace: np.ndarray = field(default_factory=lambda: np.zeros((0, TRACE_COLS), np.int64))


def histogram(cfg: OracleConfig, ids: np.ndarray):
    """O1: ids [R][T][k] int32 -> (omega [R][E] int64, flags)."""
    R, E = cfg.ranks, cfg.experts
    ids = np.ascontiguousarray(ids, dtype=np.int32).reshape(R, -1, cfg.top_k)
    omega = np.zeros((R, E), np.int64)
    flags = ctypes.c_uint32(0)
    c = cfg.c_struct()
    _load().oracle_histogram(ctypes.addressof(c), _p(ids), ids.shape[1], _p(omega),
                             ctypes.addressof(flags))
    return omega, int(flags.value)


def solve(cfg: OracleConfig, omega: np.ndarray, trace_cap: int = 0) -> SolveResult:
    """O2..O6 from a routing matrix omega [R][E]."""
    M, R, E, N = cfg.nodes, cfg.ranks, cfg.experts, cfg.slots_per_rank
    omega = np.ascontiguousarray(omega, dtype=np.int64)
    assert omega.shape == (R, E) and (omega >= 0).all()
    x = np.zeros((E, R), np.int8)
    slotmap = np.full((R, N), -1, np.int32) if N else np.zeros((R, 0), np.int32)
    slot_buf = np.full(R * N + 1, -1, np.int32)
    q = np.zeros((R, E, R), np.int64)
    U = np.zeros((E, R), np.int64)
    L = np.zeros(R, np.int64)
    D = np.zeros((M, E), np.int64)
    iters = np.zeros(M, np.int32)
    flags = ctypes.c_uint32(0)
    trace = np.zeros((max(trace_cap, 1), TRACE_COLS), np.int64)
    n_trace = ctypes.c_int64(0)
    c = cfg.c_struct()
    _load().oracle_solve(ctypes.addressof(c), _p(cfg.main_rank), _p(omega), _p(x), _p(slot_buf),
                         _p(q), _p(U), _p(L), _p(D), _p(iters), ctypes.addressof(flags),
                         _p(trace) if trace_cap else None, trace_cap,
                         ctypes.addressof(n_trace) if trace_cap else None)
    if N:
        slotmap = slot_buf[:R * N].reshape(R, N).copy()
    return SolveResult(x, slotmap, q, U, L, D, iters, int(flags.value),
                       trace[:min(int(n_trace.value), trace_cap)].copy())


def assign_tokens(cfg: OracleConfig, res: SolveResult, ids: np.ndarray) -> np.ndarray:
    """O7: ids [R][T][k] -> token_replica [R][T][k] int32 (physical instance ids)."""
    R = cfg.ranks
    ids = np.ascontiguousarray(ids, dtype=np.int32).reshape(R, -1, cfg.top_k)
    out = np.empty_like(ids)
    slot_buf = np.concatenate([res.slotmap.ravel(), [-1]]).astype(np.int32)
    c = cfg.c_struct()
    _load().oracle_assign_tokens(ctypes.addressof(c), _p(cfg.main_rank), _p(slot_buf), _p(ids),
                                 ids.shape[1], _p(res.q), _p(out))
    return out


def layout(cfg: OracleConfig, res: SolveResult):
    """O8: (counts [R][R], offsets [2][R][R+1], instance_counts [P]) int32."""
    R = cfg.ranks
    counts = np.zeros((R, R), np.int32)
    offsets = np.zeros((2, R, R + 1), np.int32)
    inst = np.zeros(cfg.instances, np.int32)
    slot_buf = np.concatenate([res.slotmap.ravel(), [-1]]).astype(np.int32)
    c = cfg.c_struct()
    _load().oracle_layout(ctypes.addressof(c), _p(cfg.main_rank), _p(slot_buf), _p(res.q),
                          _p(res.U), _p(counts), _p(offsets), _p(inst))
    return counts, offsets, inst


def summary(cfg: OracleConfig, res: SolveResult) -> np.ndarray:
    """O9: one SUMMARY_DTYPE record."""
    out = np.zeros(1, SUMMARY_DTYPE)
    c = cfg.c_struct()
    _load().oracle_summary_of(ctypes.addressof(c), _p(cfg.main_rank), _p(res.x), _p(res.q),
                              _p(res.L), _p(res.iters), _p(out))
    return out[0]


def dispatch_positions(cfg: OracleConfig, token_replica: np.ndarray):
    """O10 for one plan: token_replica [R][T][k] -> (send_pos, recv_pos, instance_offsets)."""
    R = cfg.ranks
    tr = np.ascontiguousarray(token_replica, dtype=np.int32).reshape(R, -1, cfg.top_k)
    send = np.empty_like(tr)
    recv = np.empty_like(tr)
    inst_off = np.zeros((R, cfg.s_phys + 1), np.int32)
    c = cfg.c_struct()
    _load().oracle_dispatch_positions(ctypes.addressof(c), _p(cfg.main_rank), tr.shape[1], _p(tr),
                                      _p(send), _p(recv), _p(inst_off))
    return send, recv, inst_off


def replica_pull(cfg: OracleConfig, slotmap: np.ndarray, main_params: np.ndarray,
                 replica_buf: np.ndarray) -> np.ndarray:
    """O11: main_params [R][E_loc][W] uint8, replica_buf [R][N_slot][W] uint8 -> updated copy."""
    R, N = cfg.ranks, cfg.slots_per_rank
    mp = np.ascontiguousarray(main_params, dtype=np.uint8)
    out = np.array(replica_buf, dtype=np.uint8, order="C", copy=True)
    W = mp.shape[-1]
    assert mp.shape == (R, cfg.e_loc, W) and out.shape == (R, N, W)
    sm = np.concatenate([np.asarray(slotmap, np.int32).ravel(), [-1]]).astype(np.int32)
    c = cfg.c_struct()
    _load().oracle_replica_pull(ctypes.addressof(c), _p(cfg.main_rank), _p(sm), ctypes.c_int64(W),
                                _p(mp), _p(out))
    return out


def replica_grad_return(cfg: OracleConfig, slotmap: np.ndarray, replica_buf: np.ndarray,
                        grad_acc: np.ndarray) -> np.ndarray:
    """O12: replica_buf [R][N_slot][W], grad_acc [R][R][E_loc][W] uint8 -> updated copy."""
    R, N = cfg.ranks, cfg.slots_per_rank
    rb = np.ascontiguousarray(replica_buf, dtype=np.uint8)
    out = np.array(grad_acc, dtype=np.uint8, order="C", copy=True)
    W = rb.shape[-1]
    assert rb.shape == (R, N, W) and out.shape == (R, R, cfg.e_loc, W)
    sm = np.concatenate([np.asarray(slotmap, np.int32).ravel(), [-1]]).astype(np.int32)
    c = cfg.c_struct()
    _load().oracle_replica_grad_return(ctypes.addressof(c), _p(cfg.main_rank), _p(sm),
                                       ctypes.c_int64(W), _p(rb), _p(out))
    return out


@dataclass
class PlanResult:
    replica_map: np.ndarray       # [B][R][N_slot]
    token_replica: Optional[np.ndarray]  # [B][R][T][k]
    dispatch_counts: np.ndarray   # [B][R][R]
    dispatch_offsets: np.ndarray  # [B][2][R][R+1]
    instance_counts: np.ndarray   # [B][P]
    omega: np.ndarray             # [B][R][E]
    rank_load: np.ndarray         # [B][R]
    refine_iters: np.ndarray      # [B][M]
    q_instances: Optional[np.ndarray]    # [B][R][P]
    summaries: np.ndarray         # [B] SUMMARY_DTYPE
    flags: int


def plan(cfg: OracleConfig, ids: np.ndarray, want_tokens: bool = True,
         want_q: bool = True) -> PlanResult:
    """The whole path for ids [B][R][T][k] int32; outputs laid out like the library's."""
    M, R, E, N, k = cfg.nodes, cfg.ranks, cfg.experts, cfg.slots_per_rank, cfg.top_k
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    assert ids.ndim == 4 and ids.shape[1] == R and ids.shape[3] == k
    B, T = ids.shape[0], ids.shape[2]
    P = cfg.instances
    rm = np.full((B, R, N), -1, np.int32)
    rm_buf = np.full(B * R * N + 1, -1, np.int32)
    tr = np.empty((B, R, T, k), np.int32) if want_tokens else None
    counts = np.zeros((B, R, R), np.int32)
    offsets = np.zeros((B, 2, R, R + 1), np.int32)
    inst = np.zeros((B, P), np.int32)
    omega = np.zeros((B, R, E), np.int32)
    load = np.zeros((B, R), np.int32)
    iters = np.zeros((B, M), np.int32)
    qi = np.zeros((B, R, P), np.int32) if want_q else None
    summ = np.zeros(max(B, 1), SUMMARY_DTYPE)
    flags = ctypes.c_uint32(0)
    c = cfg.c_struct()
    rc = _load().oracle_plan(ctypes.addressof(c), _p(cfg.main_rank), _p(ids), T, B, _p(rm_buf),
                             _p(tr), _p(counts), _p(offsets), _p(inst), _p(omega), _p(load),
                             _p(iters), _p(qi), _p(summ), ctypes.addressof(flags))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    if N:
        rm = rm_buf[:B * R * N].reshape(B, R, N).copy()
    return PlanResult(rm, tr, counts, offsets, inst, omega, load, iters, qi, summ[:B],
                      int(flags.value))
