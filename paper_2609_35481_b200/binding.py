"""ctypes binding of libtopoep.so: argument marshalling only.

Every function has the name and argument order of its C declaration in
include/topoep.h; tensors are passed as raw device pointers, streams as raw
cudaStream_t handles.  There is no fallback: if the CUDA library is missing or
cannot be loaded, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtopoep.so")

OK = 0
FLAG_BAD_ID, FLAG_REFINE_CAP, FLAG_INTERNAL = 1, 2, 4
T_OMEGA, T_Q, T_RANK_LOAD, T_REFINE_ITERS, T_D, T_U = 0, 1, 2, 3, 4, 5
KNOB_TILE_IDS, KNOB_HIST_MODE, KNOB_PDL, KNOB_TRANSFER_MODE, KNOB_TRANSFER_SELFTEST, KNOB_CHAIN = 0, 1, 2, 3, 4, 5
KNOB_PACKED_IDS, KNOB_REROUTE_TILES = 6, 7

EXPORTS = ("topoep_create", "topoep_destroy", "topoep_workspace_bytes", "topoep_set_workspace",
           "topoep_plan", "topoep_histogram", "topoep_histogram_static", "topoep_solve", "topoep_reroute", "topoep_dispatch_scratch_bytes", "topoep_dispatch_positions", "topoep_dispatch_window",
           "topoep_summary", "topoep_read_status",
           "topoep_debug_tensor", "topoep_set_tuning", "topoep_set_rank_window", "topoep_set_policy", "topoep_replica_pull", "topoep_replica_grad_return",
           "topoep_get_layout", "topoep_plan_kernels", "topoep_plan_byte_copy",
           "topoep_launch_floor", "topoep_strerror")


class CostParams(ctypes.Structure):
    _fields_ = [("token_bytes", ctypes.c_int64), ("expert_bytes", ctypes.c_int64),
                ("c_intra", ctypes.c_int32), ("c_inter", ctypes.c_int32),
                ("t_ffn", ctypes.c_int64), ("max_refine_iters", ctypes.c_int32),
                ("min_delta", ctypes.c_int32)]


class Summary(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("assignments", "l_max", "cross_assignments", "replica_served", "replicas_inter",
                 "replicas_intra", "t_comp", "t_token", "t_replica", "cross_token_bytes",
                 "refine_iters", "reserved")] + \
               [(n, ctypes.c_double) for n in ("imbalance", "cross_fraction", "replica_fraction")]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree by paper_2609_35481_b200.build)."""
    global _lib
    if _lib is None:
        # Stale or missing library: compile it in-tree (nvcc, sm_100a).  There is no other
        # implementation to fall back to; a failed build raises.
        from . import build as _build
        path = LIB_PATH
        if os.environ.get("TOPOEP_CHECKED_BUILD") == "1":
            # the tests' bounds-checked build of the same sources (same entry points)
            path = _build.build_checked()
        else:
            _build.build()
        if not os.path.exists(path):
            raise RuntimeError("libtopoep.so could not be built (there is no CPU fallback)")
        L = ctypes.CDLL(path)
        vp, ci, i32p = ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p
        L.topoep_create.restype = ci
        L.topoep_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, ci, ci, i32p,
                                    ctypes.POINTER(CostParams)]
        L.topoep_destroy.restype = None
        L.topoep_destroy.argtypes = [vp]
        L.topoep_workspace_bytes.restype = ctypes.c_size_t
        L.topoep_workspace_bytes.argtypes = [vp]
        L.topoep_set_workspace.restype = ci
        L.topoep_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
        L.topoep_plan.restype = ci
        L.topoep_plan.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp, vp, vp]
        L.topoep_histogram.restype = ci
        L.topoep_histogram.argtypes = [vp, vp, ci, ci, vp, vp]
        L.topoep_histogram_static.restype = ci
        L.topoep_histogram_static.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp]
        L.topoep_solve.restype = ci
        L.topoep_solve.argtypes = [vp, vp, ci, vp, vp, vp, vp, vp]
        L.topoep_reroute.restype = ci
        L.topoep_reroute.argtypes = [vp, vp, ci, ci, vp, vp]
        L.topoep_dispatch_scratch_bytes.restype = ctypes.c_size_t
        L.topoep_dispatch_scratch_bytes.argtypes = [vp, ci, ci]
        L.topoep_dispatch_positions.restype = ci
        L.topoep_dispatch_positions.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.topoep_dispatch_window.restype = ci
        L.topoep_dispatch_window.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp,
                                             ctypes.c_size_t, vp]
        L.topoep_summary.restype = ci
        L.topoep_summary.argtypes = [vp, ci, vp, vp]
        L.topoep_read_status.restype = ci
        L.topoep_read_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
        L.topoep_debug_tensor.restype = ci
        L.topoep_debug_tensor.argtypes = [vp, ci, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_size_t)]
        L.topoep_set_tuning.restype = ci
        L.topoep_set_tuning.argtypes = [vp, ci, ci]
        L.topoep_set_policy.restype = ci
        L.topoep_set_policy.argtypes = [vp, ci, ci]
        L.topoep_set_rank_window.restype = ci
        L.topoep_set_rank_window.argtypes = [vp, ci, ci]
        for fn in (L.topoep_replica_pull, L.topoep_replica_grad_return):
            fn.restype = ci
            fn.argtypes = [vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.topoep_get_layout.restype = ci
        L.topoep_get_layout.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.topoep_plan_kernels.restype = ci
        L.topoep_plan_kernels.argtypes = [vp, ci, ci]
        L.topoep_plan_byte_copy.restype = ci
        L.topoep_plan_byte_copy.argtypes = [vp, ci, ci]
        L.topoep_launch_floor.restype = ci
        L.topoep_launch_floor.argtypes = [ci, vp]
        L.topoep_strerror.restype = ctypes.c_char_p
        L.topoep_strerror.argtypes = [ci]
        _lib = L
    return _lib


class TopoEPError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__("topoep status %d: %s" % (status, topoep_strerror(status)))


def _ptr(t) -> Optional[int]:
    """Raw address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def topoep_strerror(status: int) -> str:
    return lib().topoep_strerror(status).decode()


def topoep_create(nodes, gpus_per_node, experts, slots_per_rank, top_k, max_tokens_per_rank,
                  max_batch, main_rank_host, cost: CostParams):
    """Returns (status, handle).  main_rank_host: numpy int32 [E] or None."""
    h = ctypes.c_void_p()
    rc = lib().topoep_create(ctypes.byref(h), nodes, gpus_per_node, experts, slots_per_rank, top_k,
                             max_tokens_per_rank, max_batch, _ptr(main_rank_host),
                             ctypes.byref(cost) if cost is not None else None)
    return rc, (h if rc == OK else None)


def topoep_destroy(h) -> None:
    lib().topoep_destroy(h)


def topoep_workspace_bytes(h) -> int:
    return int(lib().topoep_workspace_bytes(h))


def topoep_set_workspace(h, dev_ptr, nbytes: int) -> int:
    return lib().topoep_set_workspace(h, _ptr(dev_ptr), nbytes)


def topoep_plan(h, dev_topk_ids, tokens_per_rank, batch, dev_replica_map, dev_token_replica,
                dev_dispatch_counts, dev_dispatch_offsets, dev_instance_counts, stream=0) -> int:
    return lib().topoep_plan(h, _ptr(dev_topk_ids), tokens_per_rank, batch, _ptr(dev_replica_map),
                             _ptr(dev_token_replica), _ptr(dev_dispatch_counts),
                             _ptr(dev_dispatch_offsets), _ptr(dev_instance_counts), stream or None)


def topoep_histogram(h, dev_topk_ids, tokens_per_rank, batch, dev_omega, stream=0) -> int:
    return lib().topoep_histogram(h, _ptr(dev_topk_ids), tokens_per_rank, batch, _ptr(dev_omega),
                                  stream or None)


def topoep_histogram_static(dev_topk_ids, batch, ranks, tokens_per_rank, top_k, experts, dev_omega,
                            dev_flags=None, stream=0) -> int:
    """Histogram without handle or workspace, for callers that may not allocate device memory:
    the per-tile scratch is an 8 MiB array inside the library.  Returns -11 when the problem does
    not fit that array.  Make the first call on a device outside stream capture; calls that
    overlap on the GPU race on the shared array."""
    return lib().topoep_histogram_static(_ptr(dev_topk_ids), batch, ranks, tokens_per_rank, top_k,
                                         experts, _ptr(dev_omega), _ptr(dev_flags), stream or None)


def topoep_solve(h, dev_omega, batch, dev_replica_map, dev_dispatch_counts, dev_dispatch_offsets,
                 dev_instance_counts, stream=0) -> int:
    return lib().topoep_solve(h, _ptr(dev_omega), batch, _ptr(dev_replica_map),
                              _ptr(dev_dispatch_counts), _ptr(dev_dispatch_offsets),
                              _ptr(dev_instance_counts), stream or None)


def topoep_reroute(h, dev_topk_ids, tokens_per_rank, batch, dev_token_replica, stream=0) -> int:
    return lib().topoep_reroute(h, _ptr(dev_topk_ids), tokens_per_rank, batch,
                                _ptr(dev_token_replica), stream or None)


def topoep_dispatch_scratch_bytes(h, tokens_per_rank, batch) -> int:
    return int(lib().topoep_dispatch_scratch_bytes(h, tokens_per_rank, batch))


def topoep_dispatch_positions(h, dev_token_replica, tokens_per_rank, batch, dev_send_pos,
                              dev_recv_pos, dev_instance_offsets, dev_scratch, scratch_bytes,
                              stream=0) -> int:
    return lib().topoep_dispatch_positions(h, _ptr(dev_token_replica), tokens_per_rank, batch,
                                           _ptr(dev_send_pos), _ptr(dev_recv_pos),
                                           _ptr(dev_instance_offsets), _ptr(dev_scratch),
                                           scratch_bytes, stream or None)


def topoep_dispatch_window(h, dev_token_replica, tokens_per_rank, batch, first_token, token_count,
                           dev_send_pos, dev_recv_pos, dev_instance_offsets, dev_counts,
                           dev_offsets, dev_scratch, scratch_bytes, stream=0) -> int:
    return lib().topoep_dispatch_window(h, _ptr(dev_token_replica), tokens_per_rank, batch,
                                        first_token, token_count, _ptr(dev_send_pos),
                                        _ptr(dev_recv_pos), _ptr(dev_instance_offsets),
                                        _ptr(dev_counts), _ptr(dev_offsets), _ptr(dev_scratch),
                                        scratch_bytes, stream or None)


def topoep_summary(h, batch, dev_out, stream=0) -> int:
    return lib().topoep_summary(h, batch, _ptr(dev_out), stream or None)


def topoep_read_status(h):
    """Returns (status, flags)."""
    f = ctypes.c_uint32(0)
    rc = lib().topoep_read_status(h, ctypes.byref(f))
    return rc, int(f.value)


def topoep_debug_tensor(h, which: int):
    """Returns (status, device address, bytes)."""
    p, n = ctypes.c_void_p(), ctypes.c_size_t()
    rc = lib().topoep_debug_tensor(h, which, ctypes.byref(p), ctypes.byref(n))
    return rc, (p.value or 0), int(n.value)


def topoep_set_tuning(h, knob: int, value: int) -> int:
    return lib().topoep_set_tuning(h, knob, value)


POLICY_RESERVE_SLOTS, POLICY_STAGE1_RANK = 0, 1


def topoep_set_policy(h, policy: int, value: int) -> int:
    return lib().topoep_set_policy(h, policy, value)


def topoep_set_rank_window(h, first_rank: int, rank_count: int) -> int:
    return lib().topoep_set_rank_window(h, first_rank, rank_count)


def topoep_replica_pull(h, dev_replica_map, dev_main_params, dev_replica_buf, param_bytes,
                        stream=0) -> int:
    return lib().topoep_replica_pull(h, _ptr(dev_replica_map), _ptr(dev_main_params),
                                     _ptr(dev_replica_buf), param_bytes, stream or None)


def topoep_replica_grad_return(h, dev_replica_map, dev_replica_buf, dev_grad_acc, param_bytes,
                               stream=0) -> int:
    return lib().topoep_replica_grad_return(h, _ptr(dev_replica_map), _ptr(dev_replica_buf),
                                            _ptr(dev_grad_acc), param_bytes, stream or None)


def topoep_get_layout(h):
    """Returns (status, e_loc, s_phys, instances)."""
    a, b, c = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    rc = lib().topoep_get_layout(h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    return rc, a.value, b.value, c.value


def topoep_plan_kernels(h, tokens_per_rank: int, batch: int) -> int:
    """Kernels topoep_plan would enqueue for a call of this size (5, or 2 for a small call)."""
    return lib().topoep_plan_kernels(h, tokens_per_rank, batch)


def topoep_plan_byte_copy(h, tokens_per_rank: int, batch: int) -> int:
    """1 when a plan call of this size leaves a one-byte copy of the ids for its reroute kernel."""
    return lib().topoep_plan_byte_copy(h, tokens_per_rank, batch)


def topoep_launch_floor(count: int, stream=0) -> int:
    return lib().topoep_launch_floor(count, stream or None)
