"""Convenience holder around the C handle: owns the torch workspace and output tensors.

Marshalling only -- every step of the planning path runs in the CUDA library.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import binding as B


@dataclass
class PlanOutputs:
    replica_map: torch.Tensor       # [B][R][N_slot] int32
    token_replica: torch.Tensor     # [B][R][T][k]   int32
    dispatch_counts: torch.Tensor   # [B][R][R]      int32
    dispatch_offsets: torch.Tensor  # [B][2][R][R+1] int32
    instance_counts: torch.Tensor   # [B][P]         int32


class Planner:
    """topoep_create + workspace on the current CUDA device."""

    def __init__(self, nodes, gpus_per_node, experts, slots_per_rank, top_k, max_tokens_per_rank,
                 max_batch=1, token_bytes=0, expert_bytes=0, c_intra=1, c_inter=8, t_ffn=0,
                 max_refine_iters=0, min_delta=0, main_rank: Optional[np.ndarray] = None,
                 device: Optional[torch.device] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("TopoEP planning needs a CUDA device; there is no CPU path")
        self.device = torch.device(device) if device is not None else torch.device(
            "cuda", torch.cuda.current_device())
        self.M, self.G, self.E, self.N, self.k = nodes, gpus_per_node, experts, slots_per_rank, top_k
        self.R = nodes * gpus_per_node
        self.max_tokens, self.max_batch = max_tokens_per_rank, max_batch
        cost = B.CostParams(token_bytes, expert_bytes, c_intra, c_inter, t_ffn, max_refine_iters,
                            min_delta)
        mr = None if main_rank is None else np.ascontiguousarray(main_rank, dtype=np.int32)
        rc, self.handle = B.topoep_create(nodes, gpus_per_node, experts, slots_per_rank, top_k,
                                          max_tokens_per_rank, max_batch, mr, cost)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        rc, self.e_loc, self.s_phys, self.P = B.topoep_get_layout(self.handle)
        self.window = (0, self.R)
        nbytes = B.topoep_workspace_bytes(self.handle)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            rc = B.topoep_set_workspace(self.handle, self._ws_ptr, nbytes)
        if rc != B.OK:
            B.topoep_destroy(self.handle)
            self.handle = None
            raise B.TopoEPError(rc)

    def close(self):
        if getattr(self, "handle", None) is not None:
            B.topoep_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:   # interpreter shutdown: the binding module may already be gone
            pass

    def alloc_outputs(self, batch: int, tokens_per_rank: int) -> PlanOutputs:
        i32 = dict(dtype=torch.int32, device=self.device)
        R = self.R
        return PlanOutputs(torch.empty((batch, R, self.N), **i32),
                           torch.empty((batch, self.window[1], tokens_per_rank, self.k), **i32),
                           torch.empty((batch, R, R), **i32),
                           torch.empty((batch, 2, R, R + 1), **i32),
                           torch.empty((batch, self.P), **i32))

    def plan(self, topk_ids: torch.Tensor, out: Optional[PlanOutputs] = None,
             stream: Optional[torch.cuda.Stream] = None) -> PlanOutputs:
        """topoep_plan on ids [B][R][T][k] (int32, contiguous, on this device)."""
        assert topk_ids.dtype == torch.int32 and topk_ids.is_contiguous() and topk_ids.is_cuda
        Bn, R, T, k = topk_ids.shape
        assert R == self.R and k == self.k
        if out is None:
            out = self.alloc_outputs(Bn, T)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = B.topoep_plan(self.handle, topk_ids, T, Bn, out.replica_map, out.token_replica,
                           out.dispatch_counts, out.dispatch_offsets, out.instance_counts,
                           st.cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        return out

    def dispatch_positions(self, token_replica: torch.Tensor, stream=None):
        """(send_pos, recv_pos, instance_offsets) of the plan that produced token_replica."""
        Bn, R, T, k = token_replica.shape
        i32 = dict(dtype=torch.int32, device=self.device)
        send = torch.empty((Bn, R, T, k), **i32)
        recv = torch.empty((Bn, R, T, k), **i32)
        inst_off = torch.empty((Bn, R, self.s_phys + 1), **i32)
        nbytes = B.topoep_dispatch_scratch_bytes(self.handle, T, Bn)
        scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        ptr = (scratch.data_ptr() + 255) // 256 * 256
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = B.topoep_dispatch_positions(self.handle, token_replica, T, Bn, send, recv, inst_off,
                                         ptr, nbytes, st.cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        st.synchronize()   # the scratch tensor is released when this returns
        return send, recv, inst_off

    def dispatch_window(self, token_replica: torch.Tensor, first_token: int, token_count: int,
                        stream=None):
        """(send_pos, recv_pos, instance_offsets, counts, offsets) of one chunk of tokens,
        first_token .. first_token + token_count - 1 of every source rank."""
        Bn, R, T, k = token_replica.shape
        i32 = dict(dtype=torch.int32, device=self.device)
        send = torch.empty((Bn, R, token_count, k), **i32)
        recv = torch.empty((Bn, R, token_count, k), **i32)
        inst_off = torch.empty((Bn, R, self.s_phys + 1), **i32)
        counts = torch.empty((Bn, R, R), **i32)
        offsets = torch.empty((Bn, 2, R, R + 1), **i32)
        nbytes = B.topoep_dispatch_scratch_bytes(self.handle, token_count, Bn)
        scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        ptr = (scratch.data_ptr() + 255) // 256 * 256
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = B.topoep_dispatch_window(self.handle, token_replica, T, Bn, first_token, token_count,
                                      send, recv, inst_off, counts, offsets, ptr, nbytes,
                                      st.cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        st.synchronize()   # the scratch tensor is released when this returns
        return send, recv, inst_off, counts, offsets

    def histogram(self, topk_ids: torch.Tensor, stream=None) -> torch.Tensor:
        """topoep_histogram on ids [B][rank window][T][k]; returns Omega rows [B][window][E]."""
        Bn, R, T, k = topk_ids.shape
        assert R == self.window[1]
        omega = torch.empty((Bn, R, self.E), dtype=torch.int32, device=self.device)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = B.topoep_histogram(self.handle, topk_ids, T, Bn, omega, st.cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        return omega

    def set_rank_window(self, first_rank: int, rank_count: int):
        """Sharded deployment: this process holds the ids of ranks first..first+count-1 only."""
        rc = B.topoep_set_rank_window(self.handle, first_rank, rank_count)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        self.window = (first_rank, rank_count)

    def solve(self, omega: Optional[torch.Tensor], batch: int, out: Optional[PlanOutputs] = None,
              tokens_per_rank: int = 0, stream=None) -> PlanOutputs:
        """topoep_solve on the gathered Omega [B][R][E] (None: the one topoep_histogram left)."""
        if out is None:
            out = self.alloc_outputs(batch, tokens_per_rank)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = B.topoep_solve(self.handle, omega, batch, out.replica_map, out.dispatch_counts,
                            out.dispatch_offsets, out.instance_counts, st.cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        return out

    def reroute(self, topk_ids: torch.Tensor, stream=None) -> torch.Tensor:
        """topoep_reroute on the ids given to histogram(); returns token_replica of the window."""
        Bn, R, T, k = topk_ids.shape
        assert R == self.window[1]
        tr = torch.empty((Bn, R, T, k), dtype=torch.int32, device=self.device)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = B.topoep_reroute(self.handle, topk_ids, T, Bn, tr, st.cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        return tr

    def plan_sharded(self, my_topk_ids: torch.Tensor, group=None,
                     out: Optional[PlanOutputs] = None) -> PlanOutputs:
        """One planning step of a process that owns a window of source ranks.

        Every process of `group` (torch.distributed; NCCL, or gloo through host memory) calls this with the ids of its own
        window [B][count][T][k]; windows are equal-sized and ordered by group rank.  The rows of
        the routing matrix are all-gathered (the only exchange: B*R*E int32, never the ids), every
        process solves the whole group's plan from the same matrix, and reroutes its own ids.
        token_replica of the result covers this process's window; the other outputs cover all
        ranks and are identical on every process.
        """
        import torch.distributed as dist
        Bn, cnt, T, _ = my_topk_ids.shape
        world = dist.get_world_size(group)
        me = dist.get_rank(group)
        if cnt * world != self.R:
            raise ValueError("windows of %d ranks x %d processes do not cover %d ranks"
                             % (cnt, world, self.R))
        if self.window != (me * cnt, cnt):
            self.set_rank_window(me * cnt, cnt)
        rows = self.histogram(my_topk_ids)                       # [B][cnt][E]
        if dist.get_backend(group) == "gloo":
            # a host-side group (tests, or processes that share one GPU): the rows travel through
            # host memory, then return to the device
            host = rows.cpu()
            parts = [torch.empty_like(host) for _ in range(world)]
            dist.all_gather(parts, host, group=group)
            allrows = torch.stack(parts).to(self.device)
        else:
            allrows = torch.empty((world,) + tuple(rows.shape), dtype=rows.dtype, device=self.device)
            dist.all_gather_into_tensor(allrows, rows, group=group)
        omega = allrows.permute(1, 0, 2, 3).reshape(Bn, self.R, self.E).contiguous()
        out = self.solve(omega, Bn, out=out, tokens_per_rank=T)
        rc = B.topoep_reroute(self.handle, my_topk_ids, T, Bn, out.token_replica,
                              torch.cuda.current_stream(self.device).cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        return out

    def replica_pull(self, replica_map: torch.Tensor, main_params: torch.Tensor,
                     replica_buf: torch.Tensor, stream=None):
        """topoep_replica_pull for ONE plan: replica_map [R][N_slot] int32, main_params
        [R][E_loc][W] and replica_buf [R][N_slot][W] as uint8 (contiguous, on this device)."""
        self._transfer(B.topoep_replica_pull, replica_map, main_params, replica_buf,
                       (self.R, self.e_loc), (self.R, self.N), stream)

    def replica_grad_return(self, replica_map: torch.Tensor, replica_buf: torch.Tensor,
                            grad_acc: torch.Tensor, stream=None):
        """topoep_replica_grad_return for ONE plan: grad_acc [R][R][E_loc][W] uint8."""
        self._transfer(B.topoep_replica_grad_return, replica_map, replica_buf, grad_acc,
                       (self.R, self.N), (self.R, self.R, self.e_loc), stream)

    def _transfer(self, fn, replica_map, src, dst, src_lead, dst_lead, stream):
        assert replica_map.dtype == torch.int32 and replica_map.is_contiguous()
        assert tuple(replica_map.shape) == (self.R, self.N)
        W = src.shape[-1]
        for t, lead in ((src, src_lead), (dst, dst_lead)):
            assert t.dtype == torch.uint8 and t.is_contiguous() and t.is_cuda
            assert tuple(t.shape) == tuple(lead) + (W,)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = fn(self.handle, replica_map, src, dst, W, st.cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)

    def summary(self, batch: int) -> np.ndarray:
        """Summaries of the last plan as a numpy record array (synchronises)."""
        n = ctypes.sizeof(B.Summary)
        buf = torch.empty(batch * n, dtype=torch.uint8, device=self.device)
        rc = B.topoep_summary(self.handle, batch, buf, torch.cuda.current_stream(self.device).cuda_stream)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        names = [f[0] for f in B.Summary._fields_]
        dt = np.dtype([(nm, np.int64 if i < 12 else np.float64) for i, nm in enumerate(names)])
        return np.frombuffer(buf.cpu().numpy().tobytes(), dtype=dt)

    def status(self) -> int:
        rc, flags = B.topoep_read_status(self.handle)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        return flags

    def debug_tensor(self, which: int, batch: int) -> torch.Tensor:
        """Copy of an intermediate tensor for the first `batch` plans (int32, on the host)."""
        rc, ptr, nbytes = B.topoep_debug_tensor(self.handle, which)
        if rc != B.OK:
            raise B.TopoEPError(rc)
        shape = {B.T_OMEGA: (self.R, self.E), B.T_Q: (self.R, self.P), B.T_RANK_LOAD: (self.R,),
                 B.T_REFINE_ITERS: (self.M,), B.T_D: (self.M, self.E), B.T_U: (self.P,)}[which]
        off = (ptr - self.workspace.data_ptr())
        per = int(np.prod(shape)) * 4
        torch.cuda.synchronize(self.device)
        raw = self.workspace[off:off + batch * per].cpu().numpy()
        return torch.from_numpy(raw.view(np.int32).reshape((batch,) + shape).copy())

    def plans_with_two_kernels(self, tokens_per_rank: int, batch: int) -> bool:
        """True when topoep_plan would take its two-kernel chain for a call of this size."""
        return B.topoep_plan_kernels(self.handle, tokens_per_rank, batch) == 2

    def set_policy(self, policy: int, value: int):
        """Policy variants change the plan (unlike tuning knobs); see topoep_set_policy."""
        rc = B.topoep_set_policy(self.handle, policy, value)
        if rc != B.OK:
            raise B.TopoEPError(rc)

    def set_tuning(self, knob: int, value: int):
        rc = B.topoep_set_tuning(self.handle, knob, value)
        if rc != B.OK:
            raise B.TopoEPError(rc)
