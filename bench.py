#!/usr/bin/env python3
"""Benchmark of the TopoEP planning step on B200.

One "step" = one topoep_plan call (histogram -> solver + layout -> reroute) over one batch of
seeded synthetic routing.  Prints ONE JSON line:

  value      top-k assignments planned per second, device-timed with CUDA events over a captured
             CUDA graph of K plans, inputs resident in HBM, rotating over enough distinct buffer
             sets to exceed L2 (so every pass reads its ids from DRAM)
  e2e        the same metric through the public call with HOST buffers: pinned ids copied to the
             device, the plan, every output copied back, all inside the timed region
  roofline   for the kernel with the largest share of the plan: algorithmic bytes / its measured
             launch time against the measured HBM copy bandwidth
  cpu_baseline  the CPU oracle, as it stands, timed on this machine's host cores on a bounded sample

`--impl reference` times only the oracle (the stand-in for a reference implementation: the paper
has no released code).  Under torchrun every rank plans its own seeded batches on its own GPU
(independent replicas, no collective on the data path); times are the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
NCU_REROUTE_ROWS_READ_16 = 42320896   # dram__bytes_read.sum of reroute_rows_kernel, 16 plans
NCU_HIST_PACK_READ_16 = 134238720     # ... of hist_kernel when it also writes the byte copy
NOMINAL_HBM_GBS = 8000.0   # the figure the target statement names; context beside the measured peak
REPEATS = 11               # timed replays of every graph: the median is reported, min and max beside it
# DRAM bytes per PLAN of the DeepSeek-V3-shaped layer.  READS come from the committed ncu captures of
# a 16-plan call (profiles/reroute_kernel_dsv3_batch16.md, profiles/hist_kernel_dsv3_batch16.md and,
# for calls that keep a one-byte copy of the ids, profiles/byte_copy_kernels_dsv3_batch16.md) and
# grow in proportion to the plans of a call (every CTA reads only its own tiles and its source's
# tables).  WRITES do not scale from those captures: the 134 MB of output partly stayed dirty in the
# 126 MB L2 at kernel end, a constant, not a proportion -- a full-size call writes 1.9 GB through
# the same L2, so its DRAM writes are its output bytes (reroute: 4 per assignment; histogram: the
# 16-bit tile counts, E per tile, and with the byte copy 1 per assignment).
NCU_READ_BYTES_PER_PLAN = {("reroute", False): 137112320 / 16, ("hist", False): 134235136 / 16,
                           ("reroute", True): NCU_REROUTE_ROWS_READ_16 / 16, ("hist", True): NCU_HIST_PACK_READ_16 / 16}


def ncu_traffic(w, kernel, tile_ids=4096, byte_copy=False):
    if w.name in ("dsv3", "dsv3_batched") and (kernel, byte_copy) in NCU_READ_BYTES_PER_PLAN:
        per_plan_ids = w.assignments // w.batch
        writes = {"reroute": 4 * per_plan_ids,
                  "hist": 2 * w.experts * (per_plan_ids // tile_ids) + (per_plan_ids if byte_copy else 0)}[kernel]
        return int((NCU_READ_BYTES_PER_PLAN[(kernel, byte_copy)] + writes) * w.batch)
    return None


def rank_plan_base(rank: int, set_index: int) -> int:
    """First plan index of buffer set `set_index` on `rank`: ranks and sets never share a plan."""
    return (rank * 64 + set_index) * 100000


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time (all-reduce MAX); the job is as fast as its slowest replica."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, assignments_per_step: int, steps: int, ms_total: float) -> float:
    """Whole-job assignments per second: every rank plans its own batch each step (weak scaling)."""
    return world * assignments_per_step * steps / (ms_total * 1e-3)


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Polls NVML for SM clock, power and clock-event reasons while the GPU is under load."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks",
               0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self.power = []
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as exc:  # pragma: no cover
            self.err = repr(exc)

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2.0)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0,
                    "note": getattr(self, "err", "no samples")}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": round(max(self.power), 1) if self.power else None}


# ------------------------------------------------------------------------------------------------
# the oracle leg (CPU baseline / --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_config(w):
    import oracle as orc
    return orc.OracleConfig(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                            w.token_bytes, w.expert_bytes, w.c_intra, w.c_inter, w.t_ffn,
                            main_rank=w.main_rank())


def time_oracle(w, ids, budget_s, threads=1):
    """Run the oracle plan by plan on `ids` [B][R][T][k] until the budget is used up.  With
    threads > 1 the independent plans of the batch are dealt to that many host threads (the
    oracle is a C routine behind ctypes, which releases the interpreter lock while it runs)."""
    import oracle as orc
    cfg = oracle_config(w)
    per_plan = ids.shape[1] * ids.shape[2] * ids.shape[3]
    t0 = time.perf_counter()
    if threads <= 1:
        done = 0
        while True:
            b = done % ids.shape[0]
            orc.plan(cfg, ids[b:b + 1], want_q=False)
            done += 1
            if time.perf_counter() - t0 >= budget_s:
                break
        dt = time.perf_counter() - t0
        return done * per_plan / dt, done, dt
    from concurrent.futures import ThreadPoolExecutor
    counts = [0] * threads

    def worker(i):
        n = 0
        while time.perf_counter() - t0 < budget_s:
            b = (i + n * threads) % ids.shape[0]
            orc.plan(cfg, ids[b:b + 1], want_q=False)
            n += 1
        counts[i] = n

    with ThreadPoolExecutor(max_workers=threads) as pool:
        list(pool.map(worker, range(threads)))
    dt = time.perf_counter() - t0
    done = sum(counts)
    return done * per_plan / dt, done, dt


def run_reference(args, w):
    """The oracle as the reference arm: each step plans a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as orc
    orc.build()
    cfg = oracle_config(w)
    # sample: one plan of the workload's shape, tokens per rank cut so that K+W steps fit ~2 min
    probe_T = min(w.tokens_per_rank, 1024)
    ids = wl.make_topk_ids(w.replace(tokens_per_rank=probe_T), seed=wl.BASE_SEED, batch=1)
    t0 = time.perf_counter()
    orc.plan(cfg, ids, want_q=False)
    per_assign = (time.perf_counter() - t0) / ids.size
    budget = 120.0 / max(args.steps + args.warmup, 1)
    T = int(min(w.tokens_per_rank, max(64, budget / per_assign / (w.ranks * w.top_k))))
    ids = wl.make_topk_ids(w.replace(tokens_per_rank=T), seed=wl.BASE_SEED, batch=1)
    for _ in range(args.warmup):
        orc.plan(cfg, ids, want_q=False)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.plan(cfg, ids, want_q=False)
    dt = time.perf_counter() - t0
    value = args.steps * ids.size / dt
    sample = "one plan of the %s shape with %d of %d tokens per rank per step" % (w.name, T, w.tokens_per_rank)
    # the step this arm runs: ONE plan of the workload's shape with T tokens per rank
    step_w = w.replace(tokens_per_rank=T, batch=1)
    cfg_line = workload_config(step_w, 1, None)
    cfg_line["workload"] = w.name
    cfg_line["sampled_from"] = {"tokens_per_rank": w.tokens_per_rank, "plans_per_step": w.batch}
    line = {"impl": "reference", "metric": "topk_assignments_per_s", "value": value,
            "unit": "assignments/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": cfg_line,
            "cpu_baseline": {"value": value, "unit": "assignments/s", "cores": 1, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "assignments/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(w, nsets, l2_policy):
    cfg = {"workload": w.name, "nodes": w.nodes, "gpus_per_node": w.gpus_per_node,
           "ranks": w.ranks, "experts": w.experts, "slots_per_rank": w.slots_per_rank,
           "top_k": w.top_k, "tokens_per_rank": w.tokens_per_rank, "plans_per_step": w.batch,
           "assignments_per_step": w.assignments, "main_map": w.main_map, "seed": wl.BASE_SEED}
    if l2_policy is not None:   # only the GPU arm has buffer sets and an L2 to defeat
        cfg["buffer_sets"] = nsets
        cfg["l2"] = l2_policy
    return cfg


# ------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------
def spread(ms_list, per):
    """median / min / max of repeated timings, each divided by `per`, in microseconds."""
    v = sorted(m / per * 1e3 for m in ms_list)
    return {"median": round(v[len(v) // 2], 3), "min": round(v[0], 3), "max": round(v[-1], 3),
            "repeats": len(v)}


def measure(w, K, W, rank, world, dev, args, stages=True, chain=-1, warm_l2=False):
    """Device-timed K plans of workload w inside one captured CUDA graph, plus per-stage graphs.
    chain: TOPOEP_KNOB_CHAIN for the plan graph (-1: the library's choice).  warm_l2: one buffer
    set only, so that every replay finds its ids in L2 (reported beside the rotating figures)."""
    import torch
    import torch.distributed as dist
    from paper_2609_35481_b200 import Planner, binding as B

    # inputs: nsets distinct seeded batches, each with its own planner, workspace and outputs, so
    # that a rotation over them touches more than twice L2 before any buffer repeats
    ids_bytes = w.assignments * 4
    nsets = 1 if warm_l2 else int(max(1, min(32, -(-2 * L2_BYTES // (2 * ids_bytes)))))
    l2_policy = ("one buffer set: ids and outputs stay in L2 (warm)" if warm_l2 and 2 * ids_bytes < L2_BYTES
                 else "inputs+outputs of one step exceed L2" if nsets == 1 else
                 "rotation over %d distinct input/output/workspace sets (%.0f MB) exceeds L2"
                 % (nsets, nsets * 2 * ids_bytes / 1e6))
    sets = []
    for i in range(nsets):
        ids = wl.make_topk_ids(w, seed=wl.BASE_SEED, plan_base=rank_plan_base(rank, i))
        pl = Planner(w.nodes, w.gpus_per_node, w.experts, w.slots_per_rank, w.top_k,
                     w.tokens_per_rank, max_batch=w.batch, token_bytes=w.token_bytes,
                     expert_bytes=w.expert_bytes, c_intra=w.c_intra, c_inter=w.c_inter,
                     t_ffn=w.t_ffn, main_rank=w.main_rank(), device=dev)
        if args.tile_ids:
            pl.set_tuning(B.KNOB_TILE_IDS, args.tile_ids)
        if args.hist_mode >= 0:
            pl.set_tuning(B.KNOB_HIST_MODE, args.hist_mode)
        if args.pdl >= 0:
            pl.set_tuning(B.KNOB_PDL, args.pdl)
        if chain >= 0:
            pl.set_tuning(B.KNOB_CHAIN, chain)
        if args.packed_ids >= 0:
            pl.set_tuning(B.KNOB_PACKED_IDS, args.packed_ids)
        ids_dev = torch.from_numpy(ids).to(dev)
        sets.append({"pl": pl, "ids_host": ids, "ids": ids_dev,
                     "out": pl.alloc_outputs(w.batch, w.tokens_per_rank)})

    stream = torch.cuda.Stream(device=dev)
    sh = stream.cuda_stream

    def plan(i):
        s = sets[i % nsets]
        s["pl"].plan(s["ids"], s["out"], stream=stream)

    def hist(i):
        s = sets[i % nsets]
        rc = B.topoep_histogram(s["pl"].handle, s["ids"], w.tokens_per_rank, w.batch, None, sh)
        assert rc == 0, rc

    def solve(i):
        s, o = sets[i % nsets], sets[i % nsets]["out"]
        rc = B.topoep_solve(s["pl"].handle, None, w.batch, o.replica_map, o.dispatch_counts,
                            o.dispatch_offsets, o.instance_counts, sh)
        assert rc == 0, rc

    def reroute(i):
        s = sets[i % nsets]
        rc = B.topoep_reroute(s["pl"].handle, s["ids"], w.tokens_per_rank, w.batch,
                              s["out"].token_replica, sh)
        assert rc == 0, rc

    kernels_per_plan = B.topoep_plan_kernels(sets[0]["pl"].handle, w.tokens_per_rank, w.batch)
    byte_copy = B.topoep_plan_byte_copy(sets[0]["pl"].handle, w.tokens_per_rank, w.batch) == 1

    def floor(i):
        assert B.topoep_launch_floor(kernels_per_plan, sh) == 0

    def floor1(i):
        assert B.topoep_launch_floor(1, sh) == 0

    def capture(fn, n):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                for i in range(n):
                    fn(i)
        return g

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed_replay(g):
        """ms of one replay of graph g, events on the launching stream, max over ranks."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(stream):
            e0.record(stream)
            g.replay()
            e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev)

    # warm-up: W eager plans, and every set at least once so each workspace holds its own plan
    with torch.cuda.stream(stream):
        for i in range(max(W, nsets)):
            plan(i)
    torch.cuda.synchronize(dev)
    for s in sets:
        flags = s["pl"].status()
        assert flags == 0, "device status flags %d" % flags

    g_plan = capture(plan, K)
    g_plan.replay()                      # one untimed replay of the captured graph
    plan_ms = [timed_replay(g_plan) for _ in range(REPEATS)]   # each replay: EXACTLY K steps
    ms_total = sorted(plan_ms)[len(plan_ms) // 2]
    del g_plan

    # per-stage times through the stage entry points (same rotation; hist = tile histogram + omega,
    # solve = solver + route tables, reroute: the kernels of the five-kernel chain) and the launch
    # floor: as many empty kernels as the plan has kernels, and one empty kernel
    stage_us, stage_spread = {}, {}
    names = (("hist", hist), ("solve", solve), ("reroute", reroute), ("floor", floor),
             ("floor1", floor1))
    for name, fn in (names if stages else names[3:]):
        g = capture(fn, K)
        g.replay()
        ms = [timed_replay(g) for _ in range(REPEATS)]
        stage_spread[name] = spread(ms, K)
        stage_us[name] = stage_spread[name]["median"]
        del g
    # leave every workspace consistent again (the stage graphs ran stages out of order)
    with torch.cuda.stream(stream):
        for i in range(nsets):
            plan(i)
    torch.cuda.synchronize(dev)
    return {"sets": sets, "nsets": nsets, "l2_policy": l2_policy, "stream": stream,
            "ms_total": ms_total, "ms_step": ms_total / K, "stage_us": stage_us,
            "plan_spread": spread(plan_ms, K), "stage_spread": stage_spread,
            "kernels_per_plan": kernels_per_plan, "byte_copy": byte_copy, "barrier": barrier}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="dsv3_batched", choices=sorted(wl.CONFIGS))
    ap.add_argument("--no-single-plan", action="store_true")
    ap.add_argument("--no-dispatch", action="store_true")
    ap.add_argument("--no-transfer", action="store_true")
    ap.add_argument("--transfer-bytes", type=int, default=0,
                    help="bytes per expert block of the replica transfers (default: the layer's)")
    ap.add_argument("--batch", type=int, default=0, help="override plans per step")
    ap.add_argument("--impl", default="topoep", choices=["topoep", "reference"])
    ap.add_argument("--tile-ids", type=int, default=0)
    ap.add_argument("--hist-mode", type=int, default=-1)
    ap.add_argument("--pdl", type=int, default=-1)
    ap.add_argument("--chain", type=int, default=-1,
                    help="TOPOEP_KNOB_CHAIN for the timed plan (default: the library's choice)")
    ap.add_argument("--packed-ids", type=int, default=-1,
                    help="TOPOEP_KNOB_PACKED_IDS (default: the library's choice; 1 = never)")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = wl.CONFIGS[args.workload]
    if args.batch:
        w = w.replace(batch=args.batch)

    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_35481_b200 import Planner, binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the planning path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    K, W = args.steps, args.warmup

    sampler = ClockSampler(local)
    sampler.start()
    m = measure(w, K, W, rank, world, dev, args, chain=args.chain)
    sets, nsets, l2_policy, stream = m["sets"], m["nsets"], m["l2_policy"], m["stream"]
    ms_step, ms_total, stage_us = m["ms_step"], m["ms_total"], m["stage_us"]
    value = job_throughput(world, w.assignments, K, ms_total)
    barrier = m["barrier"]

    # ---- end to end through the public call with host buffers
    s0 = sets[0]
    host_ids = torch.from_numpy(s0["ids_host"]).pin_memory()
    o = s0["out"]
    dev_outs = [o.replica_map, o.token_replica, o.dispatch_counts, o.dispatch_offsets,
                o.instance_counts]
    host_outs = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in dev_outs]
    h2d = host_ids.numel() * 4
    d2h = sum(t.numel() * 4 for t in dev_outs)

    # The copies of consecutive steps overlap as a user's pipeline would: inputs of step i+1 go up
    # while step i is planned and step i-1's outputs come down (two device buffer sets, three
    # streams).  Every step still moves all its inputs and all its outputs inside the timed region.
    ids2 = [s0["ids"], torch.empty_like(s0["ids"])]
    outs2 = [o, s0["pl"].alloc_outputs(w.batch, w.tokens_per_rank)]
    up, down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_up = [torch.cuda.Event() for _ in range(2)]
    ev_plan = [torch.cuda.Event() for _ in range(2)]
    ev_down = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        j = i & 1
        oj = outs2[j]
        douts = [oj.replica_map, oj.token_replica, oj.dispatch_counts, oj.dispatch_offsets,
                 oj.instance_counts]
        with torch.cuda.stream(up):
            if i >= 2:
                up.wait_event(ev_plan[j])          # the plan two steps back has read this buffer
            ids2[j].copy_(host_ids, non_blocking=True)
            ev_up[j].record(up)
        with torch.cuda.stream(stream):
            stream.wait_event(ev_up[j])
            if i >= 2:
                stream.wait_event(ev_down[j])      # its outputs have been copied out
            s0["pl"].plan(ids2[j], oj, stream=stream)
            ev_plan[j].record(stream)
        with torch.cuda.stream(down):
            down.wait_event(ev_plan[j])
            for hbuf, dbuf in zip(host_outs, douts):
                hbuf.copy_(dbuf, non_blocking=True)
            ev_down[j].record(down)

    k_e2e = max(4, min(K, int(2.0 / max(ms_step * 1e-3 + max(h2d, d2h) / 20e9, 1e-6))))
    s0["pl"].set_tuning(B.KNOB_CHAIN, 0)
    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with torch.cuda.stream(stream):
        e0.record(stream)
    up.wait_event(e0)
    for i in range(k_e2e):
        e2e_step(i + 4)
    with torch.cuda.stream(stream):
        stream.wait_event(ev_down[0])
        stream.wait_event(ev_down[1])
        e1.record(stream)
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev)
    e2e_value = job_throughput(world, w.assignments, k_e2e, ms_e2e)

    # ---- the step after the path: dispatch permutation of the same batch (reported, not timed
    # into `value`)
    dispatch = None
    if not args.no_dispatch:
        pl0 = s0["pl"]
        nb = B.topoep_dispatch_scratch_bytes(pl0.handle, w.tokens_per_rank, w.batch)
        scratch = torch.empty(nb + 256, dtype=torch.uint8, device=dev)
        sptr = (scratch.data_ptr() + 255) // 256 * 256
        send = torch.empty_like(o.token_replica)
        recv = torch.empty_like(o.token_replica)
        ioff = torch.empty((w.batch, w.ranks, pl0.s_phys + 1), dtype=torch.int32, device=dev)

        def dispatch_once():
            rc = B.topoep_dispatch_positions(pl0.handle, o.token_replica, w.tokens_per_rank, w.batch,
                                             send, recv, ioff, sptr, nb, stream.cuda_stream)
            assert rc == 0, rc

        with torch.cuda.stream(stream):
            s0["pl"].plan(s0["ids"], o, stream=stream)
            for _ in range(3):
                dispatch_once()
        n_d = 10
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(stream):
            d0.record(stream)
            for _ in range(n_d):
                dispatch_once()
            d1.record(stream)
        barrier()
        us = max_over_ranks(d0.elapsed_time(d1), world, dev) / n_d * 1e3
        dispatch = {"us_per_call": round(us, 2), "us_per_layer_plan": round(us / w.batch, 3),
                    "bytes_per_assignment": 16,
                    "hbm_frac": round(16 * w.assignments / (us * 1e-6) / 1e9 / measured_peak_gbs()[0], 4),
                    "note": "send/recv positions of every assignment; off the planning path, bound by the per-warp chain of ranking steps"}
        del scratch, send, recv, ioff

    # ---- replica parameter executor driven by plan 0 of the batch (reported, not timed into
    # `value`): forward pull at the layer's full expert size, gradient return at 1/16 of it (the
    # accumulation buffers of all simulated ranks, R*R*E_loc blocks, must fit one GPU)
    transfer = None
    if not args.no_transfer and w.slots_per_rank > 0 and w.expert_bytes >= 256:
        pl0 = s0["pl"]
        R, N, e_loc = w.ranks, w.slots_per_rank, pl0.e_loc
        w_pull = (args.transfer_bytes or w.expert_bytes) // 16 * 16
        while R * e_loc * w_pull > 48 * 2**30:
            w_pull = w_pull // 32 * 16
        w_ret = w_pull
        while R * R * e_loc * w_ret > 48 * 2**30:
            w_ret = w_ret // 32 * 16
        rmap = o.replica_map[0]
        n_occ = int((rmap >= 0).sum().item())
        u8 = dict(dtype=torch.uint8, device=dev)
        main = torch.empty((R, e_loc, w_pull), **u8)
        slots = torch.empty((R, N, w_pull), **u8)
        gslots = torch.empty((R, N, w_ret), **u8)
        acc = torch.empty((R, R, e_loc, w_ret), **u8)
        peak = measured_peak_gbs()[0]

        def time_transfer(fn, a, b_, wb, n_it=10):
            with torch.cuda.stream(stream):
                for _ in range(3):
                    assert fn(pl0.handle, rmap, a, b_, wb, stream.cuda_stream) == 0
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            with torch.cuda.stream(stream):
                t0.record(stream)
                for _ in range(n_it):
                    fn(pl0.handle, rmap, a, b_, wb, stream.cuda_stream)
                t1.record(stream)
            barrier()
            us = max_over_ranks(t0.elapsed_time(t1), world, dev) / n_it * 1e3
            gbs = 2.0 * wb * n_occ / (us * 1e-6) / 1e9 if n_occ else 0.0
            return {"us": round(us, 2), "gbs": round(gbs, 1), "hbm_frac": round(gbs / peak, 4),
                    "param_bytes": wb}

        transfer = {"occupied_slots": n_occ, "slots": R * N,
                    "bytes_per_slot": "read |W| + write |W|"}
        for mode, name in ((0, "bulk"), (1, "plain")):
            pl0.set_tuning(B.KNOB_TRANSFER_MODE, mode)
            transfer[name] = {"pull": time_transfer(B.topoep_replica_pull, main, slots, w_pull),
                              "grad_return": time_transfer(B.topoep_replica_grad_return, gslots,
                                                           acc, w_ret)}
        pl0.set_tuning(B.KNOB_TRANSFER_MODE, 0)
        assert pl0.status() == 0
        del main, slots, gslots, acc

    # ---- latency of ONE layer plan (the single-plan shape of the same layer), same protocol:
    # the library's choice of chain (two kernels for a call this small), the five-kernel chain
    # beside it, and both again with one buffer set (ids warm in L2)
    single = None
    if not args.no_single_plan:
        w1 = wl.CONFIGS["dsv3"] if w.name == "dsv3_batched" else w.replace(batch=1)
        for s_ in sets[1:]:
            s_["pl"].close()

        def close_sets(m):
            for s_ in m["sets"]:
                s_["pl"].close()

        m1 = measure(w1, 200, 20, rank, world, dev, args)
        us = m1["plan_spread"]["median"]
        roof_us = 12 * w1.assignments / measured_peak_gbs()[0] / 1e3
        single = {"workload": w1.name, "steps": 200, "warmup": 20,
                  "us_per_layer_plan": us, "spread_us": m1["plan_spread"],
                  "kernels_per_plan": m1["kernels_per_plan"],
                  "launch_floor_us": m1["stage_us"]["floor"],
                  "launch_floor_one_kernel_us": m1["stage_us"]["floor1"],
                  "vs_launch_floor": round(us / m1["stage_us"]["floor"], 2),
                  "hbm_roofline_us": round(roof_us, 3),
                  "hbm_frac": round(roof_us / us, 4),
                  "hbm_frac_8B": round(roof_us * 8 / 12 / us, 4),
                  "hbm_frac_nominal": round(12 * w1.assignments / NOMINAL_HBM_GBS / 1e3 / us, 4),
                  "five_kernel_stage_us": {n: m1["stage_us"][n] for n in ("hist", "solve", "reroute")},
                  "l2": m1["l2_policy"]}
        close_sets(m1)
        m5 = measure(w1, 200, 20, rank, world, dev, args, stages=False, chain=1)
        single["five_kernel_chain"] = {"us_per_layer_plan": m5["plan_spread"]["median"],
                                       "spread_us": m5["plan_spread"],
                                       "launch_floor_us": m5["stage_us"]["floor"]}
        close_sets(m5)
        mw = measure(w1, 200, 20, rank, world, dev, args, stages=False, warm_l2=True)
        single["warm_l2"] = {"us_per_layer_plan": mw["plan_spread"]["median"],
                             "spread_us": mw["plan_spread"], "l2": mw["l2_policy"]}
        close_sets(mw)
        mw5 = measure(w1, 200, 20, rank, world, dev, args, stages=False, chain=1, warm_l2=True)
        single["warm_l2"]["five_kernel_chain_us"] = mw5["plan_spread"]["median"]
        close_sets(mw5)
    clocks = sampler.finish()

    # the e2e outputs came back to the host: check them against the device copies of the same plan
    assert np.array_equal(host_outs[1].numpy(), o.token_replica.cpu().numpy())

    # ---- roofline of the dominant kernel
    peak, peak_kind = measured_peak_gbs()
    A = w.assignments
    algo_bytes = {"hist": 4 * A, "reroute": 8 * A, "solve": None}
    byte_copy = m["byte_copy"]
    # what the two streaming kernels move when the histogram leaves a one-byte copy of the ids for
    # the reroute kernel: 4 + 1 and 1 + 4 bytes per assignment instead of 4 and 4 + 4
    moved_bytes = {"hist": 5 * A, "reroute": 5 * A} if byte_copy else {"hist": 4 * A, "reroute": 8 * A}
    dominant = max(("hist", "solve", "reroute"), key=lambda n: stage_us[n])
    hbm_kernels = {n: {"us": round(stage_us[n], 3),
                       "achieved_gbs": round(algo_bytes[n] / (stage_us[n] * 1e-6) / 1e9, 1),
                       "frac": round(algo_bytes[n] / (stage_us[n] * 1e-6) / 1e9 / peak, 4),
                       "moved_gbs": round(moved_bytes[n] / (stage_us[n] * 1e-6) / 1e9, 1),
                       "frac_moved": round(moved_bytes[n] / (stage_us[n] * 1e-6) / 1e9 / peak, 4)}
                   for n in ("hist", "reroute")}
    if dominant == "solve":
        # latency-bound: a few CTAs of serial integer work; judged against the launch floor, and
        # reported here with the bytes it has to touch (omega in, q and layout out)
        dom_bytes = 4 * w.batch * (w.ranks * w.experts + w.ranks * sets[0]["pl"].P
                                   + 3 * w.ranks * w.ranks)
        dom_moved = dom_bytes
    else:
        dom_bytes = algo_bytes[dominant]
        dom_moved = moved_bytes[dominant]
    # With the byte copy the dominant kernel's bytes are the ones it moves (its input IS the copy);
    # the 12 B-per-assignment definition of the whole plan stays in plan_frac, and the kernel's
    # figure under that definition in frac_12B_definition.
    achieved = dom_moved / (stage_us[dominant] * 1e-6) / 1e9
    plan_gbs = 12 * A / (ms_step * 1e-3) / 1e9
    plan_moved = (10 if byte_copy else 12) * A
    roofline = {"bound": "hbm", "kernel": {"hist": "hist_kernel", "solve": "solve_kernel",
                                           "reroute": "reroute_rows_kernel" if byte_copy else "reroute_kernel"}[dominant],
                "achieved": round(achieved, 2), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "peak_source": "of " + peak_kind,
                "frac_nominal": round(achieved / NOMINAL_HBM_GBS, 4),
                "traffic": ncu_traffic(w, dominant, args.tile_ids or 4096, byte_copy),
                "traffic_note": "reads: ncu capture of a 16-plan call scaled by plans; writes: "
                                "output bytes (see the comment at NCU_READ_BYTES_PER_PLAN)",
                "algorithmic_bytes_per_launch": dom_moved,
                "byte_copy": byte_copy,
                "bytes_per_launch_12B_definition": dom_bytes,
                "frac_12B_definition": round(dom_bytes / (stage_us[dominant] * 1e-6) / 1e9 / peak, 4),
                "byte_copy_note": "the 12 B-per-assignment definition of a plan counts a second 4-byte read "
                                  "of every id by the reroute kernel; with at most 256 experts the histogram "
                                  "kernel leaves a one-byte copy instead, so the plan moves 10 B per "
                                  "assignment (histogram 4 + 1, reroute 1 + 4) and fractions of the 12 B "
                                  "definition can exceed 1; achieved and frac count the bytes the kernel "
                                  "moves" if byte_copy else None,
                "plan_bytes": 12 * A,
                "plan_frac": round(plan_gbs / peak, 4),
                "plan_moved_bytes": plan_moved,
                "plan_frac_moved": round(plan_gbs * plan_moved / (12 * A) / peak, 4),
                # the whole plan against 8 B per assignment: ids read from DRAM once (second pass
                # from L2), outputs written once
                "plan_frac_8B": round(plan_gbs * 8 / 12 / peak, 4),
                "plan_frac_nominal": round(plan_gbs / NOMINAL_HBM_GBS, 4),
                "hbm_kernels": hbm_kernels,
                "note": "peak is a plain read+write copy; a kernel with the same traffic mix can land "
                        "a few percent above it (the full-size parity tests run this launch configuration)"}

    line = {"metric": "topk_assignments_per_s", "value": value, "unit": "assignments/s",
            "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_step,
            "us_per_layer_plan": ms_step * 1e3 / w.batch,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
            "data": "synthetic", "impl": "topoep_b200",
            "config": workload_config(w, nsets, l2_policy),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "assignments/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": k_e2e,
                    "us_per_layer_plan": ms_e2e * 1e3 / k_e2e / w.batch},
            "gpu_launches": m["kernels_per_plan"] * K,
            "repeats": m["plan_spread"]["repeats"],
            "us_per_step": m["plan_spread"],
            "kernel_us": {n: round(stage_us[n], 3) for n in ("hist", "solve", "reroute")},
            "kernel_us_spread": {n: m["stage_spread"][n] for n in ("hist", "solve", "reroute")},
            "launch_floor_us": round(stage_us["floor"], 3),
            "vs_launch_floor": round(ms_step * 1e3 / stage_us["floor"], 2),
            "roofline": roofline}
    if single is not None:
        line["single_plan"] = single
    if dispatch is not None:
        line["dispatch_positions"] = dispatch
    if transfer is not None:
        line["replica_transfer"] = transfer

    if rank == 0 and not args.no_cpu_baseline:
        ncores = os.cpu_count() or 1
        sample_ids = s0["ids_host"][:min(w.batch, max(8, ncores))]
        v, plans, dt = time_oracle(w, sample_ids, args.cpu_seconds)
        line["cpu_baseline"] = {"value": v, "unit": "assignments/s", "cores": 1, "kind": "oracle",
                                "sample": "%d whole plans of the %s shape in %.1f s (host has %d cores)"
                                          % (plans, w.name, dt, ncores)}
        if w.batch > 1 and ncores > 1:
            # the plans of a batch are independent: the same oracle, one plan per host thread
            va, plans_a, dta = time_oracle(w, sample_ids, args.cpu_seconds, threads=ncores)
            line["cpu_baseline_all_cores"] = {
                "value": va, "unit": "assignments/s", "cores": ncores, "kind": "oracle",
                "sample": "%d whole plans of the %s shape in %.1f s, independent plans dealt to "
                          "%d host threads" % (plans_a, w.name, dta, ncores)}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
