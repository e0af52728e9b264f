#!/usr/bin/env python
"""Benchmark of the ExactOBS / OBQ layer solver on synthetic layers shaped like the paper's workloads.

One "step" is one pass of the whole hot path over one layer, through the C ABI:
  Hessian (2 X X^T) -> dampened inverse -> per-row elimination (prune trace or OBQ) -> global mask ->
  final weights (per configuration; see WORKLOADS).
Prints ONE JSON line.  `value` = eliminated (pruned or quantised) weights per second over the whole job with
inputs resident in HBM; `e2e` = the same with host<->device copies inside the timed region;
`roofline` = the elimination kernel's bytes over its CUDA-event time against the measured HBM copy rate (bound "hbm"):
for the blocked engine the bytes of its own schedule (the triangle once per block of deferred updates; the flops of
the rank-B updates against the TF32 tensor peak are reported beside it), for the streaming engine the triangle bytes
per step; the 8 m^2-per-step model of the step-by-step method is reported in both cases;
`cpu_baseline` = the FP64 oracle on a bounded sample of the same rows on this machine's host cores.

The default workload is C5 (768 x 3072, the largest configuration; it fits one GPU), and the line nests a compact
record of C3 (256 x 2304) under "other_workloads", so that both row lengths the bandwidth target names are measured
by one command.  `--gpus N` without a launcher starts N ranks itself (one process per GPU).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C1..C5] [--engine blocked|streaming] [--impl reference]
  python bench.py --small-case prune,1152,148      (one engine launch on a small seeded layer, for profiler captures)
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import obc_synth  # noqa: E402

METRIC = "eliminated_weights_per_s"
UNIT = "weights/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0        # the "~8 TB/s" the bandwidth target is stated against
FALLBACK_BF16_SUSTAINED_TFLOPS = 1400.0
# DRAM bytes per algorithmic byte of the row engine, from the ncu capture summarised in
# profiles/streaming_engine_d1152_rows148_ncu_full.txt (291.0 GB moved for 603.3 GB of 8 m^2 model bytes); the
# traffic of a full-size launch is scaled from it by the algorithmic bytes (traffic grows with them).
ENGINE_TRAFFIC_PER_ALGORITHMIC_BYTE = 291.0 / 603.3
# The same for the blocked engine, relative to ITS algorithmic bytes (blocked_bytes_flops), per captured row length:
# profiles/blocked_engine_d2304_rows148_ncu_full.txt: 120.04 GB moved for 98.13 GB;
# profiles/blocked_engine_d3072_rows148_ncu_full.txt: 201.79 GB for 147.73 GB.  Other row lengths run other
# configurations of the kernel (threads per row, pending vectors in L2) and have no capture: traffic is null there.
BLOCKED_TRAFFIC_PER_ALGORITHMIC_BYTE = {2304: 120.04 / 98.13, 3072: 201.79 / 147.73}


def model_bytes_full(d: int, first: int | None = None, steps: int | None = None) -> int:
    """Algorithmic bytes of `steps` eliminations starting at active size `first`: read + write of the active
    m x m FP32 block per step = 8 m^2 (the symmetric half actually moved is stated separately)."""
    first = d if first is None else first
    steps = first if steps is None else steps
    m = np.arange(first, first - steps, -1, dtype=np.float64)
    return int((8.0 * m * m).sum())


def pending_stride(m: int) -> int:
    """Floats between two pending update vectors of a row of m slots (the stride obc_engine_plan documents)."""
    return (m + 8 + 31) // 32 * 32 + 8


def blocked_schedule(plan: dict, first: int, steps: int):
    """(m_after_flush, updates_applied) for every pass the blocked engine makes over a row's matrix when `steps`
    eliminations start at active size `first`: it defers min(max_pending, panel_floats // pending_stride(m) + l2_vectors)
    updates, flushes early when the live size reaches the on-chip threshold, and finishes in shared memory below it."""
    ms, panel, maxp = plan["on_chip_below"], plan["panel_floats"], plan["max_pending"]
    out, m0, left = [], first, steps
    if first <= ms:
        return out
    while left > 0 and m0 > ms:
        b = max(1, min(maxp, panel // pending_stride(m0) + plan.get("l2_vectors", 0)))
        nb = min(b, m0 - ms, left)
        left -= nb
        if left <= 0:
            break                      # the last block of a row is never written back
        m0 -= nb
        out.append((m0, nb))
    return out


def blocked_bytes_flops(plan: dict, d: int, first: int | None = None, steps: int | None = None):
    """Bytes and flops one row of the blocked engine has to move / execute: the private lower triangle written once,
    then per pass one read and one write of the compacted triangle (4 bytes per element) and 2 flops per element
    and deferred update."""
    first = d if first is None else first
    steps = first if steps is None else steps
    nbytes = 4.0 * d * (d + 1) / 2 if d > plan["on_chip_below"] else 0.0
    flops = 0.0
    for m1, nb in blocked_schedule(plan, first, steps):
        tri = m1 * (m1 + 1) / 2
        nbytes += 8.0 * tri
        flops += 2.0 * tri * nb
    return nbytes, flops


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return float(j["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def tf32_peak():
    """Dense TF32 tensor peak in TFLOP/s: the measured sustained bf16 GEMM rate (the kernel runs inside a long step)
    times the nominal TF32 : BF16 ratio 1.1 : 2.25."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    ratio = 1.1 / 2.25
    if os.path.exists(p):
        j = json.load(open(p))
        return float(j.get("bf16_tflops_sustained", j["bf16_tflops"])) * ratio, "measured sustained bf16 GEMM x 1.1/2.25 (nominal TF32:BF16)"
    return FALLBACK_BF16_SUSTAINED_TFLOPS * ratio, "fallback sustained bf16 GEMM x 1.1/2.25 (nominal TF32:BF16)"


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs (read-only)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        late = False
        if not self.rows:          # timed region shorter than the sampling period: take the first sample that arrives
            late = True
            for _ in range(30):
                if self.rows:
                    break
                time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for nme, v in zip(names, r[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(nme)
            except Exception:
                pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
               "samples": len(sm)}
        if late:
            out["note"] = "timed region shorter than the 200 ms sampling period: sample taken right after it"
        return out


# ------------------------------------------------------------------------------------------------------------------
class Layer:
    """Device buffers and the stage sequence of one workload, all through the C ABI."""

    def __init__(self, name: str, W: np.ndarray, X: np.ndarray, dev, prec: int, row_begin: int = 0, row_count: int | None = None,
                 group_world: int = 1, engine: str = "blocked"):
        import torch
        import paper_2208_11580_b200 as obc
        self.obc, self.torch, self.name, self.dev, self.prec = obc, torch, name, dev, prec
        self.opts = obc.engine_opts(obc.ENGINE_BLOCKED if engine == "blocked" else obc.ENGINE_STREAMING)
        self.spec = obc_synth.SPECS[name]
        self.R, self.d = W.shape
        self.n = X.shape[1]
        # rows this process eliminates (all of them unless one layer is sharded over several GPUs)
        self.rb, self.rc = row_begin, (W.shape[0] - row_begin if row_count is None else row_count)
        self.group_world = group_world
        R, d = self.R, self.d
        t = torch
        self.W = t.empty(R, d, dtype=t.float32, device=dev)
        self.X = t.empty(d, self.n, dtype=t.float32, device=dev)
        self.H = t.empty(d, d, dtype=t.float32, device=dev)
        self.Hinv = t.empty(d, d, dtype=t.float32, device=dev)
        self.info = t.zeros(1, dtype=t.int32, device=dev)
        self.status = t.zeros(R, dtype=t.int32, device=dev)
        self.order = t.zeros(R, d, dtype=t.int32, device=dev)
        self.loss = t.zeros(R, d, dtype=t.float32, device=dev)
        task = self.spec.task
        self.trace = None
        if task in ("prune", "prune+quant"):
            if self.rc == R:
                self.trace = t.empty(R, d + 1, d, dtype=t.float32, device=dev)
            # (a rank that holds a row range of a sharded layer keeps no weight trace: its final weights come from
            # the forced-order replay, so its memory shrinks with its share of the rows)
        if task != "quant":
            self.ks = [obc_synth.pruned_count(R, d, s) for s in self.spec.sparsities]
            self.counts = [t.zeros(R, dtype=t.int32, device=dev) for _ in self.ks]
            self.masks = [t.zeros(R, d, dtype=t.uint8, device=dev) for _ in self.ks]
            self.What = [t.zeros(R, d, dtype=t.float32, device=dev) for _ in self.ks]
        if task in ("quant", "prune+quant", "compound"):
            self.scale = t.zeros(R, dtype=t.float32, device=dev)
            self.zero = t.zeros(R, dtype=t.float32, device=dev)
            self.Wq = t.zeros(R, d, dtype=t.float32, device=dev)
            self.codes = t.zeros(R, d, dtype=t.int32, device=dev)
        need = max(obc.obc_workspace_bytes(obc.OP_HESSIAN, 0, d, self.n), obc.obc_workspace_bytes(obc.OP_INVERSE, 0, d),
                   obc.obc_workspace_bytes(obc.OP_PRUNE_TRACE, max(1, self.rc), d), obc.obc_workspace_bytes(obc.OP_SELECT, R, d))
        self.ws = t.empty(need, dtype=t.uint8, device=dev)
        self.W.copy_(t.from_numpy(W))
        self.X.copy_(t.from_numpy(X))
        self.engine_ms = []          # (label, CUDA-event ms, launch info) per engine launch since reset_timers()
        self._info = {}
        self._pending = []
        self.eliminated = self.rc * d * (2 if task == "prune+quant" else 1)

    def _timed(self, label, nbytes, fn):
        t = self.torch
        e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        self._pending.append((label, nbytes, e0, e1))

    def step(self):
        """Enqueue one pass of the hot path on the current stream (no synchronisation)."""
        o, R, d, task = self.obc, self.R, self.d, self.spec.task
        self._timed("hessian", 0, lambda: o.obc_hessian(self.X, self.H, prec=self.prec, ws=self.ws))
        self._timed("inverse", 0, lambda: o.obc_hessian_inverse(self.H, obc_synth.DAMP_REL, Hinv=self.Hinv, info=self.info, ws=self.ws))
        full = self.launch_info(with_trace=False)
        if task in ("prune", "prune+quant", "compound"):
            full_t = self.launch_info(with_trace=self.trace is not None)
            self._timed("engine:prune_trace", full_t, lambda: o.obc_prune_trace(self.W, self.Hinv, self.order, self.loss, self.status,
                                                                              w_trace=self.trace, row_begin=self.rb, row_count=self.rc, ws=self.ws, opts=self.opts))
            if self.group_world > 1:   # the one exchange step of a row-sharded layer: traces of all rows to every rank
                self._timed("exchange", 0, self._exchange)
            for i, k in enumerate(self.ks):
                self._timed("select", 0, lambda i=i, k=k: o.obc_select_global_mask(self.loss, self.order, k, self.counts[i], self.masks[i], ws=self.ws))
                if task != "compound":
                    self._timed("apply", 0, lambda i=i: o.obc_prune_apply(self.W, self.Hinv, self.order, self.counts[i], self.What[i], self.status,
                                                                           w_trace=self.trace, trace_steps=d, row_begin=self.rb, row_count=self.rc, ws=self.ws, opts=self.opts))
        if task in ("quant", "prune+quant"):
            self._timed("grid", 0, lambda: o.obc_minmax_grid(self.W, self.spec.bits, self.spec.symmetric, self.scale, self.zero))
            self._timed("engine:quantize", full, lambda: o.obc_quantize(self.W, self.Hinv, self.scale, self.zero, self.spec.bits, self.spec.symmetric,
                                                                        self.Wq, self.codes, self.status, row_begin=self.rb, row_count=self.rc, ws=self.ws, opts=self.opts))
        if task == "compound":
            # replay of counts[r] pruning steps + quantisation of the survivors: again every size d..1 once per row
            self._timed("engine:replay_quantize", full, lambda: o.obc_quantize(
                self.W, self.Hinv, self.scale, self.zero, self.spec.bits, self.spec.symmetric, self.Wq, self.codes, self.status,
                prune_order=self.order, prune_counts=self.counts[0], row_begin=self.rb, row_count=self.rc, ws=self.ws, opts=self.opts))

    def _exchange(self):
        from paper_2208_11580_b200.sharding import gather_traces
        L, P = gather_traces(self.loss[self.rb:self.rb + self.rc], self.order[self.rb:self.rb + self.rc], self.R)
        self.loss.copy_(L)
        self.order.copy_(P)

    def launch_info(self, with_trace: bool):
        """What one engine launch over all rows (every active size d..1 once per row) has to move and compute."""
        R, d = self.rc, self.d
        key = bool(with_trace)
        if key not in self._info:
            plan = self.obc.obc_engine_plan(d, with_trace, R, opts=self.opts)
            info = {"model_bytes": R * model_bytes_full(d), "plan": plan}
            if plan["engine"] == self.obc.ENGINE_BLOCKED:
                b, f = blocked_bytes_flops(plan, d)
                info["own_bytes"], info["flops"] = R * b, R * f
            else:   # streaming: one read + one write of the active lower triangle per step
                m = np.arange(1, d + 1, dtype=np.float64)
                info["own_bytes"], info["flops"] = R * float((4.0 * m * (m + 1)).sum()), R * float((m * (m + 1)).sum())
            self._info[key] = info
        return self._info[key]

    def reset_timers(self):
        self._pending = []

    def collect(self):
        """After a synchronize: CUDA-event milliseconds per stage, summed over the steps since reset_timers()."""
        out = {}
        self.engine_ms = []
        for label, nbytes, e0, e1 in self._pending:
            ms = e0.elapsed_time(e1)
            out[label] = out.get(label, 0.0) + ms
            if label.startswith("engine"):
                self.engine_ms.append((label, ms, nbytes))
        return out

    def results_to_host(self, host):
        """Device->host read of the step's results (final weights / codes / masks) into pinned buffers."""
        task = self.spec.task
        n = 0
        if task != "quant" and task != "compound":
            for i in range(len(self.ks)):
                host["What"][i].copy_(self.What[i], non_blocking=True)
                host["mask"][i].copy_(self.masks[i], non_blocking=True)
                n += self.What[i].numel() * 4 + self.masks[i].numel()
        if task in ("quant", "prune+quant", "compound"):
            host["Wq"].copy_(self.Wq, non_blocking=True)
            host["codes"].copy_(self.codes, non_blocking=True)
            n += self.Wq.numel() * 4 + self.codes.numel() * 4
        return n


def dist_context(args):
    """(rank, world, local_rank); checks that the launcher's world size is the --gpus the caller asked for."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started WORLD_SIZE={world} ranks")
    return rank, world, local


def measure(args, name, steps, warmup, rank, world, dev, with_cpu=True, with_e2e=True):
    """Times `steps` passes of workload `name` after `warmup` untimed ones; returns the result record (rank 0) or
    None (other ranks)."""
    import torch
    import torch.distributed as dist
    import paper_2208_11580_b200 as obc

    local = dev.index
    W, X, spec = obc_synth.make_layer(name)          # every rank builds the same seeded layer
    prec = {"fp32": obc.PREC_FP32, "tf32": obc.PREC_TF32, "bf16x3": obc.PREC_BF16X3}[args.hessian_prec]
    if args.shard_rows and world > 1:
        from paper_2208_11580_b200.sharding import row_range
        rb, rc = row_range(W.shape[0], world, rank)        # ONE layer, its rows split over the GPUs
        layer = Layer(name, W, X, dev, prec, rb, rc, world, engine=args.engine)
    else:
        layer = Layer(name, W, X, dev, prec, engine=args.engine)   # every GPU compresses its own copy of the layer

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        layer.step()
    barrier()
    assert int(layer.info.item()) == 0 and int(layer.status.abs().sum()) == 0, "solver reported a failure status"
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = obc.obc_kernel_launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    layer.reset_timers()
    ev0.record()
    for _ in range(steps):
        layer.step()
    ev1.record()
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    launches = obc.obc_kernel_launches() - launches0
    clocks = sampler.stop() if rank == 0 else None
    stage_sum = {k: v / steps for k, v in layer.collect().items()}     # per-step averages over the timed region
    engine_runs = list(layer.engine_ms)                                  # every engine launch of the timed region
    if world > 1:
        tmax = torch.tensor([total_ms], device=dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        total_ms = float(tmax.item())
    ms_per_step = total_ms / steps
    sharded = args.shard_rows and world > 1
    total_units = layer.R * layer.d * (2 if spec.task == "prune+quant" else 1) * (1 if sharded else world)
    value = total_units / (ms_per_step * 1e-3)

    # ---- end to end: pinned host inputs -> device, hot path, results -> pinned host, every step ---------------------
    e2e = None
    if with_e2e:
        t = torch
        hW, hX = t.from_numpy(W).pin_memory(), t.from_numpy(X).pin_memory()
        host = {"What": [], "mask": []}
        if spec.task not in ("quant", "compound"):
            host["What"] = [t.empty(layer.R, layer.d, dtype=t.float32).pin_memory() for _ in layer.ks]
            host["mask"] = [t.empty(layer.R, layer.d, dtype=t.uint8).pin_memory() for _ in layer.ks]
        if spec.task in ("quant", "prune+quant", "compound"):
            host["Wq"] = t.empty(layer.R, layer.d, dtype=t.float32).pin_memory()
            host["codes"] = t.empty(layer.R, layer.d, dtype=t.int32).pin_memory()
        e2e_steps = max(1, min(steps, 2))
        barrier()
        layer.reset_timers()
        ev0.record()
        d2h = 0
        for _ in range(e2e_steps):
            layer.W.copy_(hW, non_blocking=True)
            layer.X.copy_(hX, non_blocking=True)
            layer.step()
            d2h = layer.results_to_host(host)
        ev1.record()
        barrier()
        e2e_ms = ev0.elapsed_time(ev1)
        if world > 1:
            tmax = torch.tensor([e2e_ms], device=dev)
            dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
            e2e_ms = float(tmax.item())
        e2e = {"value": round(total_units / (e2e_ms / e2e_steps * 1e-3), 1), "unit": UNIT,
               "h2d_bytes_per_step": int(hW.numel() * 4 + hX.numel() * 4), "d2h_bytes_per_step": int(d2h),
               "ms_per_step": round(e2e_ms / e2e_steps, 3), "steps": e2e_steps}
        del hW, hX, host

    if rank != 0:
        return None
    peak, peak_kind = peaks()
    eng_ms = sum(ms for _, ms, _ in engine_runs)
    n_eng = max(1, len(engine_runs))
    own_bytes = sum(i["own_bytes"] for _, _, i in engine_runs)
    model_bytes = sum(i["model_bytes"] for _, _, i in engine_runs)
    flops = sum(i["flops"] for _, _, i in engine_runs)
    plan = engine_runs[0][2]["plan"] if engine_runs else obc.obc_engine_plan(layer.d, False, layer.rc, opts=layer.opts)
    blocked = plan["engine"] == obc.ENGINE_BLOCKED
    sec = eng_ms * 1e-3
    achieved = own_bytes / sec / 1e9 if sec > 0 else 0.0
    model_gbs = model_bytes / sec / 1e9 if sec > 0 else 0.0
    fp32_peak = plan["sm_count"] * 128 * 2 * (clocks.get("sm_max_mhz") or 1965.0) * 1e6 / 1e12   # TFLOP/s, FMA = 2
    hbm = {"achieved": round(achieved, 1), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
           "frac": round(achieved / peak, 4), "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
           "algorithmic_bytes_per_launch": int(own_bytes // n_eng),
           "bytes_model": ("one write of the private lower triangle, then one read + one write of the compacted "
                           "triangle per block of deferred updates" if blocked else
                           "one read + one write of the active lower triangle per step")}
    tflops = flops / sec / 1e12 if sec > 0 else 0.0
    alu = {"achieved": round(tflops, 2), "peak": round(fp32_peak, 1), "peak_kind": "derived: SMs x 128 FP32 lanes x 2 x max SM clock",
           "unit": "TFLOP/s", "frac": round(tflops / fp32_peak, 4), "flops_per_launch": int(flops // n_eng),
           "flops_model": "2 flops per element of the active lower triangle and update"}
    tpeak, tpeak_kind = tf32_peak()
    tensor = {"achieved": round(tflops, 2), "executed": round(3.0 * tflops, 2), "peak": round(tpeak, 1), "peak_kind": tpeak_kind,
              "unit": "TFLOP/s", "frac": round(tflops / tpeak, 4), "frac_executed": round(3.0 * tflops / tpeak, 4),
              "flops_per_launch": int(flops // n_eng),
              "flops_model": "2 flops per element of the active lower triangle and deferred update (rank-B update on the tensor "
                             "cores, TF32 m16n8k8); executed = 3 x that: every FP32 operand is split into two TF32 parts and "
                             "three of the four partial products are formed"}
    if blocked and plan.get("l2_vectors", 0) > 0:
        tensor["note"] = ("rows this long keep %d of their deferred updates per pass in global memory (resident in L2); the rank-B "
                          "update reads their operands from there in the MMA fragment layout" % plan["l2_vectors"])
    # Both engines are reported against HBM.  The streaming engine moves the active triangle once per step.  The blocked
    # engine moves it once per block of deferred updates and applies the block as one rank-B update on the tensor cores;
    # the per-step phase (argmin, pivot column, correction) moves no matrix bytes and is inside the same time.
    main, other = hbm, (tensor if blocked else alu)
    roofline = {"bound": "hbm", "kernel": "blocked_engine_kernel" if blocked else "row_engine_kernel",
                "achieved": main["achieved"], "peak": main["peak"], "peak_kind": main["peak_kind"], "unit": main["unit"],
                "frac": main["frac"],
                "frac_own_schedule": main["frac"],
                "frac_own_schedule_of_nominal_8TBs": main["frac_of_nominal_8TBs"],
                "frac_step_by_step_model": round(model_gbs / peak, 3),
                "frac_step_by_step_model_of_nominal_8TBs": round(model_gbs / NOMINAL_HBM_GBS, 3),
                "traffic": (int(own_bytes / n_eng * BLOCKED_TRAFFIC_PER_ALGORITHMIC_BYTE[layer.d])
                            if layer.d in BLOCKED_TRAFFIC_PER_ALGORITHMIC_BYTE else None) if blocked
                           else int(model_bytes / n_eng * ENGINE_TRAFFIC_PER_ALGORITHMIC_BYTE),
                "traffic_source": (("DRAM bytes, scaled from the d=%d x 148-row ncu capture of this kernel by algorithmic bytes" % layer.d
                                    if layer.d in BLOCKED_TRAFFIC_PER_ALGORITHMIC_BYTE else
                                    "no ncu capture of the kernel configuration this row length runs") if blocked else
                                   "DRAM bytes, scaled from the d=1152 x 148-row ncu capture by algorithmic bytes"),
                "ms_per_launch": round(eng_ms / n_eng, 3), "launches_timed": len(engine_runs),
                "hbm": main, "tensor" if blocked else "alu": other,
                "step_by_step_model": {"bytes_per_launch": int(model_bytes // n_eng),
                                       "GBps_equivalent": round(model_gbs, 1),
                                       "over_hbm_peak": round(model_gbs / peak, 3),
                                       "note": "8 m^2 bytes per elimination step (read + write of the full active block), "
                                               "the figure the step-by-step method has to move; the blocked engine moves "
                                               "about 1/(2B) of it, so this is not a bandwidth claim"},
                "plan": plan}
    if blocked and args.compare_streaming:
        roofline["streaming_engine"] = streaming_reference(layer, peak)
    out = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": steps,
           "warmup": warmup, "ms_per_step": round(ms_per_step, 3), "higher_is_better": True,
           "scaling": "strong" if sharded else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": f"{name}: {spec.note}", "d_row": layer.R, "d_col": layer.d, "n_calib": layer.n,
                      "task": spec.task, "bits": spec.bits, "sparsities": list(spec.sparsities),
                      "hessian_prec": args.hessian_prec, "engine": args.engine, "damp_rel": obc_synth.DAMP_REL,
                      "l2": "per-row inverse-Hessian working set exceeds L2 (inputs larger than L2)"
                            if layer.R * layer.d * layer.d * 2 > 126e6 else "working set fits L2 (small case)",
                      "parallelism": (f"rows of ONE layer split over {world} GPUs, one all-gather of the traces before the global mask"
                                      if sharded else f"rows of one layer per GPU; {world} independent layer(s)")},
           "stage_ms": {k: round(v, 3) for k, v in stage_sum.items()},
           "clocks": clocks, "gpu_launches": int(launches),
           "e2e": e2e, "roofline": roofline}
    if with_cpu:
        out["cpu_baseline"] = cpu_baseline(name, W, layer.Hinv.cpu().numpy(), args.cpu_seconds)
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2208_11580_b200 as obc

    rank, world, local = dist_context(args)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    obc.load_library()
    out = measure(args, args.workload, args.steps, args.warmup, rank, world, dev)
    torch.cuda.empty_cache()
    also = {}
    for name in [w for w in args.also.split(",") if w and w != args.workload]:
        # a compact record of a further workload in the same line (fewer steps; same timing rules)
        rec = measure(args, name, max(3, min(args.steps, 5)), 3, rank, world, dev, with_cpu=False, with_e2e=False)
        torch.cuda.empty_cache()
        if rec is not None:
            r = rec["roofline"]
            also[name] = {"workload": rec["config"]["workload"], "d_row": rec["config"]["d_row"], "d_col": rec["config"]["d_col"],
                          "value": rec["value"], "unit": UNIT, "ms_per_step": rec["ms_per_step"], "steps": rec["steps"],
                          "warmup": rec["warmup"], "stage_ms": rec["stage_ms"], "gpu_launches": rec["gpu_launches"],
                          "clocks": rec["clocks"],
                          "roofline": {k: r[k] for k in ("bound", "kernel", "achieved", "peak", "unit", "frac", "frac_own_schedule",
                                                         "frac_own_schedule_of_nominal_8TBs", "frac_step_by_step_model",
                                                         "ms_per_launch", "plan") if k in r} |
                                      ({"streaming_engine": r["streaming_engine"]} if "streaming_engine" in r else {})}
    if rank == 0:
        if also:
            out["other_workloads"] = also
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def streaming_reference(layer, peak):
    """The step-by-step (streaming) engine on one wave of rows of the same layer, timed alone after the main
    measurement: its achieved bytes per second against the HBM peak, for comparison with the blocked engine."""
    import torch
    obc = layer.obc
    spec, d = layer.spec, layer.d
    rows = min(layer.rc, 148)
    opts = obc.engine_opts(obc.ENGINE_STREAMING)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]

    def call():
        if spec.task == "quant":
            obc.obc_quantize(layer.W, layer.Hinv, layer.scale, layer.zero, spec.bits, spec.symmetric, layer.Wq, layer.codes,
                             layer.status, row_begin=layer.rb, row_count=rows, ws=layer.ws, opts=opts)
        else:
            obc.obc_prune_trace(layer.W, layer.Hinv, layer.order, layer.loss, layer.status, row_begin=layer.rb, row_count=rows,
                                ws=layer.ws, opts=opts)
    call()
    torch.cuda.synchronize()
    ev[0].record(); call(); ev[1].record()
    torch.cuda.synchronize()
    ms = ev[0].elapsed_time(ev[1])
    m = np.arange(1, d + 1, dtype=np.float64)
    tri = rows * float((4.0 * m * (m + 1)).sum())
    model = rows * model_bytes_full(d)
    return {"kernel": "row_engine_kernel", "rows": rows, "ms": round(ms, 3),
            "triangle_GBps": round(tri / (ms * 1e-3) / 1e9, 1), "frac_of_peak": round(tri / (ms * 1e-3) / 1e9 / peak, 4),
            "frac_of_nominal_8TBs": round(tri / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
            "step_by_step_model_GBps": round(model / (ms * 1e-3) / 1e9, 1),
            "note": "bytes = one read + one write of the active lower triangle per step"}


ORACLE_S_PER_UPDATE = 1.5e-9      # one inner update of the oracle on one host core (order of magnitude, for sizing only)


def oracle_sample(d: int, rows_avail: int, cores: int, budget_s: float):
    """(rows, steps) of a bounded oracle run: one row per core at least; when a full row would exceed the budget only
    the first `steps` eliminations of each row are run (those at the largest active sizes)."""
    est_row = ORACLE_S_PER_UPDATE * (2.0 / 3.0) * d ** 3 + 1e-4
    if est_row <= budget_s:
        rows = int(max(1, min(rows_avail, cores * max(1, int(budget_s / est_row)))))
        return rows, d
    rows = int(max(1, min(rows_avail, cores)))
    frac = budget_s / est_row                                  # share of a row's sum of m^2 to cover
    steps = int(max(8, min(d, round(d * (1.0 - (1.0 - frac) ** (1.0 / 3.0))))))
    return rows, steps


def full_row_factor(d: int, steps: int) -> float:
    """sum_{m=1..d} m^2 / sum_{m=d-steps+1..d} m^2: the oracle's work per step is proportional to m^2 (it updates the
    m x m remaining block), so a run of the first `steps` eliminations is scaled to a full row by this factor."""
    m = np.arange(1, d + 1, dtype=np.float64)
    return float((m * m).sum() / (m[d - steps:] ** 2).sum())


def time_oracle(name, W, Hinv, rows, steps):
    import oracle
    spec = obc_synth.SPECS[name]
    Ws = W[:rows]
    kw = {}
    if spec.task == "quant":
        sc, ze, mq = oracle.minmax_grid(Ws, spec.bits, spec.symmetric)
        kw = dict(mode="quant", scale=sc, zero=ze, maxq=mq)
    t0 = time.perf_counter()
    oracle.run_rows(Hinv, Ws, steps=steps, **kw)
    return time.perf_counter() - t0


def sample_text(name, rows, total_rows, steps, d, dt):
    part = "" if steps == d else (f", first {steps} of {d} eliminations per row, scaled to full rows by the oracle's m^2 "
                                  f"work per step (x{full_row_factor(d, steps):.2f})")
    return f"{rows} of {total_rows} rows of {name}{part}, elimination loop only (Hessian/inverse excluded), {dt:.1f} s"


def cpu_baseline(name, W, Hinv32, budget_s):
    """FP64 oracle on a bounded sample of the same workload (elimination loop), on this machine's host cores: all
    cores (OpenMP over rows), and one row on one core."""
    import oracle
    cores = oracle.threads()
    d = W.shape[1]
    Hinv = Hinv32.astype(np.float64)
    rows, steps = oracle_sample(d, W.shape[0], cores, budget_s)
    dt = time_oracle(name, W, Hinv, rows, steps)
    value = rows * d / (dt * full_row_factor(d, steps))
    r1, s1 = oracle_sample(d, 1, 1, max(2.0, budget_s / 3.0))
    dt1 = time_oracle(name, W, Hinv, 1, s1)
    return {"value": round(value, 1), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": sample_text(name, rows, W.shape[0], steps, d, dt) + ", OpenMP over rows", "seconds": round(dt, 2),
            "one_core": {"value": round(d / (dt1 * full_row_factor(d, s1)), 1), "unit": UNIT, "cores": 1,
                         "sample": sample_text(name, 1, W.shape[0], s1, d, dt1), "seconds": round(dt1, 2)}}


def run_reference(args):
    """The FP64 oracle as it stands, timed on host cores: each step = the elimination loop on a bounded sample of the
    workload (rows, and for long rows the first eliminations of each), sized so that the whole run ends within minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    name = args.workload
    W, X, spec = obc_synth.make_layer(name)
    d = W.shape[1]
    H = oracle.hessian(X)
    Hinv, info = oracle.inverse(H, obc_synth.DAMP_REL)
    assert info == 0
    cores = oracle.threads()
    per_step_budget = max(2.0, 90.0 / max(1, args.steps + args.warmup))
    rows, steps = oracle_sample(d, W.shape[0], cores, per_step_budget)
    for _ in range(args.warmup):
        time_oracle(name, W, Hinv, rows, steps)
    dts = [time_oracle(name, W, Hinv, rows, steps) for _ in range(args.steps)]
    dt = float(np.mean(dts))
    value = rows * d / (dt * full_row_factor(d, steps))
    sample = sample_text(name, rows, W.shape[0], steps, d, dt) + " per step, OpenMP over rows"
    out = {"impl": "reference", "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"{name}: {spec.note}", "d_row": W.shape[0], "d_col": d, "n_calib": X.shape[1],
                      "task": spec.task, "bits": spec.bits, "sparsities": list(spec.sparsities),
                      "hessian_prec": "f64", "engine": "oracle", "damp_rel": obc_synth.DAMP_REL},
           "cpu_baseline": {"value": round(value, 1), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": round(value, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def run_small_case(args):
    """One engine launch (or the Hessian kernel) on a small seeded layer, for profiler captures: sized by the caller so
    that the private inverse-Hessian copies exceed L2 but stay at a few GB.  --small-case MODE,D,ROWS[,N] with MODE in
    prune | quant | nm24 | hessian."""
    import torch
    import paper_2208_11580_b200 as obc
    parts = args.small_case.split(",")
    mode, d, R = parts[0], int(parts[1]), int(parts[2])
    n = int(parts[3]) if len(parts) > 3 else 2 * d
    eng = {"blocked": obc.ENGINE_BLOCKED, "streaming": obc.ENGINE_STREAMING}[args.engine]
    opts = obc.engine_opts(eng, args.threads, args.pending)
    W, X = obc_synth.make_small(R, d, n, 4242, "relu")
    Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
    H = torch.empty(d, d, dtype=torch.float32, device="cuda")
    prec = {"fp32": obc.PREC_FP32, "tf32": obc.PREC_TF32, "bf16x3": obc.PREC_BF16X3}[args.hessian_prec]

    def timed(fn):
        times = []
        for _ in range(args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        return times
    if mode == "hessian":
        ws = torch.empty(obc.obc_workspace_bytes(obc.OP_HESSIAN, 0, d, n), dtype=torch.uint8, device="cuda")
        times = timed(lambda: obc.obc_hessian(Xd, H, prec=prec, ws=ws))
        print(json.dumps({"small_case": args.small_case, "prec": args.hessian_prec, "ms": [round(t, 3) for t in times],
                          "dense_equiv_TFLOPs": round(2.0 * d * d * n / (min(times) * 1e-3) / 1e12, 1)}))
        return
    obc.obc_hessian(Xd, H, prec=prec)
    Hinv, info = obc.obc_hessian_inverse(H, obc_synth.DAMP_REL)
    order = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    loss = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    status = torch.zeros(R, dtype=torch.int32, device="cuda")
    ws = torch.empty(obc.obc_workspace_bytes(obc.OP_PRUNE_TRACE, R, d), dtype=torch.uint8, device="cuda")
    Wq = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    if mode == "quant":
        scale = torch.zeros(R, dtype=torch.float32, device="cuda")
        zero = torch.zeros(R, dtype=torch.float32, device="cuda")
        obc.obc_minmax_grid(Wd, 4, False, scale, zero)
        codes = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    if mode == "prune":
        fn = lambda: obc.obc_prune_trace(Wd, Hinv, order, loss, status, ws=ws, opts=opts)
    elif mode == "nm24":
        fn = lambda: obc.obc_prune_nm(Wd, Hinv, 2, 4, Wq, status, order=order, loss=loss, ws=ws, opts=opts)
    elif mode == "quant":
        fn = lambda: obc.obc_quantize(Wd, Hinv, scale, zero, 4, False, Wq, codes, status, ws=ws, opts=opts)
    else:
        raise SystemExit(f"unknown small-case mode {mode}")
    times = timed(fn)
    assert int(info.item()) == 0 and int(status.abs().sum()) == 0
    plan = obc.obc_engine_plan(d, False, R, opts=opts)
    rec = {"small_case": args.small_case, "engine": args.engine, "threads": args.threads, "pending": args.pending,
           "ms": [round(t, 3) for t in times], "plan": plan,
           "step_by_step_model_GBps": round(R * model_bytes_full(d) / (min(times) * 1e-3) / 1e9, 1),
           "private_copies_MB": round(min(R, 148) * d * d * 2 / 1e6, 1)}
    if plan["engine"] == obc.ENGINE_BLOCKED:
        b, f = blocked_bytes_flops(plan, d)
        rec["own_schedule_GB"] = round(R * b / 1e9, 2)
        rec["own_schedule_GBps"] = round(R * b / (min(times) * 1e-3) / 1e9, 1)
    print(json.dumps(rec))


def dry_run_ranks(args):
    """Launcher check without a GPU: every rank joins a gloo group and rank 0 prints the ranks that arrived."""
    import torch
    import torch.distributed as dist
    rank, world, local = dist_context(args)
    if world > 1:
        dist.init_process_group("gloo")
    got = torch.zeros(world, dtype=torch.int64)
    got[rank] = rank + 1
    if world > 1:
        dist.all_reduce(got)
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "ranks": [int(x) - 1 for x in got], "local_rank0": local,
                          "workload": args.workload, "shard_rows": bool(args.shard_rows)}))
    if world > 1:
        dist.destroy_process_group()


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def relaunch_with_ranks(args) -> int:
    """--gpus N > 1 without a launcher: start N ranks of this script (one process per GPU) through torch's launcher
    on this node and return its exit code.  NCCL's version / topology lines are left on so that the rank count shows."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "VERSION")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C5", choices=sorted(obc_synth.SPECS))
    ap.add_argument("--also", default=None,
                    help="comma-separated further workloads whose compact records are nested in the line "
                         "(default: C3 when the workload is C5 on one GPU, else none)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--hessian-prec", default="bf16x3", choices=["fp32", "tf32", "bf16x3"])
    ap.add_argument("--cpu-seconds", type=float, default=18.0)
    ap.add_argument("--engine", default="blocked", choices=["blocked", "streaming"],
                    help="row elimination engine: deferred block updates (default) or one pass per step")
    ap.add_argument("--threads", type=int, default=0, help="--small-case: threads per row of the blocked engine (0 = from d_col)")
    ap.add_argument("--pending", type=int, default=0, help="--small-case: limit on deferred updates (0 = as many as fit)")
    ap.add_argument("--shard-rows", action="store_true",
                    help="with --gpus N > 1: split the rows of ONE layer over the GPUs (strong scaling) instead of one layer per GPU")
    ap.add_argument("--no-compare-streaming", dest="compare_streaming", action="store_false",
                    help="skip the extra timing of the streaming engine on one wave of rows")
    ap.add_argument("--small-case", default=None, help="MODE,D,ROWS[,N]: one small engine / Hessian launch for profiler captures")
    ap.add_argument("--dry-run-ranks", action="store_true", help="launcher check on CPU: ranks join a gloo group, nothing is timed")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be >= 1")
    if args.also is None:
        args.also = "C3" if (args.workload == "C5" and args.gpus == 1 and args.impl == "ours") else ""
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not args.small_case:
        sys.exit(relaunch_with_ranks(args))
    if args.small_case:
        run_small_case(args)
    elif args.dry_run_ranks:
        dry_run_ranks(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
