#!/usr/bin/env python
"""Benchmark of the PRAC per-layer path on B200: one LLaMA-shaped transformer block.

A step = the whole hot path for one block of synthetic activations: for each of the block's
distinct saved inputs (q/k/v share one, o, up/gate share one, down) fit U, Q, c and compress
Z = X [U|Q]; for each of the 7 linears form dW = (dY^T Z) diag(1,c) [U|Q]^T.
metric = layer-tokens per second = N * (number of linears) / step time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama1b] [--rank 256]
  python bench.py --impl reference ...      # the CPU oracle on a bounded sample
  python bench.py --sharded ...             # every rank holds N / world tokens of every input

Under torchrun (N > 1) every rank runs its own block (data-parallel replicas: independent
micro-batches, no data-path collective); the time is the max over ranks.  With --sharded the
ranks share one batch instead: the Gram matrix of each fit and the middle factor dY^T Z of each
weight gradient are summed over the ranks (NCCL all-reduce), everything else is local.

Besides the headline line the default run reports, under extra keys and within a wall-time
budget: the other workloads and ranks of the sweep, the variant without subspace sharing, the
split of the fit, the lazy-update drift study, and the oracle at full size on the two small
workloads.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_23111_b200 import inputs  # noqa: E402

# DRAM bytes (read + write) of one launch of the roofline kernel, from an ncu capture of that
# workload (dram__bytes_read.sum + dram__bytes_write.sum); None where the kernel has changed since.
ROOFLINE_TRAFFIC = {("llama1b", 256, 32768): 395.3e6}

SPREAD_COMPRESS = os.environ.get("PRAC_BENCH_SPREAD_COMPRESS", "1") != "0"
GRAD_STREAMS = int(os.environ.get("PRAC_GRAD_STREAMS", "4"))

METRIC = "compressed tokens/s per layer (fit+compress+dW)"
UNIT = "layer-tokens/s"
NOMINAL_BF16_TFLOPS = 2250.0        # dense bf16 of the part's data sheet, for context beside the measured peak


# ----------------------------------------------------------------------------- helpers

def workload_label(w, kr, N, shared=True):
    lin = w.linears()
    n_in = len({l.input_id for l in lin}) if shared else len(lin)
    return (f"{w.name} block (N={N}, d={w.d}, ffn={w.ffn}), k=r={kr}, {len(lin)} linears over {n_in} "
            f"{'shared' if shared else 'separate'} inputs, basis refit every step")


def dist_info():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def reduce_max(value: float, world: int, device=None) -> float:
    """Max over ranks of a scalar (all ranks get it); identity when not distributed."""
    if world <= 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float, slack: float = 0.15):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.rows:
            if ts < t0 - (slack - 0.15) or ts > t1 + slack:
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            if slack < 1.0:      # a timed region shorter than the sampling period: take the samples next to it
                return self.summary(t0, t1, slack=1.0)
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm)}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured",
                "how": p.get("how"), "when": p.get("when")}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback",
            "how": "an earlier measurement on this pool", "when": None}


def timed(fn, reps: int):
    """Mean milliseconds of fn over reps back-to-back calls, CUDA events on the current stream."""
    return timed_stats(fn, reps)["mean"]


def timed_stats(fn, reps: int):
    """mean / median / best milliseconds of fn over reps back-to-back calls: one CUDA event after
    every call on the current stream, so the per-call times come from the same run as the mean."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(reps):
        fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    per = [ev[i].elapsed_time(ev[i + 1]) for i in range(reps)]
    return {"mean": ev[0].elapsed_time(ev[reps]) / reps, "median": statistics.median(per), "best": min(per)}


L2_BYTES = 126 * 1000 * 1000
FLUSH_BYTES = 256 << 20
_flush_buf = {}


def timed_stats_flushed(fn, reps: int):
    """As timed_stats, for launches whose operands would otherwise be served from L2: a buffer
    larger than L2 is overwritten before every call, and each call has its own pair of events."""
    dev = torch.cuda.current_device()
    if dev not in _flush_buf:
        _flush_buf[dev] = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    buf = _flush_buf[dev]
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(reps)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(reps)]
    torch.cuda.synchronize()
    for i in range(reps):
        buf.fill_(i & 0xFF)
        e0[i].record()
        fn()
        e1[i].record()
    torch.cuda.synchronize()
    per = [e0[i].elapsed_time(e1[i]) for i in range(reps)]
    return {"mean": sum(per) / reps, "median": statistics.median(per), "best": min(per)}


# ----------------------------------------------------------------------------- the block

class Block:
    """Device-resident synthetic block: distinct inputs, output gradients, bases, outputs.
    shared=False gives every linear its own saved input (no subspace sharing: 7 fits, 7
    compresses, 7 weight gradients)."""

    def __init__(self, w: inputs.Workload, rank: int, N: int, device, seed: int, fused: bool = True,
                 shared: bool = True):
        from paper_2602_23111_b200 import api
        self.api = api
        self.w, self.N, self.k, self.r = w, N, rank, rank
        self.device = device
        self.dtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        self.linears = w.linears()
        if not shared:
            self.linears = [inputs.Linear(l.name, l.d_in, l.d_out, j) for j, l in enumerate(self.linears)]
            fused = False
        ids = sorted({l.input_id for l in self.linears})
        self.X, self.basis, self.Z = {}, {}, {}
        for i in ids:
            d_in = next(l.d_in for l in self.linears if l.input_id == i)
            x = inputs.workload_activation(w, d_in, seed=seed + 10 * i, device=device, N=N, ld=inputs.pad64(d_in))
            self.X[i] = self._store(x)
            self.basis[i] = api.Basis(d_in, self.k, self.r, self.dtype, device=device)
            s = self.k + self.r
            self.Z[i] = torch.empty(N, inputs.pad64(s), dtype=self.dtype, device=device)[:, :s]
        # Linears that read the same input (q/k/v; up/gate) are evaluated in one weight-gradient
        # call over their output gradients side by side, the layout of a fused QKV / gate-up
        # projection: dY_group is N x sum(d_out), dW_group is sum(d_out) x d_in, and each linear's
        # dY / dW is a column / row slice of them.  fused=False gives one call per linear.
        self.groups = []               # lists of linear indices
        for j, l in enumerate(self.linears):
            if fused and self.groups and self.linears[self.groups[-1][0]].input_id == l.input_id:
                self.groups[-1].append(j)
            else:
                self.groups.append([j])
        self.dY, self.dW = [None] * len(self.linears), [None] * len(self.linears)
        self.dYg, self.dWg = [], []
        for grp in self.groups:
            widths = [self.linears[j].d_out for j in grp]
            d_in = self.linears[grp[0]].d_in
            total = sum(widths)
            buf = torch.zeros(N, inputs.pad64(total), dtype=self.dtype, device=device)
            # gradient rows start on 128-byte boundaries too (32 floats): tile stores need 16-byte rows
            wbuf = torch.empty(total, (d_in + 31) // 32 * 32, dtype=torch.float32, device=device)[:, :d_in]
            c0 = 0
            for j, wd in zip(grp, widths):
                g = inputs.make_grad(N, wd, seed=seed + 100 + j, device=device, dtype=w.dtype)
                buf[:, c0:c0 + wd] = g.to(self.dtype)
                self.dY[j] = buf[:, c0:c0 + wd]
                self.dW[j] = wbuf[c0:c0 + wd]
                c0 += wd
            self.dYg.append(buf[:, :total])
            self.dWg.append(wbuf)
        # The fits of the block's distinct inputs are independent: each runs on its own stream
        # with its own workspace, so their many small latency-bound kernels overlap.
        def stream_ws_bytes(i, b):
            need = [b.fit_workspace_bytes(N)] + [b.grad_workspace_bytes(N, g.shape[1])
                                                 for grp, g in zip(self.groups, self.dYg)
                                                 if self.linears[grp[0]].input_id == i]
            return max(need)
        self.fit_ws = {i: torch.empty(stream_ws_bytes(i, b), dtype=torch.uint8, device=device)
                       for i, b in self.basis.items()}
        # (the widest input has the longest chain of dependent kernels: its stream gets priority, so
        # that its next kernel never queues behind the other inputs' work)
        widest = max(self.basis, key=lambda i: self.basis[i].d)
        self.fit_stream = {i: torch.cuda.Stream(device=device, priority=-1 if i == widest else 0) for i in self.basis}
        # the widest input has the longest pipeline: enqueue it first
        self.basis = dict(sorted(self.basis.items(), key=lambda kv: -kv[1].d))
        grad_ws = max(self.basis[self.linears[grp[0]].input_id].grad_workspace_bytes(N, g.shape[1])
                      for grp, g in zip(self.groups, self.dYg))
        self.ws = torch.empty(grad_ws, dtype=torch.uint8, device=device)
        # The weight gradients of different linears are independent too: they alternate between
        # GRAD_STREAMS streams (own workspace each), so the short reduction / stage-2 kernels of one
        # linear fill the SMs that the tail of another linear's stage 1 leaves idle.
        self.grad_ws = [self.ws] + [torch.empty(grad_ws, dtype=torch.uint8, device=device)
                                    for _ in range(GRAD_STREAMS - 1)]
        self.grad_stream = [torch.cuda.Stream(device=device) for _ in range(GRAD_STREAMS)]
        self.draw = 0

    def _store(self, x: torch.Tensor) -> torch.Tensor:
        """fp32 view with padded rows -> storage dtype, same padding."""
        n, m = x.shape
        ld = x.stride(0)
        buf = torch.empty(n, ld, dtype=self.dtype, device=x.device)
        buf[:, :m] = x.to(self.dtype)
        if ld > m:
            buf[:, m:] = 0
        return buf[:, :m]

    def _fan_out(self, body):
        """Runs body(i, basis) for every input on that input's stream, joined on the current one."""
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        for i, b in self.basis.items():
            side = self.fit_stream[i]
            side.wait_event(start)
            with torch.cuda.stream(side):
                body(i, b)
                done = torch.cuda.Event()
                done.record(side)
            main.wait_event(done)

    # the three phases of a step ------------------------------------------------------
    def fit(self):
        self.draw += 1
        self._fan_out(lambda i, b: b.fit(self.X[i], seed=1234 + i, draw_counter=self.draw, ws=self.fit_ws[i]))

    def refresh(self):
        """Warm-started update of every U (two iterations from the current U) plus a new Q: what a
        T_1 refresh of the lazy schedule costs once a basis exists."""
        self.draw += 1

        def body(i, b):
            b.refresh_principal(self.X[i], seed=1234 + i, draw_counter=self.draw, iters=2, ws=self.fit_ws[i])
            b.draw_random(seed=1234 + i, draw_counter=self.draw, ws=self.fit_ws[i])
        self._fan_out(body)

    def compress(self):
        # independent launches, one per input, on the inputs' own streams (as in step()): the
        # CTAs of the next launch take the SMs that the last, partly filled round of tiles of
        # the one before leaves idle
        # (short launches stay on one stream: the event hops would cost more than the tails)
        if not SPREAD_COMPRESS or self.flops()["compress"] < 1e11:
            for i, b in self.basis.items():
                b.compress(self.X[i], out=self.Z[i])
            return
        self._fan_out(lambda i, b: b.compress(self.X[i], out=self.Z[i]))

    def grad(self):
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        for side in self.grad_stream:
            side.wait_event(start)
        for j, (grp, dY, dW) in enumerate(zip(self.groups, self.dYg, self.dWg)):
            i = self.linears[grp[0]].input_id
            with torch.cuda.stream(self.grad_stream[j % GRAD_STREAMS]):
                self.basis[i].weight_grad(dY, self.Z[i], out=dW, ws=self.grad_ws[j % GRAD_STREAMS])
        for side in self.grad_stream:
            done = torch.cuda.Event()
            done.record(side)
            main.wait_event(done)

    def step(self, host=None):
        """The whole path for the block.  Each distinct input is its own pipeline on its own
        stream: fit -> compress -> the weight gradients of the linears that read it; an input
        whose fit is done does not wait for the slowest fit of the block."""
        self.draw += 1

        def body(i, b):
            if host is not None:      # end-to-end mode: this pipeline's input arrives from pinned host memory
                self.X[i].copy_(host["X"][i], non_blocking=True)
            b.fit(self.X[i], seed=1234 + i, draw_counter=self.draw, ws=self.fit_ws[i])
            b.compress(self.X[i], out=self.Z[i])
            for j, (grp, dY, dW) in enumerate(zip(self.groups, self.dYg, self.dWg)):
                if self.linears[grp[0]].input_id == i:
                    if host is not None:
                        dY.copy_(host["dY"][j], non_blocking=True)
                    # the fit is over on this stream: its workspace serves the gradients
                    b.weight_grad(dY, self.Z[i], out=dW, ws=self.fit_ws[i])
                    if host is not None:  # ... and the result goes back to the host
                        host["dW"][j].copy_(dW, non_blocking=True)
        self._fan_out(body)

    # algorithmic work ------------------------------------------------------------------
    def flops(self):
        s, N = self.k + self.r, self.N
        ids = {l.input_id: l.d_in for l in self.linears}
        comp = sum(2.0 * N * d * s for d in ids.values())
        dw1 = sum(2.0 * N * l.d_out * s for l in self.linears)
        dw2 = sum(2.0 * l.d_out * s * l.d_in for l in self.linears)
        gram = sum(2.0 * N * d * d for d in ids.values())
        return {"compress": comp, "dw1": dw1, "dw2": dw2, "gram": gram}

    def bytes_in(self):
        e = 2 if self.dtype == torch.bfloat16 else 4
        return sum(x.shape[0] * x.shape[1] * e for x in self.X.values()) + \
            sum(g.shape[0] * g.shape[1] * e for g in self.dYg)

    def bytes_out(self):
        return sum(w.numel() * 4 for w in self.dWg)

    def statuses(self):
        return [b.status() for b in self.basis.values()]


def roofline_of_compress(blk: Block, peaks, reps: int):
    """The roofline object of one workload: its widest compress (one launch of the K-major
    tensor-core kernel per call), scored against the roof its arithmetic intensity puts it under."""
    w, N, s = blk.w, blk.N, blk.k + blk.r
    big = max(blk.basis, key=lambda i: blk.basis[i].d)
    d = blk.basis[big].d
    esz = 2 if w.dtype == "bf16" else 4
    fl = 2.0 * N * d * s
    by = float(esz) * (N * d + N * s + d * s)
    call = lambda: blk.basis[big].compress(blk.X[big], out=blk.Z[big])
    if by > 1.25 * L2_BYTES:
        st = timed_stats(call, reps)
        l2 = f"operands of a launch ({by / 1e6:.0f} MB) exceed L2 ({L2_BYTES / 1e6:.0f} MB); back-to-back launches, no flush"
    else:
        st = timed_stats_flushed(call, reps)
        l2 = (f"operands of a launch ({by / 1e6:.0f} MB) would stay in L2 ({L2_BYTES / 1e6:.0f} MB): "
              f"{FLUSH_BYTES >> 20} MiB written between launches, each launch timed by its own pair of events")
    ms = st["mean"]
    tf = fl / (ms * 1e-3) / 1e12
    gbs = by / (ms * 1e-3) / 1e9
    ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    if w.dtype == "bf16" and fl / by >= ridge:
        bound, unit, peak, ach = "tensor", "TFLOP/s", peaks["bf16_tflops"], tf
        src = f"{peaks['source']} burst bf16 (the kernel is timed alone)"
    else:
        bound, unit, peak, ach = "hbm", "GB/s", peaks["hbm_gbs"], gbs
        src = f"{peaks['source']} HBM copy bandwidth"
    kind = "gemm_tc_kernel (K-major, bf16 out)" if w.dtype == "bf16" else "gemm_simt_kernel (fp32 FMA)"
    out = {"bound": bound,
           "kernel": f"{kind}: Z = X [U|Q] for the widest input (N={N}, d={d}, s={s}); one launch per prac_compress call",
           "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak, "peak_source": src,
           "arithmetic_intensity": fl / by, "ridge": ridge, "tflops": tf, "gbs": gbs,
           "traffic": ROOFLINE_TRAFFIC.get((w.name, blk.k, N)),
           "launch_ms": ms, "launch_ms_median": st["median"], "launch_ms_best": st["best"],
           "flops_per_launch": fl, "algorithmic_bytes_per_launch": by, "l2": l2}
    if bound == "tensor":
        out["frac_of_nominal_dense_bf16"] = tf / NOMINAL_BF16_TFLOPS
    return out, big, ms


def steady_state(blk: Block, comp_ms, grad_ms, fit_ms, peaks):
    fl = blk.flops()
    hot_ms = comp_ms + grad_ms
    hot_flops = fl["compress"] + fl["dw1"] + fl["dw2"]
    tf = hot_flops / (hot_ms * 1e-3) / 1e12
    return {"note": "compress + weight-grad only (basis reused, as between refreshes)",
            "ms": hot_ms, "layer_tokens_per_s": blk.N * len(blk.linears) / (hot_ms * 1e-3), "tflops": tf,
            "frac_of_bf16_peak": tf / peaks["bf16_tflops"],
            "frac_of_bf16_peak_sustained": tf / peaks["bf16_tflops_sustained"],
            "frac_of_nominal_dense_bf16": tf / NOMINAL_BF16_TFLOPS,
            "amortised_ms_T100": hot_ms + fit_ms / 100, "amortised_ms_T500": hot_ms + fit_ms / 500}


def quick_config(w, kr, N, device, peaks, steps=5, warmup=3, shared=True):
    """step / fit / compress / dW of one more workload, with its own roofline object."""
    from paper_2602_23111_b200 import api
    blk = Block(w, kr, N, device, seed=7, shared=shared)
    for _ in range(warmup):
        blk.step()
    if any(s != api.PRAC_OK for s in blk.statuses()):
        raise RuntimeError(f"device status after warm-up of {w.name}: {blk.statuses()}")
    st = timed_stats(blk.step, steps)
    fit = timed_stats(blk.fit, 3)
    warm = timed_stats(blk.refresh, 3)
    comp = timed_stats(blk.compress, steps)
    grad = timed_stats(blk.grad, steps)
    roof, _, _ = roofline_of_compress(blk, peaks, steps)
    n_lin = len(blk.linears)
    out = {"workload": workload_label(w, kr, N, shared), "dtype": w.dtype,
           "ms_per_step": st["mean"], "ms_per_step_median": st["median"], "ms_per_step_best": st["best"],
           "value": N * n_lin / (st["mean"] * 1e-3), "unit": UNIT,
           "phases_ms": {"fit_per_refresh": fit["mean"], "warm_refresh": warm["mean"], "compress": comp["mean"],
                         "weight_grad": grad["mean"]},
           "steady_state": steady_state(blk, comp["mean"], grad["mean"], fit["mean"], peaks) if w.dtype == "bf16" else
           {"ms": comp["mean"] + grad["mean"], "note": "fp32 FMA path: launch-latency bound, not scored on a roofline"},
           "roofline": roof, "device_status": blk.statuses()}
    del blk
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- fit split

def fit_split(w, kr, N, d, device):
    """Where one fit of a d-wide input goes: Gram matrix / the q subspace iterations / the last
    orthonormalisation + Rayleigh-Ritz step / the random draw with its projections and QR.  The
    iteration's share comes from fits with 1 and with q iterations on the same Gram matrix."""
    from paper_2602_23111_b200 import api
    dtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    x = inputs.workload_activation(w, d, seed=3, device=device, N=N, ld=inputs.pad64(d))
    X = torch.zeros(N, inputs.pad64(d), dtype=dtype, device=device)
    X[:, :d] = x.to(dtype)
    X = X[:, :d]
    del x
    b = api.Basis(d, kr, kr, dtype, device=device)
    b1 = api.Basis(d, kr, kr, dtype, iters=1, device=device)
    ws = torch.empty(b.fit_workspace_bytes(N), dtype=torch.uint8, device=device)
    b.fit(X, seed=1, draw_counter=0, ws=ws)
    C = b.gram(X, ws=ws)
    q = b.fit_report(N, ws)["iterations"]
    t_all = timed_stats(lambda: b.fit(X, seed=1, draw_counter=1, ws=ws), 5)
    t_gram = timed(lambda: b.gram(X, ws=ws), 5)
    t_q = timed(lambda: b.fit_principal_gram(C, seed=1, draw_counter=1, ws=ws), 5)
    t_1 = timed(lambda: b1.fit_principal_gram(C, seed=1, draw_counter=1, ws=ws), 5)
    b.fit_principal(X, seed=1, draw_counter=1, ws=ws)
    t_draw = timed(lambda: b.draw_random(seed=1, draw_counter=1, ws=ws), 5)
    rep = b.fit_report(N, ws)
    b.refresh_principal(X, seed=1, draw_counter=2, iters=2, ws=ws)
    rep_warm = b.fit_report(N, ws)
    t_warm = timed(lambda: (b.refresh_principal(X, seed=1, draw_counter=2, iters=2, ws=ws),
                            b.draw_random(seed=1, draw_counter=2, ws=ws)), 5)
    per_iter = (t_q - t_1) / max(q - 1, 1)
    out = {"input": f"N={N}, d={d}, k=r={kr}", "fit_ms": t_all["mean"], "fit_ms_median": t_all["median"],
           "fit_ms_best": t_all["best"], "gram_ms": t_gram, "iterations_ms": per_iter * q, "per_iteration_ms": per_iter,
           "iterations": q, "orthonormalise_and_rayleigh_ritz_ms": t_1 - per_iter, "draw_project_qr_ms": t_draw,
           "warm_refresh_ms": t_warm, "panel_cols": rep["panel_cols"], "eig_size": rep["eig_size"],
           "jacobi_sweeps": rep["jacobi_sweeps"], "jacobi_sweeps_warm_refresh": rep_warm["jacobi_sweeps"],
           "status": b.status()}
    del b, b1, ws, X, C
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- lazy-update drift study

def lazy_update_study(device, hot_ms, fit_ms, warm_ms):
    """Algorithm 1's lazy update on a slowly rotating planted spectrum: X_t = A diag(s) V_t^T with
    V_t = V_0 exp(t * delta * K) (K a fixed skew-symmetric generator of unit spectral norm), so the
    exact top-k right singular subspace at step t is span(V_t[:, :k]) in closed form.  For each
    refresh interval T the basis is fitted cold at t = 0 and refreshed (cold again, or warm-started
    from the previous U) at multiples of T; reported: the projector distance ||U U^T - V_k V_k^T||_F
    and the captured energy ||X U||^2 / ||X V_k||^2 right after a refresh and at the end of an interval
    (staleness T - 1), next to the amortised step time of the headline workload at that T."""
    from paper_2602_23111_b200 import api
    N, d, k, r = 4096, 512, 64, 64
    delta = 2e-4                       # radians of rotation per training step
    g = torch.Generator(device=device).manual_seed(77)
    A, _ = torch.linalg.qr(torch.randn(N, d, generator=g, device=device, dtype=torch.float64))
    V0, _ = torch.linalg.qr(torch.randn(d, d, generator=g, device=device, dtype=torch.float64))
    Kg = torch.randn(d, d, generator=g, device=device, dtype=torch.float64)
    Kg = Kg - Kg.T
    Kg = Kg / torch.linalg.matrix_norm(Kg, ord=2)
    s = torch.full((d,), 0.05, device=device, dtype=torch.float64)
    s[:k] = 0.2 * torch.linspace(2.0, 1.0, k, device=device, dtype=torch.float64)

    def data(t):
        Vt = V0 @ torch.linalg.matrix_exp((t * delta) * Kg)
        X = ((A * s[None, :]) @ Vt.T) * math.sqrt(N)
        return X.to(torch.float32), Vt[:, :k]       # fp32 storage: rounding X to bf16 would itself move the
        #                                             subspace by 3e-3, more than what is being measured

    def quality(b, X, Vk):
        U = b.get()[0].double()
        ra = U - Vk @ (Vk.T @ U)
        rb = Vk - U @ (U.T @ Vk)
        dist = math.sqrt(float((ra * ra).sum() + (rb * rb).sum()))
        Xd = X.double()
        return dist, float(((Xd @ U) ** 2).sum() / ((Xd @ Vk) ** 2).sum())

    rows = []
    for T in (1, 10, 100, 500):
        for mode in ("cold", "warm"):
            b = api.Basis(d, k, r, torch.float32, device=device)
            ws = torch.empty(b.fit_workspace_bytes(N), dtype=torch.uint8, device=device)
            X, Vk = data(0)
            b.fit(X, seed=5, draw_counter=0, ws=ws)
            sweeps = []
            stale_d, stale_e, fresh_d = 0.0, 1.0, 0.0
            for n_ref in range(1, 4):            # three refresh intervals
                t_end = n_ref * T - 1            # last step served by the basis of the previous refresh
                Xe, Vke = data(t_end)
                de, ee = quality(b, Xe, Vke)
                stale_d, stale_e = max(stale_d, de), min(stale_e, ee)
                Xr, Vkr = data(n_ref * T)
                if mode == "cold":
                    b.fit(Xr, seed=5, draw_counter=n_ref * T, ws=ws)
                else:
                    b.refresh_principal(Xr, seed=5, draw_counter=n_ref * T, iters=2, ws=ws)
                    b.draw_random(seed=5, draw_counter=n_ref * T, ws=ws)
                sweeps.append(b.fit_report(N, ws)["jacobi_sweeps"])
                fresh_d = max(fresh_d, quality(b, Xr, Vkr)[0])
            refresh_ms = fit_ms if mode == "cold" else warm_ms
            rows.append({"T": T, "refresh": mode, "projector_distance_after_refresh": fresh_d,
                         "projector_distance_at_staleness_T_minus_1": stale_d,
                         "captured_energy_at_staleness_T_minus_1": stale_e, "jacobi_sweeps": sweeps,
                         "amortised_ms_per_step_headline_workload": hot_ms + refresh_ms / T,
                         "status": b.status()})
            del b, ws
    return {"input": f"planted gap 4, fp32 storage, N={N}, d={d}, k=r={k}, subspace rotating {delta} rad per step "
                     f"(exact subspace known in closed form)", "rows": rows,
            "note": "warm = two iterations started from [previous U | fresh Gaussian columns]; amortised time = "
                    "compress + weight-grad of the headline workload + its refresh cost / T"}


# ----------------------------------------------------------------------------- CPU oracle arm

def oracle_sample_step(w: inputs.Workload, rank: int, n_tokens: int, seed: int = 0):
    """One pass of the oracle over the attention-input group (one input, q/k/v linears) on a
    token sample.  Returns (seconds, layer-tokens processed)."""
    import numpy as np
    from oracle import prac_oracle as orc
    d = w.d
    lin = [l for l in w.linears() if l.input_id == 0]
    X = inputs.workload_activation(w, d, seed=seed, N=n_tokens).numpy().astype(np.float64)
    dYs = [inputs.make_grad(n_tokens, l.d_out, seed=seed + 100 + j, dtype=w.dtype).numpy().astype(np.float64)
           for j, l in enumerate(lin)]
    t0 = time.perf_counter()
    U, Q, c = orc.fit_basis(X, rank, rank, seed=1234, draw_counter=1)
    Z = orc.compress(X, U, Q)
    for dY in dYs:
        orc.weight_grad(dY, Z, U, Q, c)
    return time.perf_counter() - t0, n_tokens * len(lin)


def oracle_full_block(w: inputs.Workload, rank: int):
    """The oracle over a whole block at full size (every distinct input fitted and compressed, every
    linear's gradient), as the GPU step does it.  Returns (seconds, layer-tokens)."""
    import numpy as np
    from oracle import prac_oracle as orc
    lin = w.linears()
    ids = sorted({l.input_id for l in lin})
    Xs = {i: inputs.workload_activation(w, next(l.d_in for l in lin if l.input_id == i), seed=10 * i,
                                        N=w.N).numpy().astype(np.float64) for i in ids}
    dYs = [inputs.make_grad(w.N, l.d_out, seed=100 + j, dtype=w.dtype).numpy().astype(np.float64)
           for j, l in enumerate(lin)]
    t0 = time.perf_counter()
    fitted = {}
    for i in ids:
        U, Q, c = orc.fit_basis(Xs[i], rank, rank, seed=1234 + i, draw_counter=1)
        fitted[i] = (U, Q, c, orc.compress(Xs[i], U, Q))
    for l, dY in zip(lin, dYs):
        U, Q, c, Z = fitted[l.input_id]
        orc.weight_grad(dY, Z, U, Q, c)
    return time.perf_counter() - t0, w.N * len(lin)


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(w: inputs.Workload, rank: int, n_tokens: int, passes: int = 3):
    sec, units = 0.0, 0
    for _ in range(passes):
        s_, u_ = oracle_sample_step(w, rank, n_tokens)
        sec += s_
        units += u_
    return {"value": units / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{w.name}: attention-input group (d={w.d}, q/k/v), k=r={rank}, {n_tokens} of {w.N} tokens, "
                      f"{passes} passes of fit+compress+3 dW in float64 numpy, {sec:.2f} s; the fit's "
                      f"eigendecomposition does not shrink with the sample, so the full-size rate is higher by "
                      f"up to N / sample"}


def cpu_baseline_full_size():
    """The oracle on the two workloads small enough to run at full size (the single fp32 layer and
    the LLaMA-130M block)."""
    rows = []
    for name in ("single_f32", "llama130m"):
        w = inputs.WORKLOADS[name]
        kr = w.ranks[len(w.ranks) // 2]
        sec, units = oracle_full_block(w, kr)
        rows.append({"workload": workload_label(w, kr, w.N), "value": units / sec, "unit": UNIT, "seconds": sec,
                     "cores": blas_threads(), "kind": "oracle", "sample": "the whole block at full size, one pass"})
    return rows


def run_reference(args, w, rank_kr):
    rank, world, _ = dist_info()
    if rank != 0:
        return
    n_tok = max(256, w.N // 4)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(w, rank_kr, n_tok)
    tot_s, tot_u = 0.0, 0
    steps = max(1, min(args.steps, 5))
    for _ in range(steps):
        s, u = oracle_sample_step(w, rank_kr, n_tok)
        tot_s += s
        tot_u += u
    value = tot_u / tot_s
    sample = (f"{w.name}: attention-input group (d={w.d}, q/k/v), k=r={rank_kr}, {n_tok} of {w.N} tokens per step, "
              f"float64 numpy oracle")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * tot_s / steps,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": workload_label(w, rank_kr, w.N), "sample": sample},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def fit_timeline(blk, path):
    """Kernel timeline of the block's fits (one per distinct input, each on its own stream), from
    torch's profiler: per stream the span, the time its kernels ran, the time between them, and the
    kernels that took longest with their individual durations.  Shows how the chains interfere; the
    durations are under a profiler and are not bench values."""
    import collections
    from torch.profiler import ProfilerActivity, profile
    for _ in range(2):
        blk.fit()
    torch.cuda.synchronize()
    with profile(activities=[ProfilerActivity.CUDA]) as prof:
        blk.fit()
        blk.fit()
        torch.cuda.synchronize()
    tmp = path + ".trace.json"
    prof.export_chrome_trace(tmp)
    with open(tmp) as f:
        events = json.load(f)["traceEvents"]
    os.remove(tmp)
    ks = sorted((e["ts"], e["dur"], e["args"].get("stream"), e["name"]) for e in events if e.get("cat") == "kernel")
    ks = ks[len(ks) // 2:]                       # the second of the two profiled phases
    t0 = ks[0][0]
    streams = collections.defaultdict(list)
    for ts, dur, st, name in ks:
        streams[st].append((ts - t0, dur, name.replace("prac::(anonymous namespace)::", "").replace("void ", "")[:44]))
    lines = [f"fit phase of {blk.w.name}, k=r={blk.k}, N={blk.N}: {len(ks)} kernels on {len(streams)} streams, "
             f"span {max(ts + d for ts, d, _, _ in ks) - t0:.0f} us"]
    for st, lst in streams.items():
        busy = sum(d for _, d, _ in lst)
        gaps = sum(lst[i][0] - (lst[i - 1][0] + lst[i - 1][1]) for i in range(1, len(lst)))
        lines.append(f"stream {st}: {len(lst)} kernels, first start {lst[0][0]:.0f} us, end {lst[-1][0] + lst[-1][1]:.0f} us, "
                     f"kernels ran {busy:.0f} us, between kernels {gaps:.0f} us")
        agg = collections.OrderedDict()
        for _, d, n in lst:
            a = agg.setdefault(n, [0.0, []])
            a[0] += d
            a[1].append(round(d))
        for n, (tot, each) in sorted(agg.items(), key=lambda kv: -kv[1][0])[:6]:
            lines.append(f"    {tot:8.0f} us  n={len(each):3d}  {n:46s} {each[:10]}")
    with open(path, "w") as f:
        f.write("\n".join(lines) + "\n")
    print("\n".join(lines), file=sys.stderr)


# ----------------------------------------------------------------------------- token-sharded mode

def sharded_bytes_per_step(w, kr, world):
    """Bytes one rank puts through collectives per step: one Gram matrix per distinct input, one
    middle factor dY^T Z per group of linears sharing an input (nothing when alone)."""
    if world <= 1:
        return 0
    lin = w.linears()
    ids = {l.input_id: l.d_in for l in lin}
    gram = sum(4 * d * d for d in ids.values())
    mid = sum(4 * l.d_out * 2 * kr for l in lin)
    return gram + mid


def run_sharded(args, w, kr):
    """One batch of N tokens spread over the ranks: every rank fits on the all-reduced Gram matrix
    of its token slice, compresses its slice, and forms the weight gradients from the all-reduced
    middle factor dY^T Z."""
    rank, world, local = dist_info()
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2602_23111_b200 import api
    from paper_2602_23111_b200.sharded import ShardedCompressor, shard_rows
    N = args.tokens if args.tokens > 0 else w.N
    b0, b1 = shard_rows(N, world, rank)
    n_loc = b1 - b0
    blk = Block(w, kr, n_loc, device, seed=1000 * rank)     # this rank's slice of every input
    comps = {i: ShardedCompressor(b) for i, b in blk.basis.items()}
    Wm = max(args.warmup, 3)
    K = max(args.steps, 1)
    draw = [0]

    def step():
        draw[0] += 1
        for i, sc in comps.items():
            sc.fit(blk.X[i], seed=1234 + i, draw_counter=draw[0], ws=blk.fit_ws[i])
            sc.compress(blk.X[i], out=blk.Z[i])
            for grp, dY, dW in zip(blk.groups, blk.dYg, blk.dWg):
                if blk.linears[grp[0]].input_id == i:
                    sc.weight_grad(dY, blk.Z[i], out=dW, ws=blk.fit_ws[i])

    for _ in range(Wm):
        step()
    st = blk.statuses()
    if any(s_ != api.PRAC_OK for s_ in st):
        raise SystemExit(f"device status after warm-up: {st}")
    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3)
    for sc in comps.values():
        sc.bytes_reduced = 0
    launches0 = api.kernel_launches()
    barrier(world)
    torch.cuda.synchronize()
    t0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(K):
        step()
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    t1 = time.time()
    ms_step = reduce_max(e0.elapsed_time(e1) / K, world, device)
    launches = api.kernel_launches() - launches0
    reduced = sum(sc.bytes_reduced for sc in comps.values()) // K
    clocks = sampler.summary(t0, t1) if sampler else None
    if sampler:
        sampler.stop()
    if rank == 0:
        n_lin = len(blk.linears)
        out = {"metric": METRIC, "value": N * n_lin / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
               "warmup": Wm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong",
               "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
               "config": {"workload": workload_label(w, kr, N), "tokens": N, "tokens_per_rank": n_loc,
                          "linears": n_lin, "parallelism": f"token-sharded x{world}",
                          "l2": "inputs exceed L2; no flush"},
               "bytes_reduced_per_step": int(reduced), "bytes_reduced_expected": sharded_bytes_per_step(w, kr, world),
               "clocks": clocks, "gpu_launches": int(launches), "device_status": blk.statuses()}
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama1b", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--rank", type=int, default=0, help="k = r (0: the workload's middle value)")
    ap.add_argument("--tokens", type=int, default=0, help="override N (profiling on a smaller case)")
    ap.add_argument("--separate-linears", action="store_true",
                    help="one weight-gradient call per linear instead of one per group of linears sharing an input")
    ap.add_argument("--sharded", action="store_true", help="one batch spread over the ranks (token shards)")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-forward", action="store_true", help="skip the forward-linear and consumer timings")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-sweep", action="store_true", help="skip the other workloads / ranks and the studies")
    ap.add_argument("--sweep-seconds", type=float, default=60.0, help="wall-time budget of the extra sections")
    ap.add_argument("--fit-timeline", metavar="PATH", default="",
                    help="instead of the bench: write a per-stream summary of the kernel timeline of the block's "
                         "concurrent fits (torch profiler; for analysis, not a timing) to PATH")
    args = ap.parse_args()
    w = inputs.WORKLOADS[args.workload]
    kr = args.rank if args.rank > 0 else w.ranks[len(w.ranks) // 2]
    if args.impl == "reference":
        run_reference(args, w, kr)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    if args.sharded:
        run_sharded(args, w, kr)
        return

    rank, world, local = dist_info()
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2602_23111_b200 import api

    N = args.tokens if args.tokens > 0 else w.N
    W = max(args.warmup, 3)
    K = max(args.steps, 1)
    blk = Block(w, kr, N, device, seed=1000 * rank, fused=not args.separate_linears)
    n_lin = len(blk.linears)

    for _ in range(W):
        blk.step()
    st = blk.statuses()
    if any(s != api.PRAC_OK for s in st):
        raise SystemExit(f"device status after warm-up: {st}")
    if args.fit_timeline:
        fit_timeline(blk, args.fit_timeline)
        return

    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3)

    # ---- device-resident timing: exactly K steps, barrier + synchronize on both sides; one event
    # per step inside the region gives the median and the best step beside the mean
    launches0 = api.kernel_launches()
    barrier(world)
    torch.cuda.synchronize()
    t_mark0 = time.time()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    ev[0].record()
    for i in range(K):
        blk.step()
        ev[i + 1].record()
    torch.cuda.synchronize()
    barrier(world)
    launches = api.kernel_launches() - launches0
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(K)]
    ms_step = reduce_max(ev[0].elapsed_time(ev[K]) / K, world, device)

    # ---- per-phase and per-kernel timings (outside the headline region, same inputs)
    peaks = load_peaks()
    reps = max(3, min(K, 10))
    fit_st = timed_stats(blk.fit, max(3, reps // 2))
    refresh_st = timed_stats(blk.refresh, max(3, reps // 2))
    comp_st = timed_stats(blk.compress, reps)
    grad_st = timed_stats(blk.grad, reps)
    fit_ms, refresh_ms, comp_ms, grad_ms = fit_st["mean"], refresh_st["mean"], comp_st["mean"], grad_st["mean"]
    # roofline kernel: the tensor-core GEMM kernel, timed where one API call is exactly one launch
    # of it (prac_compress of the widest input).  The weight-gradient call of the widest linear
    # (three launches: dY^T Z, ordered reduction, M' P^T) is timed beside it as a whole.
    roof, comp_big, comp_call_ms = roofline_of_compress(blk, peaks, reps)
    big = max(range(len(blk.groups)), key=lambda g: blk.dYg[g].shape[1])
    big_dout = blk.dYg[big].shape[1]
    lb = blk.linears[blk.groups[big][0]]
    bb = blk.basis[lb.input_id]
    dw_call_ms = timed(lambda: bb.weight_grad(blk.dYg[big], blk.Z[lb.input_id], out=blk.dWg[big], ws=blk.ws), reps)
    s = 2 * kr
    dw1_flops = 2.0 * N * big_dout * s
    roof["weight_grad_call"] = {"d_out": big_dout, "linears": len(blk.groups[big]), "ms": dw_call_ms, "launches": 3,
                                "tflops_stage1": dw1_flops / (dw_call_ms * 1e-3) / 1e12,
                                "tflops_all_stages": (dw1_flops + 2.0 * big_dout * s * lb.d_in) / (dw_call_ms * 1e-3) / 1e12}
    # forward pass of the first linear of every input (Algorithm 2): Y = X W^T alone, Y and Z from
    # one launch, against compress alone: what the compressed copy costs when X is read once
    fwd = None
    if w.dtype == "bf16" and not args.skip_forward:
        fwd = {"linear_only_ms": 0.0, "linear_with_z_ms": 0.0, "compress_ms": 0.0}
        for i, b in blk.basis.items():
            l0 = next(l for l in blk.linears if l.input_id == i)
            Wt = torch.zeros(l0.d_out, inputs.pad64(l0.d_in), dtype=blk.dtype, device=device)
            Wt[:, :l0.d_in] = inputs.make_grad(l0.d_out, l0.d_in, seed=7 + i, device=device, dtype=w.dtype) * 0.02
            Wt = Wt[:, :l0.d_in]
            Y = torch.empty(N, inputs.pad64(l0.d_out), dtype=blk.dtype, device=device)[:, :l0.d_out]
            b.linear_forward(blk.X[i], Wt, out_y=Y, want_z=False)
            b.linear_forward(blk.X[i], Wt, out_y=Y, out_z=blk.Z[i])
            fwd["linear_only_ms"] += timed(lambda: b.linear_forward(blk.X[i], Wt, out_y=Y, want_z=False), reps)
            fwd["linear_with_z_ms"] += timed(lambda: b.linear_forward(blk.X[i], Wt, out_y=Y, out_z=blk.Z[i]), reps)
            fwd["compress_ms"] += timed(lambda: b.compress(blk.X[i], out=blk.Z[i]), reps)
            del Wt, Y
        fwd["marginal_ms_of_z"] = fwd["linear_with_z_ms"] - fwd["linear_only_ms"]
        fwd["note"] = ("sum over the block's distinct inputs, first linear of each; one launch of "
                       "prac_linear_forward writes Y and Z, reading X once")
    # Section 5.1's non-linear consumer: backward of the MLP's SiLU on its rebuilt input (the gate
    # projection's output, N x ffn, rank 0.2 n + 0.2 n), the rebuilt tile consumed in tensor memory
    actb = None
    if w.dtype == "bf16" and not args.skip_forward:
        dff = w.ffn
        ka = int(0.2 * dff)
        ba = api.Basis(dff, ka, ka, blk.dtype)
        qa, _ = torch.linalg.qr(torch.randn(dff, 2 * ka, device=device, dtype=torch.float32,
                                            generator=torch.Generator(device=device).manual_seed(5)))
        ba.set(qa[:, :ka].contiguous(), qa[:, ka:].contiguous(), (dff - ka) / ka)
        Za = torch.empty(N, inputs.pad64(2 * ka), dtype=blk.dtype, device=device)[:, :2 * ka]
        Za.copy_(inputs.make_grad(N, 2 * ka, seed=11, device=device, dtype=w.dtype))
        dYa = torch.zeros(N, inputs.pad64(dff), dtype=blk.dtype, device=device)[:, :dff]
        dYa.copy_(inputs.make_grad(N, dff, seed=12, device=device, dtype=w.dtype))
        dXa = torch.empty(N, inputs.pad64(dff), dtype=blk.dtype, device=device)[:, :dff]
        ba.activation_backward(Za, dYa, "silu", out=dXa)
        act_st = timed_stats(lambda: ba.activation_backward(Za, dYa, "silu", out=dXa), reps)
        act_ms = act_st["mean"]
        act_flops = 2.0 * N * dff * 2 * ka
        act_bytes = 2.0 * (N * 2 * ka + 2 * N * dff + dff * 2 * ka)
        actb = {"op": f"dX = dY * silu'(Z [U|cQ]^T), N={N}, d={dff}, k=r={ka}", "ms": act_ms, "ms_best": act_st["best"],
                "tflops": act_flops / (act_ms * 1e-3) / 1e12, "gbs": act_bytes / (act_ms * 1e-3) / 1e9,
                "frac_of_bf16_peak": act_flops / (act_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                "unfused_extra_bytes": 2.0 * 4 * N * dff,
                "note": "one launch; the rebuilt input (N x d fp32) is never written or re-read"}
        del ba, Za, dYa, dXa
    # and the block's pre-attention RMSNorm (N x d, rank 0.2 n + 0.2 n): two passes over the rebuilt input
    rmsb = None
    if w.dtype == "bf16" and not args.skip_forward and w.d > 128:
        dn = w.d
        kn = int(0.2 * dn)
        bn_ = api.Basis(dn, kn, kn, blk.dtype)
        qn, _ = torch.linalg.qr(torch.randn(dn, 2 * kn, device=device, dtype=torch.float32,
                                            generator=torch.Generator(device=device).manual_seed(6)))
        bn_.set(qn[:, :kn].contiguous(), qn[:, kn:].contiguous(), (dn - kn) / kn)
        Zn = torch.empty(N, inputs.pad64(2 * kn), dtype=blk.dtype, device=device)[:, :2 * kn]
        Zn.copy_(inputs.make_grad(N, 2 * kn, seed=13, device=device, dtype=w.dtype))
        dYn = torch.zeros(N, inputs.pad64(dn), dtype=blk.dtype, device=device)[:, :dn]
        dYn.copy_(inputs.make_grad(N, dn, seed=14, device=device, dtype=w.dtype))
        dXn = torch.empty(N, inputs.pad64(dn), dtype=blk.dtype, device=device)[:, :dn]
        rstd = torch.rand(N, device=device, dtype=torch.float32) + 0.5
        gain = torch.ones(dn, device=device, dtype=torch.float32)
        wsn = torch.empty(api.lib.prac_rmsnorm_workspace_bytes(ctypes.byref(bn_.params), N),
                          dtype=torch.uint8, device=device)
        bn_.rmsnorm_backward(Zn, dYn, rstd, gain, out=dXn, ws=wsn)
        rms_st = timed_stats(lambda: bn_.rmsnorm_backward(Zn, dYn, rstd, gain, out=dXn, ws=wsn), reps)
        rms_ms = rms_st["mean"]
        rms_flops = 2 * 2.0 * N * dn * 2 * kn
        rms_bytes = 2.0 * (2 * N * 2 * kn + 3 * N * dn)
        rmsb = {"op": f"RMSNorm backward on the rebuilt input, N={N}, d={dn}, k=r={kn}", "ms": rms_ms,
                "ms_best": rms_st["best"], "launches": 3,
                "tflops": rms_flops / (rms_ms * 1e-3) / 1e12, "gbs": rms_bytes / (rms_ms * 1e-3) / 1e9,
                "hbm_frac": rms_bytes / (rms_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                "note": "two GEMM passes (Z read twice, dY twice, dX written once) + the reductions between them"}
        del bn_, Zn, dYn, dXn, wsn
    # the same compress with the layout a framework hands over when the width is not a multiple of 8
    # (contiguous rows, e.g. 5461 bf16 = 10922 bytes): rows off the 16-byte grid, which the library
    # fetches by TMA as classes of rows with the same offset from that grid
    unpadded = None
    comp_d = blk.basis[comp_big].d
    if w.dtype == "bf16" and not args.skip_forward and comp_d % 8 != 0:
        Xc = blk.X[comp_big].contiguous()
        assert Xc.stride(0) == comp_d
        Zc = torch.empty_like(blk.Z[comp_big])
        blk.basis[comp_big].compress(Xc, out=Zc)
        Zp = blk.basis[comp_big].compress(blk.X[comp_big], out=blk.Z[comp_big])
        differing = float((Zc != Zp).float().mean())
        max_rel = float(((Zc.float() - Zp.float()).abs() / (Zp.float().abs() + 1e-3 * float(Zp.float().abs().max()))).max())
        un_ms = timed(lambda: blk.basis[comp_big].compress(Xc, out=Zc), reps)
        unpadded = {"unpadded_compress_ms": un_ms, "padded_compress_ms": comp_call_ms, "ratio": un_ms / comp_call_ms,
                    "fraction_of_elements_differing_from_padded": differing, "max_rel_diff_vs_padded": max_rel,
                    "difference": "fp32 summation order only (k runs shifted by up to 7 inside each class)",
                    "note": f"Z = X [U|Q], N={N}, d={comp_d}: leading dimension {comp_d} (row pitch {2 * comp_d} bytes) "
                            f"against rows padded to {inputs.pad64(comp_d)}"}
        del Xc, Zc
    clocks = sampler.summary(t_mark0, time.time()) if sampler else None

    # ---- end to end: host buffers in, host result out, through the same calls
    e2e = None
    if not args.skip_e2e:
        hX = {i: x.cpu().pin_memory() for i, x in blk.X.items()}
        hY = [g.cpu().pin_memory() for g in blk.dYg]
        hW = [torch.empty_like(wg, device="cpu").pin_memory() for wg in blk.dWg]
        host = {"X": hX, "dY": hY, "dW": hW}

        def e2e_step():
            # host -> device copies of every input and device -> host copies of every gradient are
            # inside the step, each on the stream of the pipeline that consumes / produces it
            blk.step(host=host)

        e2e_step()
        ke = max(2, min(K, 5))
        barrier(world)
        e2e_ms = reduce_max(timed(e2e_step, ke), world, device)
        e2e = {"value": world * N * n_lin / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": blk.bytes_in(), "d2h_bytes_per_step": blk.bytes_out()}
        del hX, hY, hW, host
    if sampler:
        sampler.stop()

    st = blk.statuses()
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    steady = steady_state(blk, comp_ms, grad_ms, fit_ms, peaks)
    out = {
        "metric": METRIC, "value": world * N * n_lin / (ms_step * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
        "data": "synthetic",
        "ms_per_step_median": statistics.median(per_step), "ms_per_step_best": min(per_step),
        "config": {"workload": workload_label(w, kr, N), "tokens": N, "linears": n_lin,
                   "grad_calls": f"{len(blk.groups)} (linears sharing an input are one call over their dY side by side)",
                   "l2": "inputs (2.2 GB per block) exceed L2; no flush",
                   "layout": "rows of X, dY, Z and dW padded to 128-byte multiples", "parallelism": f"replicas x{world}"},
        "phases_ms": {"fit_per_refresh": fit_ms, "warm_refresh": refresh_ms, "compress": comp_ms, "weight_grad": grad_ms,
                      "median": {"fit_per_refresh": fit_st["median"], "warm_refresh": refresh_st["median"],
                                 "compress": comp_st["median"], "weight_grad": grad_st["median"]},
                      "best": {"fit_per_refresh": fit_st["best"], "warm_refresh": refresh_st["best"],
                               "compress": comp_st["best"], "weight_grad": grad_st["best"]}},
        "steady_state": steady,
        "peaks": {"bf16_tflops_burst": peaks["bf16_tflops"], "bf16_tflops_sustained": peaks["bf16_tflops_sustained"],
                  "hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"], "how": peaks["how"], "when": peaks["when"],
                  "nominal_dense_bf16_tflops": NOMINAL_BF16_TFLOPS,
                  "note": "fractions named frac / frac_of_bf16_peak divide by the measured burst figure; the "
                          "fraction of the data-sheet dense bf16 peak is given beside them"},
        "roofline": roof, "unpadded_layout": unpadded,
        "forward_with_compress": fwd, "activation_backward": actb, "rmsnorm_backward": rmsb, "clocks": clocks,
        "e2e": e2e, "gpu_launches": int(launches), "device_status": st,
    }
    del blk
    torch.cuda.empty_cache()

    # ---- extra sections, each inside the wall-time budget; a section that does not fit is named in `skipped_sections`
    if not args.skip_sweep and world == 1 and args.tokens == 0:
        t_budget = time.time() + args.sweep_seconds
        skipped = []

        def within(label, est_s):
            if time.time() + est_s <= t_budget:
                return True
            skipped.append(label)
            return False

        if within("fit_split", 3):
            out["fit_split"] = [fit_split(w, kr, N, d_, device) for d_ in sorted({w.d, w.ffn} - {0})]
        sweep = []
        plan = [(args.workload, r_) for r_ in w.ranks if r_ != kr]
        plan += [(nm, inputs.WORKLOADS[nm].ranks[len(inputs.WORKLOADS[nm].ranks) // 2])
                 for nm in ("llama130m", "llama350m", "llama7b", "single_f32") if nm != args.workload]
        for nm, r_ in plan:
            if within(f"sweep:{nm}:k{r_}", 6):
                wk = inputs.WORKLOADS[nm]
                sweep.append(quick_config(wk, r_, wk.N, device, peaks))
        out["sweep"] = sweep
        if within("unshared", 6):
            out["unshared_inputs"] = quick_config(w, kr, N, device, peaks, shared=False)
        if within("lazy_update", 8):
            out["lazy_update"] = lazy_update_study(device, steady["ms"], fit_ms, refresh_ms)
        out["skipped_sections"] = skipped
    if not args.skip_cpu:
        out["cpu_baseline"] = cpu_baseline(w, kr, max(256, w.N // 4))
        if not args.skip_sweep and world == 1:
            out["cpu_baseline_full_size"] = cpu_baseline_full_size()
    print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
