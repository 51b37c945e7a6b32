#!/usr/bin/env python
"""Benchmark of the PRAC per-layer path on B200: one LLaMA-shaped transformer block.

A step = the whole hot path for one block of synthetic activations: for each of the block's
distinct saved inputs (q/k/v share one, o, up/gate share one, down) fit U, Q, c and compress
Z = X [U|Q]; for each of the 7 linears form dW = (dY^T Z) diag(1,c) [U|Q]^T.
metric = layer-tokens per second = N * (number of linears) / step time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama1b] [--rank 256]
  python bench.py --impl reference ...      # the CPU oracle on a bounded sample

Under torchrun (N > 1) every rank runs its own block (data-parallel replicas: independent
micro-batches, no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
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

# DRAM bytes (read + write) of one launch of the roofline kernel, from an ncu capture of this
# workload (see profiles/); None where no capture of the current kernel exists.
ROOFLINE_TRAFFIC = {("llama1b", 256, 32768): 404.9e6}   # profiles/gemm_tc_kernel_llama1b_k256.md

SPREAD_COMPRESS = os.environ.get("PRAC_BENCH_SPREAD_COMPRESS", "1") != "0"
GRAD_STREAMS = int(os.environ.get("PRAC_GRAD_STREAMS", "3"))

METRIC = "compressed tokens/s per layer (fit+compress+dW)"
UNIT = "layer-tokens/s"


# ----------------------------------------------------------------------------- helpers

def workload_label(w, kr, N):
    lin = w.linears()
    n_in = len({l.input_id for l in lin})
    return (f"{w.name} block (N={N}, d={w.d}, ffn={w.ffn}), k=r={kr}, {len(lin)} linears over {n_in} "
            f"shared inputs, basis refit every step")


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

    def mark(self):
        return time.time()

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.rows:
            if ts < t0 or ts > t1 + 0.15:
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
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm)}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- the block

class Block:
    """Device-resident synthetic block: distinct inputs, output gradients, bases, outputs."""

    def __init__(self, w: inputs.Workload, rank: int, N: int, device, seed: int, fused: bool = True):
        from paper_2602_23111_b200 import api
        self.api = api
        self.w, self.N, self.k, self.r = w, N, rank, rank
        self.device = device
        self.dtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        self.linears = w.linears()
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

    # the three phases of a step ------------------------------------------------------
    def fit(self):
        self.draw += 1
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        for i, b in self.basis.items():
            side = self.fit_stream[i]
            side.wait_event(start)
            with torch.cuda.stream(side):
                b.fit(self.X[i], seed=1234 + i, draw_counter=self.draw, ws=self.fit_ws[i])
                done = torch.cuda.Event()
                done.record(side)
            main.wait_event(done)

    def refresh(self):
        """Warm-started update of every U (two iterations from the current U) plus a new Q: what a
        T_1 refresh of the lazy schedule costs once a basis exists."""
        self.draw += 1
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        for i, b in self.basis.items():
            side = self.fit_stream[i]
            side.wait_event(start)
            with torch.cuda.stream(side):
                b.refresh_principal(self.X[i], seed=1234 + i, draw_counter=self.draw, iters=2, ws=self.fit_ws[i])
                b.draw_random(seed=1234 + i, draw_counter=self.draw, ws=self.fit_ws[i])
                done = torch.cuda.Event()
                done.record(side)
            main.wait_event(done)

    def compress(self):
        # independent launches, one per input, on the inputs' own streams (as in step()): the
        # CTAs of the next launch take the SMs that the last, partly filled round of tiles of
        # the one before leaves idle
        # (short launches stay on one stream: the event hops would cost more than the tails)
        if not SPREAD_COMPRESS or self.flops()["compress"] < 1e11:
            for i, b in self.basis.items():
                b.compress(self.X[i], out=self.Z[i])
            return
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        for i, b in self.basis.items():
            side = self.fit_stream[i]
            side.wait_event(start)
            with torch.cuda.stream(side):
                b.compress(self.X[i], out=self.Z[i])
                done = torch.cuda.Event()
                done.record(side)
            main.wait_event(done)

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
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        for i, b in self.basis.items():
            side = self.fit_stream[i]
            side.wait_event(start)
            with torch.cuda.stream(side):
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
                done = torch.cuda.Event()
                done.record(side)
            main.wait_event(done)

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


def timed(fn, reps: int):
    """Mean milliseconds of fn over reps back-to-back calls, CUDA events on the current stream."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


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
                      f"{passes} passes of fit+compress+3 dW in float64 numpy, {sec:.2f} s"}


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
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-forward", action="store_true", help="skip the forward-linear timings")
    ap.add_argument("--skip-cpu", action="store_true")
    args = ap.parse_args()
    w = inputs.WORKLOADS[args.workload]
    kr = args.rank if args.rank > 0 else w.ranks[len(w.ranks) // 2]
    if args.impl == "reference":
        run_reference(args, w, kr)
        return

    rank, world, local = dist_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
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
    st = [b.status() for b in blk.basis.values()]
    if any(s != api.PRAC_OK for s in st):
        raise SystemExit(f"device status after warm-up: {st}")

    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3)

    # ---- device-resident timing: exactly K steps, barrier + synchronize on both sides
    launches0 = api.kernel_launches()
    barrier(world)
    torch.cuda.synchronize()
    t_mark0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(K):
        blk.step()
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    t_mark1 = time.time()
    launches = api.kernel_launches() - launches0
    ms_step = reduce_max(e0.elapsed_time(e1) / K, world, device)

    # ---- per-phase and per-kernel timings (outside the headline region, same inputs)
    reps = max(3, min(K, 10))
    fit_ms = timed(blk.fit, max(2, reps // 2))
    refresh_ms = timed(blk.refresh, max(2, reps // 2))
    comp_ms = timed(blk.compress, reps)
    grad_ms = timed(blk.grad, reps)
    # roofline kernel: the tensor-core GEMM kernel, timed where one API call is exactly one launch
    # of it (prac_compress of the widest input).  The weight-gradient call of the widest linear
    # (three launches: dY^T Z, ordered reduction, M' P^T) is timed beside it as a whole.
    big = max(range(len(blk.groups)), key=lambda g: blk.dYg[g].shape[1])
    big_dout = blk.dYg[big].shape[1]
    lb = blk.linears[blk.groups[big][0]]
    bb = blk.basis[lb.input_id]
    dw_call_ms = timed(lambda: bb.weight_grad(blk.dYg[big], blk.Z[lb.input_id], out=blk.dWg[big], ws=blk.ws), reps)
    comp_big = max(blk.basis, key=lambda i: blk.basis[i].d)
    comp_call_ms = timed(lambda: blk.basis[comp_big].compress(blk.X[comp_big], out=blk.Z[comp_big]), reps)
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
        act_ms = timed(lambda: ba.activation_backward(Za, dYa, "silu", out=dXa), reps)
        act_flops = 2.0 * N * dff * 2 * ka
        act_bytes = 2.0 * (N * 2 * ka + 2 * N * dff + dff * 2 * ka)
        actb = {"op": f"dX = dY * silu'(Z [U|cQ]^T), N={N}, d={dff}, k=r={ka}", "ms": act_ms,
                "tflops": act_flops / (act_ms * 1e-3) / 1e12, "gbs": act_bytes / (act_ms * 1e-3) / 1e9,
                "frac_of_bf16_peak": act_flops / (act_ms * 1e-3) / 1e12 / load_peaks()["bf16_tflops"],
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
        wsn = torch.empty(api.lib.prac_rmsnorm_workspace_bytes(__import__("ctypes").byref(bn_.params), N),
                          dtype=torch.uint8, device=device)
        bn_.rmsnorm_backward(Zn, dYn, rstd, gain, out=dXn, ws=wsn)
        rms_ms = timed(lambda: bn_.rmsnorm_backward(Zn, dYn, rstd, gain, out=dXn, ws=wsn), reps)
        rms_flops = 2 * 2.0 * N * dn * 2 * kn
        rms_bytes = 2.0 * (2 * N * 2 * kn + 3 * N * dn)
        rmsb = {"op": f"RMSNorm backward on the rebuilt input, N={N}, d={dn}, k=r={kn}", "ms": rms_ms, "launches": 3,
                "tflops": rms_flops / (rms_ms * 1e-3) / 1e12, "gbs": rms_bytes / (rms_ms * 1e-3) / 1e9,
                "hbm_frac": rms_bytes / (rms_ms * 1e-3) / 1e9 / load_peaks()["hbm_gbs"],
                "note": "two GEMM passes (Z read twice, dY twice, dX written once) + the reductions between them"}
        del bn_, Zn, dYn, dXn, wsn
    # the same compress with the layout a framework hands over when the width is not a multiple of 8
    # (contiguous rows, e.g. 5461 bf16 = 10922 bytes): rows off the 16-byte grid, fetched with plain
    # loads inside the same tensor-core kernel instead of TMA
    unpadded = None
    comp_d = blk.basis[comp_big].d
    if w.dtype == "bf16" and not args.skip_forward and comp_d % 8 != 0:
        Xc = blk.X[comp_big].contiguous()
        assert Xc.stride(0) == comp_d
        Zc = torch.empty_like(blk.Z[comp_big])
        blk.basis[comp_big].compress(Xc, out=Zc)
        same = bool(torch.equal(Zc, blk.basis[comp_big].compress(blk.X[comp_big], out=blk.Z[comp_big])))
        un_ms = timed(lambda: blk.basis[comp_big].compress(Xc, out=Zc), reps)
        unpadded = {"unpadded_compress_ms": un_ms, "padded_compress_ms": comp_call_ms, "ratio": un_ms / comp_call_ms,
                    "bit_identical_to_padded": same,
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
    if sampler:
        sampler.stop()

    st = [b.status() for b in blk.basis.values()]
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    fl = blk.flops()
    s = 2 * kr
    dw1_flops = 2.0 * N * big_dout * s
    dw_call_flops = dw1_flops + 2.0 * big_dout * s * lb.d_in
    peak_tf = peaks["bf16_tflops"]
    comp_d = blk.basis[comp_big].d
    comp_flops = 2.0 * N * comp_d * s
    achieved = comp_flops / (comp_call_ms * 1e-3) / 1e12
    esz = 2 if w.dtype == "bf16" else 4
    comp_bytes = float(esz) * (N * comp_d + N * s + comp_d * s)
    # the launch is scored against the roof it sits under: tensor cores when its arithmetic
    # intensity is above the ridge of the measured peaks, HBM otherwise
    if w.dtype == "bf16" and comp_flops / comp_bytes >= peak_tf * 1e12 / (peaks["hbm_gbs"] * 1e9):
        roof_bound, roof_unit, roof_peak, roof_achieved = "tensor", "TFLOP/s", peak_tf, achieved
        roof_source = f"{peaks['source']} burst bf16 (the kernel is timed alone)"
    else:
        roof_bound, roof_unit, roof_peak = "hbm", "GB/s", peaks["hbm_gbs"]
        roof_achieved = comp_bytes / (comp_call_ms * 1e-3) / 1e9
        roof_source = f"{peaks['source']} HBM copy bandwidth"
    hot_ms = comp_ms + grad_ms
    hot_flops = fl["compress"] + fl["dw1"] + fl["dw2"]
    out = {
        "metric": METRIC, "value": world * N * n_lin / (ms_step * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": workload_label(w, kr, N), "tokens": N, "linears": n_lin,
                   "grad_calls": f"{len(blk.groups)} (linears sharing an input are one call over their dY side by side)",
                   "l2": "inputs (2.2 GB per block) exceed L2; no flush", "layout": "rows of X, dY, Z and dW padded to 128-byte multiples", "parallelism": f"replicas x{world}"},
        "phases_ms": {"fit_per_refresh": fit_ms, "warm_refresh": refresh_ms, "compress": comp_ms,
                      "weight_grad": grad_ms},
        "steady_state": {
            "note": "compress + weight-grad only (basis reused, as between refreshes)",
            "ms": hot_ms, "layer_tokens_per_s": N * n_lin / (hot_ms * 1e-3),
            "tflops": hot_flops / (hot_ms * 1e-3) / 1e12,
            "frac_of_bf16_peak": hot_flops / (hot_ms * 1e-3) / 1e12 / peak_tf,
            "amortised_ms_T100": hot_ms + fit_ms / 100, "amortised_ms_T500": hot_ms + fit_ms / 500},
        "roofline": {"bound": roof_bound,
                     "kernel": f"gemm_tc_kernel (K-major, {'bf16' if w.dtype == 'bf16' else 'f32'} out): Z = X [U|Q] for the "
                               f"widest input (N={N}, d={comp_d}, s={s}); one launch per prac_compress call",
                     "achieved": roof_achieved, "peak": roof_peak, "unit": roof_unit, "frac": roof_achieved / roof_peak,
                     "peak_source": roof_source, "arithmetic_intensity": comp_flops / comp_bytes,
                     "ridge": peak_tf * 1e12 / (peaks["hbm_gbs"] * 1e9),
                     "tflops": achieved, "gbs": comp_bytes / (comp_call_ms * 1e-3) / 1e9,
                     "traffic": ROOFLINE_TRAFFIC.get((w.name, kr, N)),
                     "launch_ms": comp_call_ms, "flops_per_launch": comp_flops,
                     "algorithmic_bytes_per_launch": comp_bytes,
                     "weight_grad_call": {"d_out": big_dout, "linears": len(blk.groups[big]), "ms": dw_call_ms,
                                          "launches": 3,
                                          "tflops_stage1": dw1_flops / (dw_call_ms * 1e-3) / 1e12,
                                          "tflops_all_stages": dw_call_flops / (dw_call_ms * 1e-3) / 1e12}},
        "unpadded_layout": unpadded, "forward_with_compress": fwd, "activation_backward": actb, "rmsnorm_backward": rmsb, "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "device_status": st,
    }
    if not args.skip_cpu:
        out["cpu_baseline"] = cpu_baseline(w, kr, max(256, w.N // 4))
    print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
