"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

Holds no arithmetic of the method itself: only activation-shaped matrices with a chosen
singular spectrum, outlier channels and noise, Gaussian output gradients, and the table
of workload shapes.  Both the CUDA path and the CPU oracle consume the tensors made
here (the oracle after widening to float64), so rounding of the *inputs* to the storage
type is never a source of disagreement.

Recipe (stand-in for LLaMA activations, whose spectrum has a few dominant singular
values and a slowly decaying tail, Section 4.1):
    X = A diag(sigma) V^T D + eps E
with A (N x d) i.i.d. N(0,1), V a random orthogonal d x d matrix (QR of a Gaussian),
sigma_i = i^-p, D the identity except `n_outliers` channels scaled by `outlier_scale`,
E i.i.d. N(0,1); then rounded to the storage dtype.  dY is i.i.d. N(0,1).
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import torch


@dataclasses.dataclass(frozen=True)
class Linear:
    name: str
    d_in: int
    d_out: int
    input_id: int          # linears with the same id share one saved input (q/k/v; up/gate)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    dtype: str             # "f32" or "bf16" (storage of X, dY, Z)
    N: int
    d: int
    ffn: int
    ranks: tuple           # values of k = r that the workload sweeps
    p: float               # sigma_i = i^-p
    noise: float
    n_outliers: int
    outlier_scale: float

    def linears(self):
        d, f = self.d, self.ffn
        if f == 0:
            return [Linear("proj", d, d, 0)]
        return [Linear("q", d, d, 0), Linear("k", d, d, 0), Linear("v", d, d, 0),
                Linear("o", d, d, 1),
                Linear("up", d, f, 2), Linear("gate", d, f, 2),
                Linear("down", f, d, 3)]


WORKLOADS = {
    "single_f32": Workload("single_f32", "f32", 2048, 512, 0, (16,), 1.0, 1e-3, 0, 1.0),
    "llama130m": Workload("llama130m", "bf16", 32768, 768, 2048, (64,), 0.8, 1e-3, 0, 1.0),
    "llama350m": Workload("llama350m", "bf16", 32768, 1024, 2736, (128,), 0.8, 1e-3, 0, 1.0),
    "llama1b": Workload("llama1b", "bf16", 32768, 2048, 5461, (128, 256, 512), 0.7, 1e-3, 8, 20.0),
    "llama7b": Workload("llama7b", "bf16", 16384, 4096, 11008, (512,), 0.5, 1e-3, 16, 50.0),
}


def pad8(n: int) -> int:
    """Leading dimension that keeps 16-bit rows 16-byte aligned."""
    return (n + 7) // 8 * 8


def pad64(n: int) -> int:
    """Leading dimension that puts every 16-bit row on a 128-byte boundary (the TMA tile
    loads then touch whole 128-byte lines; measurably faster than 16-byte alignment when
    the width is not already a multiple of 64, e.g. 5461)."""
    return (n + 63) // 64 * 64


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def round_to(x: torch.Tensor, dtype: str) -> torch.Tensor:
    """Round an fp32 tensor to the storage dtype's value set, keep it as fp32."""
    if dtype == "bf16":
        return x.to(torch.bfloat16).to(torch.float32)
    return x


def random_orthogonal(d: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    a = torch.randn(d, d, generator=g, device=device, dtype=torch.float32)
    q, r = torch.linalg.qr(a)
    return q * torch.sign(torch.diagonal(r))[None, :]


def make_activation(N: int, d: int, p: float = 1.0, noise: float = 1e-3,
                    n_outliers: int = 0, outlier_scale: float = 1.0, seed: int = 0,
                    device="cpu", dtype: str = "f32", ld: Optional[int] = None) -> torch.Tensor:
    """X (N x d) as fp32 values representable in `dtype`.  If ld > d the result is a view
    into an (N x ld) buffer (zero padding on the right)."""
    g = _gen(seed, device)
    sigma = torch.arange(1, d + 1, device=device, dtype=torch.float32) ** (-p)
    V = random_orthogonal(d, seed + 1, device)
    Vt = (V * sigma[None, :]).t().contiguous()              # diag(sigma) V^T
    if n_outliers > 0:
        perm = torch.randperm(d, generator=_gen(seed + 2, "cpu"))[:n_outliers].to(device)
        Vt[:, perm] *= outlier_scale
    ld = d if ld is None else ld
    out = torch.zeros(N, ld, device=device, dtype=torch.float32)
    rows = 4096
    for i0 in range(0, N, rows):
        n = min(rows, N - i0)
        A = torch.randn(n, d, generator=g, device=device, dtype=torch.float32)
        E = torch.randn(n, d, generator=g, device=device, dtype=torch.float32)
        out[i0:i0 + n, :d] = round_to(A @ Vt + noise * E, dtype)
    return out[:, :d]


def make_planted(N: int, d: int, k: int, gap: float = 4.0, tail: float = 0.05,
                 seed: int = 0, device="cpu", dtype: str = "f32",
                 exact_rank: bool = False) -> torch.Tensor:
    """X = A diag(s) V^T with orthonormal A (N x d, N >= d) and s_1..s_k spread over
    [gap*tail*2, gap*tail] (so s_k / s_{k+1} = gap), tail singular values = `tail`
    (or 0 if exact_rank).  Used where the principal subspace must be well defined."""
    g = _gen(seed, device)
    A, _ = torch.linalg.qr(torch.randn(N, d, generator=g, device=device, dtype=torch.float32))
    V = random_orthogonal(d, seed + 1, device)
    s = torch.full((d,), 0.0 if exact_rank else tail, device=device, dtype=torch.float32)
    s[:k] = gap * tail * torch.linspace(2.0, 1.0, k, device=device)
    X = (A * s[None, :]) @ V.t() * (N ** 0.5)
    return round_to(X, dtype)


def make_grad(N: int, d_out: int, seed: int = 0, device="cpu", dtype: str = "f32",
              ld: Optional[int] = None) -> torch.Tensor:
    g = _gen(seed + 1000, device)
    ld = d_out if ld is None else ld
    out = torch.zeros(N, ld, device=device, dtype=torch.float32)
    rows = 4096
    for i0 in range(0, N, rows):
        n = min(rows, N - i0)
        out[i0:i0 + n, :d_out] = round_to(
            torch.randn(n, d_out, generator=g, device=device, dtype=torch.float32), dtype)
    return out[:, :d_out]


def workload_activation(w: Workload, d: int, seed: int = 0, device="cpu", N: Optional[int] = None,
                        ld: Optional[int] = None) -> torch.Tensor:
    return make_activation(w.N if N is None else N, d, w.p, w.noise, w.n_outliers,
                           w.outlier_scale, seed, device, w.dtype, ld)
