"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU
oracle on the same seeded inputs.  Tolerances: Philox words bit-exact; projector distance
<= 1e-3 on gapped spectra; Z and dW relative Frobenius error <= 1e-2 (bf16 storage, fp32
accumulation) and <= 1e-5 (fp32 storage)."""
import math

import numpy as np
import pytest
import torch

from oracle import prac_oracle as orc
from paper_2602_23111_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = {torch.bfloat16: 1e-2, torch.float32: 1e-5}


@pytest.fixture(scope="module")
def api():
    from paper_2602_23111_b200 import api as _api
    return _api


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def dev(x: torch.Tensor, dtype, ld=None) -> torch.Tensor:
    """Move an fp32 CPU tensor (already representable in dtype) to the GPU in dtype; with
    ld, into a wider buffer so the leading dimension differs from the width."""
    n, m = x.shape
    if ld is None:
        return x.to("cuda", dtype).contiguous()
    buf = torch.zeros(n, ld, device="cuda", dtype=dtype)
    buf[:, :m] = x.to("cuda", dtype)
    return buf[:, :m]


# A matrix-wide relative Frobenius error can hide a few rows (or one tile) that are entirely wrong,
# so every comparison also bounds the worst single row: max_t ||row_t - row_t^0|| / ||row_t^0||.
# bf16 results carry a rounding of 2^-9 per element plus the bf16 rounding of the basis operands, a
# few 1e-3 per row; a row that is wrong has an error of order 1.  ROW_FACTOR x the matrix tolerance
# separates the two with room on both sides.
ROW_FACTOR = 5.0


def row_errors(got: np.ndarray, want: np.ndarray):
    """(sum of squared differences, sum of squares of want, worst per-row relative error)."""
    diff = got - want
    num = np.einsum("ij,ij->i", diff, diff)
    den = np.einsum("ij,ij->i", want, want)
    floor = 1e-30 + 1e-12 * (den.mean() if den.size else 0.0)      # rows that are (almost) zero
    worst = float(np.sqrt(np.max(num / np.maximum(den, floor)))) if den.size else 0.0
    return float(num.sum()), float(den.sum()), worst


def assert_rows_close(got, want, tol, what=""):
    """Relative Frobenius error <= tol and every row within ROW_FACTOR * tol of its reference."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    num, den, worst = row_errors(got.reshape(got.shape[0], -1), want.reshape(want.shape[0], -1))
    fro = math.sqrt(num / den) if den > 0 else math.sqrt(num)
    assert fro <= tol, f"{what}: relative Frobenius error {fro:.3e} > {tol:.1e}"
    assert worst <= ROW_FACTOR * tol, f"{what}: worst row error {worst:.3e} > {ROW_FACTOR * tol:.1e}"


class BlockwiseCheck:
    """The same two bounds for a matrix compared in row blocks (the float64 reference of a full-size
    output is built a few thousand rows at a time)."""

    def __init__(self, tol, what):
        self.tol, self.what, self.num, self.den, self.worst, self.rows = tol, what, 0.0, 0.0, 0.0, 0

    def add(self, got, want):
        n, d, w = row_errors(np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64))
        self.num += n
        self.den += d
        self.worst = max(self.worst, w)
        self.rows += got.shape[0]

    def finish(self, expect_rows):
        assert self.rows == expect_rows, f"{self.what}: {self.rows} of {expect_rows} rows compared"
        fro = math.sqrt(self.num / self.den)
        assert fro <= self.tol, f"{self.what}: relative Frobenius error {fro:.3e} > {self.tol:.1e}"
        assert self.worst <= ROW_FACTOR * self.tol, f"{self.what}: worst row error {self.worst:.3e}"


def row_blocks(n, step=4096):
    return [(i, min(n, i + step)) for i in range(0, n, step)]


def random_orthonormal_pair(d, k, r, seed):
    g = torch.Generator().manual_seed(seed)
    q, _ = torch.linalg.qr(torch.randn(d, k + r, generator=g, dtype=torch.float64))
    q = q.to(torch.float32)
    return q[:, :k].contiguous(), q[:, k:].contiguous()


# ------------------------------------------------------------------------ generator

def test_philox_words_bit_exact(api):
    for seed, dc, n in [(0, 0, 4096), (0x0123456789ABCDEF, 0x7EDCBA9876543210, (1 << 20) + 3), (7, 1, 1), (7, 1, 5)]:
        got = api.prac_philox_words(seed, dc, n).cpu().numpy().view(np.uint32)
        want = orc.draw_words(seed, dc, n)
        assert np.array_equal(got, want)


def test_gaussian_matches_oracle(api):
    for seed, dc, d, r in [(0, 0, 512, 16), (3, 9, 1001, 37), (5, 0, 3, 5)]:
        got = f64(api.prac_gaussian(seed, dc, d, r))
        want = orc.gaussian_draw(seed, dc, d, r)
        assert got.shape == want.shape
        assert np.max(np.abs(got - want)) <= 2e-6


# ------------------------------------------------------------------------ compress / gradient with a given basis

SHAPES = [
    # N, d, k, r, d_out, pad (extra leading-dimension elements)
    (300, 136, 8, 8, 72, 0),          # 64-wide N tiles, ragged K block, ragged M tile
    (1000, 320, 48, 40, 200, 8),      # 128-wide N tile with ragged tail, padded leading dims
    (4096 + 77, 512, 128, 128, 768, 0),   # 256-wide tiles, several M tiles, ragged token tail
    (2048, 1000, 300, 212, 333, 0),   # s = 512 over two N tiles, d_out not a multiple of 8
    (513, 100, 10, 6, 50, 3),         # rows not 16-byte aligned: general kernels
]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape", SHAPES)
def test_compress_grad_reconstruct_stagewise(api, dtype, shape):
    N, d, k, r, d_out, pad = shape
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=1, dtype=name)
    dY = inputs.make_grad(N, d_out, seed=2, dtype=name)
    U, Q = random_orthonormal_pair(d, k, r, 3)
    c = (d - k) / r
    ldx = (d + pad) if pad else None
    ldy = (d_out + pad) if pad else None
    Xd, dYd = dev(X, dtype, ldx), dev(dY, dtype, ldy)
    b = api.Basis(d, k, r, dtype)
    b.set(U.cuda(), Q.cuda(), c)
    Ud, Qd, cd = b.get()
    assert cd == c and torch.equal(Ud.cpu(), U) and torch.equal(Qd.cpu(), Q)

    Z = b.compress(Xd)
    assert Z.shape == (N, k + r) and Z.dtype == dtype
    Z0 = orc.compress(f64(X), f64(U), f64(Q))
    assert_rows_close(f64(Z), Z0, TOL[dtype], "Z")

    # gradient from the GPU's own Z (stage-wise), fp32 output
    dW = b.weight_grad(dYd, Z)
    dW0 = orc.weight_grad(f64(dY), f64(Z), f64(U), f64(Q), c)
    assert dW.shape == (d_out, d)
    assert_rows_close(f64(dW), dW0, TOL[dtype], "dW")
    # end to end from X
    dW1 = orc.weight_grad(f64(dY), Z0, f64(U), f64(Q), c)
    assert orc.rel_fro(f64(dW), dW1) <= 2 * TOL[dtype]
    # accumulate and explicit scale override
    acc = b.weight_grad(dYd, Z, out=dW.clone(), accumulate=True, c=1.0)
    dWc1 = orc.weight_grad(f64(dY), f64(Z), f64(U), f64(Q), 1.0)
    assert orc.rel_fro(f64(acc), dW0 + dWc1) <= TOL[dtype]
    # storage-dtype output
    dWs = b.weight_grad(dYd, Z, out_dtype=dtype)
    assert dWs.dtype == dtype and orc.rel_fro(f64(dWs), dW0) <= 1e-2

    Xh = b.reconstruct(Z)
    Xh0 = orc.reconstruct(f64(Z), f64(U), f64(Q), c)
    assert_rows_close(f64(Xh), Xh0, 1e-5, "X^")
    assert b.status() == api.PRAC_OK


def test_outputs_are_deterministic(api):
    N, d, k, r, d_out = 3000, 512, 64, 64, 384
    X = dev(inputs.make_activation(N, d, seed=4, dtype="bf16"), torch.bfloat16)
    dY = dev(inputs.make_grad(N, d_out, seed=5, dtype="bf16"), torch.bfloat16)
    outs = []
    for _ in range(2):
        b = api.Basis(d, k, r, torch.bfloat16)
        b.fit(X, seed=11)
        Z = b.compress(X)
        dW = b.weight_grad(dY, Z)
        P, _ = b.projection()
        outs.append((P.clone(), Z.clone(), dW.clone()))
        assert b.status() == api.PRAC_OK
    for a, bb in zip(outs[0], outs[1]):
        assert torch.equal(a, bb)


# ------------------------------------------------------------------------ the fit

def check_basis(api, b, X64, k, r, seed, dc, energy_tol=1e-3):
    U, Q, c = b.get()
    U64, Q64 = f64(U), f64(Q)
    d = X64.shape[1]
    assert c == orc.scale_factor(d, k, r)
    if k:
        assert np.linalg.norm(U64.T @ U64 - np.eye(k)) <= 1e-5
        U0 = orc.principal_basis(X64, k)
        e, e0 = np.linalg.norm(X64 @ U64) ** 2, np.linalg.norm(X64 @ U0) ** 2
        assert e >= (1.0 - energy_tol) * e0
    if r:
        assert np.linalg.norm(Q64.T @ Q64 - np.eye(r)) <= 1e-5
        assert np.linalg.norm(U64.T @ Q64) <= 1e-5
        # Q is unique given span(U) and the draw: compare column by column
        Q0 = orc.random_basis(U64, orc.gaussian_draw(seed, dc, d, r))
        assert np.linalg.norm(Q64 - Q0) / math.sqrt(r) <= 1e-4
    return U64, Q64, c


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_fit_planted_gap_projector(api, dtype):
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    for (N, d, k, r) in [(2048, 512, 16, 16), (1536, 384, 64, 32)]:
        X = inputs.make_planted(N, d, k, gap=4.0, seed=6, dtype=name)
        b = api.Basis(d, k, r, dtype)
        b.fit(dev(X, dtype), seed=21, draw_counter=3)
        assert b.status() == api.PRAC_OK
        U64, _, _ = check_basis(api, b, f64(X), k, r, 21, 3)
        U0 = orc.principal_basis(f64(X), k)
        assert orc.projector_distance(U64, U0) <= 1e-3


def test_fit_config1_fp32_end_to_end(api):
    # single linear layer, fp32: N=2048, d_in=d_out=512, k=r=16, sigma_i = 1/i, noise 1e-3
    w = inputs.WORKLOADS["single_f32"]
    X = inputs.workload_activation(w, w.d, seed=0)
    dY = inputs.make_grad(w.N, w.d, seed=0)
    k = r = 16
    b = api.Basis(w.d, k, r, torch.float32)
    Xd, dYd = X.cuda(), dY.cuda()
    b.fit(Xd, seed=0)
    assert b.status() == api.PRAC_OK
    U64, Q64, c = check_basis(api, b, f64(X), k, r, 0, 0)
    Z = b.compress(Xd)
    assert orc.rel_fro(f64(Z), orc.compress(f64(X), U64, Q64)) <= 1e-5
    dW = b.weight_grad(dYd, Z)
    assert orc.rel_fro(f64(dW), orc.weight_grad(f64(dY), f64(Z), U64, Q64, c)) <= 1e-5
    assert orc.rel_fro(f64(dW), orc.weight_grad_materialised(f64(dY), f64(Z), U64, Q64, c)) <= 1e-5


def test_fit_bf16_power_law(api):
    # LLaMA-130M-like input at a reduced token count: power-law spectrum, no planted gap
    N, d, k, r = 4096, 768, 64, 64
    X = inputs.make_activation(N, d, p=0.8, noise=1e-3, seed=0, dtype="bf16")
    b = api.Basis(d, k, r, torch.bfloat16)
    b.fit(dev(X, torch.bfloat16), seed=1)
    assert b.status() == api.PRAC_OK
    check_basis(api, b, f64(X), k, r, 1, 0)


def test_refresh_schedule_and_stale_q(api):
    N, d, k, r = 1024, 256, 16, 16
    X = dev(inputs.make_planted(N, d, k, seed=8, dtype="bf16"), torch.bfloat16)
    b = api.Basis(d, k, r, torch.bfloat16)
    with pytest.raises(api.PracError) as e:
        b.compress(X)
    assert e.value.code == api.PRAC_ESTATE
    b.fit_principal(X, seed=1)
    with pytest.raises(api.PracError) as e:       # U changed, Q must be redrawn first
        b.compress(X)
    assert e.value.code == api.PRAC_ESTATE
    b.draw_random(seed=1, draw_counter=0)
    _, Q_a, _ = b.get()
    b.draw_random(seed=1, draw_counter=1)          # T_2 refresh: same U, new Q
    U_b, Q_b, _ = b.get()
    assert not torch.equal(Q_a, Q_b)
    b.draw_random(seed=1, draw_counter=0)
    assert torch.equal(b.get()[1], Q_a)            # (seed, counter) reproduces the draw
    assert np.linalg.norm(f64(U_b).T @ f64(Q_b)) <= 1e-5
    assert b.status() == api.PRAC_OK


# ------------------------------------------------------------------------ edge cases

def test_edge_pac_r0(api):
    N, d, k = 512, 128, 8
    X = inputs.make_planted(N, d, k, seed=9, dtype="f32")
    b = api.Basis(d, k, 0, torch.float32)
    b.fit(X.cuda(), seed=0)
    U64, _, c = check_basis(api, b, f64(X), k, 0, 0, 0)
    Z = b.compress(X.cuda())
    Xh = b.reconstruct(Z)
    assert orc.rel_fro(f64(Xh), f64(X) @ U64 @ U64.T) <= 1e-5
    assert b.status() == api.PRAC_OK


def test_edge_rac_k0(api):
    N, d, r = 512, 96, 24
    X = inputs.make_activation(N, d, seed=10, dtype="bf16")
    b = api.Basis(d, 0, r, torch.bfloat16)
    b.fit(dev(X, torch.bfloat16), seed=5, draw_counter=2)
    U64, Q64, c = check_basis(api, b, f64(X), 0, r, 5, 2)
    assert c == d / r
    Z = b.compress(dev(X, torch.bfloat16))
    assert orc.rel_fro(f64(Z), f64(X) @ Q64) <= 1e-2
    assert b.status() == api.PRAC_OK


def test_edge_full_budget_is_exact(api):
    # k + r = d: c = 1 and the reconstruction is X itself
    N, d, k = 256, 64, 24
    r = d - k
    X = inputs.make_activation(N, d, seed=12, dtype="f32")
    dY = inputs.make_grad(N, 40, seed=12)
    b = api.Basis(d, k, r, torch.float32)
    b.fit(X.cuda(), seed=3)
    assert b.c == 1.0
    Z = b.compress(X.cuda())
    assert orc.rel_fro(f64(b.reconstruct(Z)), f64(X)) <= 1e-5
    assert orc.rel_fro(f64(b.weight_grad(dY.cuda(), Z)), f64(dY).T @ f64(X)) <= 1e-5
    assert b.status() == api.PRAC_OK


def test_edge_fewer_tokens_than_features(api):
    N, d, k, r = 48, 128, 8, 8
    X = inputs.make_activation(N, d, seed=13, dtype="f32")
    b = api.Basis(d, k, r, torch.float32)
    b.fit(X.cuda(), seed=4)
    assert b.status() == api.PRAC_OK
    check_basis(api, b, f64(X), k, r, 4, 0)


def test_edge_rank_deficient_input(api):
    # rank(X) = 4 < k = 8: U must still be orthonormal and contain the row space of X
    N, d, k, r = 512, 96, 8, 8
    X = inputs.make_planted(N, d, 4, seed=14, dtype="f32", exact_rank=True)
    b = api.Basis(d, k, r, torch.float32)
    b.fit(X.cuda(), seed=6)
    assert b.status() == api.PRAC_OK          # the spare columns are completed, not reported
    U, Q, c = b.get()
    U64, Q64 = f64(U), f64(Q)
    assert np.linalg.norm(U64.T @ U64 - np.eye(k)) <= 1e-4
    assert np.linalg.norm(U64.T @ Q64) <= 1e-4
    X64 = f64(X)
    assert np.linalg.norm(X64 - X64 @ U64 @ U64.T) <= 1e-4 * np.linalg.norm(X64)
    Z = b.compress(X.cuda())
    assert orc.rel_fro(f64(b.reconstruct(Z)), X64) <= 1e-3


def test_argument_errors(api):
    with pytest.raises(api.PracError):
        api.Basis(64, 40, 40, torch.float32)           # k + r > d
    with pytest.raises(api.PracError):
        api.Basis(64, 0, 0, torch.float32)             # k + r = 0
    b = api.Basis(64, 8, 8, torch.float32)
    X = torch.zeros(32, 64, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(api.PracError) as e:
        b.fit(X, seed=0, ws=small)
    assert e.value.code == api.PRAC_EWORKSPACE
    with pytest.raises(api.PracError) as e:
        b.draw_random(seed=0, draw_counter=1 << 63)
    assert e.value.code in (api.PRAC_EINVAL, api.PRAC_ESTATE)


# ------------------------------------------------------------------------ larger ranks, full-size launches

@pytest.mark.parametrize("shape", [(4096, 1024, 256, 256), (3072, 1536, 512, 256)])
def test_fit_planted_gap_large_rank(api, shape):
    # k = 256 and k = 512: panels of 384 and 768 columns (tensor-core iteration, both register
    # variants of the eigen-solver), checked as projectors against the exact eigenvectors
    N, d, k, r = shape
    X = inputs.make_planted(N, d, k, gap=4.0, seed=16, dtype="bf16")
    b = api.Basis(d, k, r, torch.bfloat16)
    b.fit(dev(X, torch.bfloat16), seed=5, draw_counter=1)
    assert b.status() == api.PRAC_OK
    U64, _, _ = check_basis(api, b, f64(X), k, r, 5, 1)
    U0 = orc.principal_basis(f64(X), k)
    assert orc.projector_distance(U64, U0) <= 1e-3


def _padded(x: torch.Tensor, dtype) -> torch.Tensor:
    """Same values in a buffer whose rows start on 128-byte boundaries (the benchmark's layout)."""
    n, m = x.shape
    buf = torch.zeros(n, inputs.pad64(m), dtype=dtype, device=x.device)
    buf[:, :m] = x.to(dtype)
    return buf[:, :m]


@pytest.mark.parametrize("d_in,d_out", [(2048, 5461), (5461, 2048), (2048, 10922)])
def test_full_size_launch_every_element(api, d_in, d_out):
    # LLaMA-1B shapes at the benchmark's token count, rank and memory layout: the kernels run in
    # the launch configuration that is timed (every worker owns several tiles: accumulator-buffer
    # reuse, ring wrap and tile stores across tiles), and every element of Z and of dW is compared.
    # d_out = 10922 is the up and gate projections side by side, as the benchmark calls them.
    w = inputs.WORKLOADS["llama1b"]
    N, k, r = w.N, 256, 256
    Xd = _padded(inputs.workload_activation(w, d_in, seed=3, device="cuda", N=N), torch.bfloat16)
    dYd = _padded(inputs.make_grad(N, d_out, seed=4, device="cuda", dtype="bf16"), torch.bfloat16)
    U, Q = random_orthonormal_pair(d_in, k, r, 9)
    c = (d_in - k) / r
    b = api.Basis(d_in, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(Xd)
    dW = b.weight_grad(dYd, Z)
    assert b.status() == api.PRAC_OK
    U64, Q64 = f64(U), f64(Q)
    chk = BlockwiseCheck(1e-2, "Z")
    for i0, i1 in row_blocks(N):
        chk.add(f64(Z[i0:i1]), orc.compress(f64(Xd[i0:i1]), U64, Q64))
    chk.finish(N)
    dW0 = orc.weight_grad(f64(dYd), f64(Z), U64, Q64, c)
    assert_rows_close(f64(dW), dW0, 1e-2, "dW")


WORKER_PAIRS = 74      # CTA pairs of the main kernel on a 148-SM part


def test_every_worker_owns_several_tiles_kmajor(api):
    # K-major family (compress, dW stage 2) with many short tiles: N = 30000 (ragged last row tile),
    # d = 512 (8 k-blocks per tile), s = 512: 118 x 2 = 236 tiles on 74 CTA pairs, so every pair walks
    # the accumulator double buffer, the stage ring and the tile-store buffers across tile borders
    # at least three times.  Every element of Z, and of a tall dW (stage 2: 44 x 2 tiles), is compared.
    N, d, k, r = 30000, 512, 256, 256
    assert ((N + 255) // 256) * ((k + r) // 256) >= 3 * WORKER_PAIRS
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=121, device="cuda", dtype="bf16")
    U, Q = random_orthonormal_pair(d, k, r, 122)
    c = 1.0
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Xd = X.to(torch.bfloat16).contiguous()
    Z = b.compress(Xd)
    assert b.status() == api.PRAC_OK
    assert_rows_close(f64(Z), orc.compress(f64(Xd), f64(U), f64(Q)), 1e-2, "Z")
    # stage 2 with many tiles: d_out = 11264 rows of dW over d = 512 columns (44 x 2 tiles), few tokens
    Nt, d_out = 512, 11264
    dY = inputs.make_grad(Nt, d_out, seed=123, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    for out_dtype in (torch.float32, torch.bfloat16):
        dW = b.weight_grad(dY, Z[:Nt], out_dtype=out_dtype)
        assert b.status() == api.PRAC_OK
        assert_rows_close(f64(dW), orc.weight_grad(f64(dY), f64(Z[:Nt]), f64(U), f64(Q), c), 1e-2, "dW")


@pytest.mark.parametrize("d", [3072, 3101])
def test_every_worker_owns_several_wide_tiles(api, d):
    # Compress with a long K and 257..512 output columns runs on 512-wide tiles (one accumulator that
    # fills tensor memory, handed back to the MMA warp in two halves): N = 57001 gives 223 row tiles,
    # three per CTA pair and a ragged last one; s = 333 ends inside the tile's second half, so the last
    # column block of every row leaves through the masked path.  d = 3072: rows on the 16-byte grid;
    # d = 3101: contiguous rows taken by row classes (K then runs up to 7 ahead).  Every element.
    N, k, r = 57001, 170, 163
    s_ = k + r
    assert (N + 255) // 256 >= 3 * WORKER_PAIRS and 256 < s_ <= 512
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=131, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    U, Q = random_orthonormal_pair(d, k, r, 132)
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), 1.0)
    ldz = (s_ + 7) // 8 * 8 + 16
    bigZ = torch.full((N, ldz), 7.0, dtype=torch.bfloat16, device="cuda")
    Z = b.compress(X, out=bigZ[:, :s_])
    Z2 = b.compress(X, out=torch.empty_like(bigZ)[:, :s_])
    assert b.status() == api.PRAC_OK
    assert bool((bigZ[:, s_:] == 7.0).all()) and torch.equal(Z, Z2)
    U64, Q64 = f64(U), f64(Q)
    chk = BlockwiseCheck(1e-2, "Z")
    for i0, i1 in row_blocks(N):
        chk.add(f64(Z[i0:i1]), orc.compress(f64(X[i0:i1]), U64, Q64))
    chk.finish(N)


def test_every_worker_owns_several_pieces_token_major(api):
    # token-major family (dY^T Z with K pieces and the ordered reduction): the workspace query tells
    # how many (tile, K piece) items the launch deals out; with d_out = 14208 (ragged last row tile),
    # s = 512 and N = 30000 (ragged last k-block) every tile is cut into several K pieces and there
    # are at least three items per CTA pair.  Every element of dW is compared.
    N, d, k, r, d_out = 30000, 512, 256, 256, 14208
    b = api.Basis(d, k, r, torch.bfloat16)
    s = k + r
    items = (b.grad_workspace_bytes(N, d_out) - d_out * s * 4) // (256 * 256 * 4)
    assert items >= 3 * WORKER_PAIRS and items > 2 * ((d_out + 255) // 256), items     # several pieces per tile too
    U, Q = random_orthonormal_pair(d, k, r, 124)
    c = 1.0
    b.set(U.cuda(), Q.cuda(), c)
    Z = inputs.make_grad(N, s, seed=125, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    dY = inputs.make_grad(N, d_out, seed=126, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    dW = b.weight_grad(dY, Z)
    assert b.status() == api.PRAC_OK
    assert_rows_close(f64(dW), orc.weight_grad(f64(dY), f64(Z), f64(U), f64(Q), c), 1e-2, "dW")
    # and the unscaled fp32 partial product of the token-sharded path, on its own: each entry is a
    # sum of 30000 products of unit-variance bf16 values accumulated in fp32 (K pieces in tensor
    # memory, then added in order), a random walk of about sqrt(30000) * 2^-24 ~ 1e-5 relative
    M = b.weight_grad_partial(dY, Z)
    assert_rows_close(f64(M), f64(dY).T @ f64(Z), 5e-5, "dY^T Z")


def test_gram_matrix_full_size_every_element(api):
    # the symmetric token-major launch (upper-triangle tiles, K pieces, mirrored reduction) at the
    # benchmark's size: C = X^T X for N = 32768, d = 2048 against the float64 product
    w = inputs.WORKLOADS["llama1b"]
    N, d = w.N, w.d
    Xd = _padded(inputs.workload_activation(w, d, seed=13, device="cuda", N=N), torch.bfloat16)
    b = api.Basis(d, 256, 256, torch.bfloat16)
    C = b.gram(Xd)
    assert b.status() == api.PRAC_OK and torch.equal(C, C.T)
    # fp32 accumulation in tensor memory over thousands of tokens per K piece: the diagonal and the
    # outlier channels are sums of same-signed terms, whose rounding errors add up instead of
    # averaging out (measured 4.5e-5); far inside what the subspace tolerances need
    X64 = f64(Xd)
    assert_rows_close(f64(C), X64.T @ X64, 1e-4, "X^T X")


def assert_same_up_to_summation_order(a, b, what):
    """Two bf16 results of the same product whose fp32 sums ran in a different order: equal after
    rounding almost everywhere, one bf16 step (2^-8 relative, or a tiny absolute amount near zero)
    apart where a sum fell next to a rounding boundary."""
    a32, b32 = a.float(), b.float()
    diff = (a32 - b32).abs()
    bound = torch.maximum(a32.abs(), b32.abs()) * 2.0 ** -7 + 1e-6 * float(b32.abs().max())
    assert bool((diff <= bound).all()), f"{what}: {float((diff - bound).max())} beyond one rounding step"
    assert float((diff > 0).float().mean()) < 0.10, f"{what}: too many elements differ"


def test_rows_off_the_16_byte_grid_small_shapes(api):
    # odd widths, contiguous rows (leading dimension = width), and a base pointer that is itself
    # only 2-byte aligned: the tensor-core kernels fetch such an operand with plain loads, and the
    # result must be the bit pattern the TMA path gives on a padded copy of the same values.
    # Compress with a 16-byte aligned base takes the rows by classes through TMA instead, which
    # shifts the groups the tensor core sums in: equal up to that.
    for (N, d, k, r, d_out, shift) in [(3000, 333, 104, 88, 301, 0), (1111, 1001, 130, 126, 777, 1), (700, 135, 70, 60, 131, 3)]:
        s_ = k + r
        X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=131, device="cuda", dtype="bf16").to(torch.bfloat16)
        flat = torch.zeros(N * d + 8, dtype=torch.bfloat16, device="cuda")
        Xu = flat[shift:shift + N * d].view(N, d)                 # ld = d, base off by `shift` elements
        Xu.copy_(X)
        Xp = _padded(X, torch.bfloat16)
        U, Q = random_orthonormal_pair(d, k, r, 132)
        c = (d - k) / r
        b = api.Basis(d, k, r, torch.bfloat16)
        b.set(U.cuda(), Q.cuda(), c)
        Zu, Zp = b.compress(Xu), b.compress(Xp)
        assert b.status() == api.PRAC_OK
        if shift == 0:
            assert_same_up_to_summation_order(Zu, Zp, "Z")
        else:
            assert torch.equal(Zu, Zp)
        assert_rows_close(f64(Zu), orc.compress(f64(X), f64(U), f64(Q)), 1e-2, "Z")
        # dY with an odd width as the unaligned operand of the token-major kernel
        W_, Qw = random_orthonormal_pair(256, 96, 96, 133)
        bw = api.Basis(256, 96, 96, torch.bfloat16)
        bw.set(W_.cuda(), Qw.cuda(), 1.0)
        Zw = inputs.make_grad(N, 192, seed=134, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
        dY = inputs.make_grad(N, d, seed=135, device="cuda", dtype="bf16").to(torch.bfloat16)
        flat2 = torch.zeros(N * d + 8, dtype=torch.bfloat16, device="cuda")
        dYu = flat2[shift:shift + N * d].view(N, d)
        dYu.copy_(dY)
        dWu, dWp = bw.weight_grad(dYu, Zw), bw.weight_grad(_padded(dY, torch.bfloat16), Zw)
        assert bw.status() == api.PRAC_OK
        if shift == 0:
            # dY's tokens taken by classes through TMA: other pieces of K, so the bf16 middle factor
            # rounds differently here and there; dW agrees to well below the tolerance against the oracle
            assert_rows_close(f64(dWu), f64(dWp), 1e-3, "dW, contiguous against padded dY")
        else:
            assert torch.equal(dWu, dWp)
        assert_rows_close(f64(dWu), orc.weight_grad(f64(dY), f64(Zw), f64(W_), f64(Qw), 1.0), 1e-2, "dW")


@pytest.mark.parametrize("shape", [(3001, 333, 90, 71, 8), (2050, 1002, 96, 64, 4), (4097, 1004, 72, 57, 2), (261, 333, 70, 60, 8)])
def test_row_classes_with_ragged_sizes(api, shape):
    # Rows taken by classes through TMA where nothing divides evenly: token counts that are not a
    # multiple of the class count (classes of unequal length), leading dimensions with 8, 4 and 2
    # classes, and a compressed width k + r that is odd (the last block of every Z row leaves through
    # the masked path, with the rows of a class 8 / 4 / 2 apart).  Z and dW against the oracle and
    # against the padded layout; the columns of Z's buffer beyond k + r keep their values.
    N, d, k, r, classes = shape
    assert 8 // math.gcd(d, 8) == classes
    s_ = k + r
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=161, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    assert X.stride(0) == d and X.data_ptr() % 16 == 0
    U, Q = random_orthonormal_pair(d, k, r, 162)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    ldz = (s_ + 7) // 8 * 8 + 8
    bigZ = torch.full((N, ldz), 7.0, dtype=torch.bfloat16, device="cuda")
    Z = b.compress(X, out=bigZ[:, :s_])
    Zp = b.compress(_padded(X, torch.bfloat16))
    assert b.status() == api.PRAC_OK and bool((bigZ[:, s_:] == 7.0).all())
    assert_same_up_to_summation_order(Z, Zp, "Z")
    assert_rows_close(f64(Z), orc.compress(f64(X), f64(U), f64(Q)), 1e-2, "Z")
    # dY of that odd width as the token-major operand: the tokens of a class are one piece of K
    bw = api.Basis(256, 96, 96, torch.bfloat16)
    W_, Qw = random_orthonormal_pair(256, 96, 96, 163)
    bw.set(W_.cuda(), Qw.cuda(), 1.0)
    Zw = inputs.make_grad(N, 192, seed=164, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    dY = inputs.make_grad(N, d, seed=165, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    dW = bw.weight_grad(dY, Zw)
    assert bw.status() == api.PRAC_OK
    assert_rows_close(f64(dW), orc.weight_grad(f64(dY), f64(Zw), f64(W_), f64(Qw), 1.0), 1e-2, "dW")
    assert_rows_close(f64(dW), f64(bw.weight_grad(_padded(dY, torch.bfloat16), Zw)), 1e-3, "dW, contiguous against padded dY")
    # the fused consumers take such dY / dX only when every class has the same number of rows
    if N > 128 and N % classes != 0:
        with pytest.raises(api.PracError) as e:
            b.activation_backward(Zp, X, "silu", out=torch.empty(N, d, dtype=torch.bfloat16, device="cuda"))
        assert e.value.code == api.PRAC_EALIGN


def test_outputs_narrower_than_their_buffers_leave_the_rest_alone(api):
    # Outputs whose width is not a multiple of 16 bytes, written into column slices of wider
    # buffers: the columns next to the output belong to the caller and must keep their values
    # (a tile store writes whole 16-byte pieces, so row ends take another way out of the kernel).
    N, d, k, r, d_out = 2048, 512, 100, 93, 333          # s = 193, d_out = 333: both odd
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=141, device="cuda", dtype="bf16").to(torch.bfloat16)
    U, Q = random_orthonormal_pair(d, k, r, 142)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    s_ = k + r
    bigZ = torch.full((N, 200), 7.0, dtype=torch.bfloat16, device="cuda")
    Z = b.compress(X, out=bigZ[:, :s_])
    assert b.status() == api.PRAC_OK and bool((bigZ[:, s_:] == 7.0).all())
    assert_rows_close(f64(Z), orc.compress(f64(X), f64(U), f64(Q)), 1e-2, "Z")
    # a fused consumer with an odd feature count: dX (N x 333) inside a buffer of 336 columns
    dY = inputs.make_grad(N, d_out, seed=143, device="cuda", dtype="bf16").to(torch.bfloat16)
    dYp = _padded(dY, torch.bfloat16)
    dk, dr = 40, 40
    Ua, Qa = random_orthonormal_pair(d_out, dk, dr, 144)
    ca = (d_out - dk) / dr
    ba = api.Basis(d_out, dk, dr, torch.bfloat16)
    ba.set(Ua.cuda(), Qa.cuda(), ca)
    Xa = inputs.make_activation(N, d_out, p=0.6, noise=5e-2, seed=145, device="cuda", dtype="bf16").to(torch.bfloat16) * 40.0
    Za = ba.compress(_padded(Xa, torch.bfloat16))
    bigX = torch.full((N, 336), 7.0, dtype=torch.bfloat16, device="cuda")
    dX = ba.activation_backward(Za, dYp, "silu", out=bigX[:, :d_out])
    assert ba.status() == api.PRAC_OK and bool((bigX[:, d_out:] == 7.0).all())
    assert orc.rel_fro(f64(dX), orc.activation_backward(f64(dY), f64(Za), f64(Ua), f64(Qa), ca, "silu")) <= 2e-2
    # the weight gradient of a linear with that odd input width: dW (256 x 333), fp32 and bf16
    dY2 = inputs.make_grad(N, 256, seed=146, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    want = orc.weight_grad(f64(dY2), f64(Za), f64(Ua), f64(Qa), ca)
    for dt in (torch.float32, torch.bfloat16):
        bigW = torch.full((256, 336), 7.0, dtype=dt, device="cuda")
        dW = ba.weight_grad(dY2, Za.contiguous(), out=bigW[:, :d_out])
        assert ba.status() == api.PRAC_OK and bool((bigW[:, d_out:] == 7.0).all())
        assert_rows_close(f64(dW), want, 1e-2, "dW")


def test_unpadded_ffn_width_full_size_every_element(api):
    # the layout a framework hands over for the LLaMA-1B FFN activation: N x 5461 bf16, contiguous
    # (row pitch 10922 bytes).  Compress, the weight gradient with dY of that width, the forward
    # linear and the fit, every element against the oracle and against the padded layout.
    w = inputs.WORKLOADS["llama1b"]
    N, d, k, r = w.N, w.ffn, 256, 256
    X = inputs.workload_activation(w, d, seed=3, device="cuda", N=N).to(torch.bfloat16).contiguous()
    assert X.stride(0) == d and (d * 2) % 16 != 0
    Xp = _padded(X, torch.bfloat16)
    U, Q = random_orthonormal_pair(d, k, r, 9)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(X)
    Zp = b.compress(Xp)
    assert b.status() == api.PRAC_OK
    assert_same_up_to_summation_order(Z, Zp, "Z")      # rows taken by classes through TMA
    U64, Q64 = f64(U), f64(Q)
    chk = BlockwiseCheck(1e-2, "Z")
    for i0, i1 in row_blocks(N):
        chk.add(f64(Z[i0:i1]), orc.compress(f64(X[i0:i1]), U64, Q64))
    chk.finish(N)
    # forward linear with that X (the down projection: W is 2048 x 5461, rows padded)
    Wd = _padded(inputs.make_grad(2048, d, seed=6, device="cuda", dtype="bf16") * 0.02, torch.bfloat16)
    Y, Z2 = b.linear_forward(X, Wd)
    assert b.status() == api.PRAC_OK and torch.equal(Z2, Zp)   # plain loads: the padded layout's bits
    W64 = f64(Wd)
    chk = BlockwiseCheck(1e-2, "Y")
    for i0, i1 in row_blocks(N):
        chk.add(f64(Y[i0:i1]), f64(X[i0:i1]) @ W64.T)
    chk.finish(N)
    # weight gradient of a linear whose output has that width (up / gate): dY is N x 5461 contiguous
    d_in = w.d
    Ui, Qi = random_orthonormal_pair(d_in, k, r, 10)
    bi = api.Basis(d_in, k, r, torch.bfloat16)
    ci = (d_in - k) / r
    bi.set(Ui.cuda(), Qi.cuda(), ci)
    Zi = inputs.make_grad(N, k + r, seed=7, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    dY = inputs.make_grad(N, d, seed=4, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    dW = bi.weight_grad(dY, Zi)
    assert bi.status() == api.PRAC_OK
    assert_rows_close(f64(dW), f64(bi.weight_grad(_padded(dY, torch.bfloat16), Zi)), 1e-3,
                      "dW, contiguous against padded dY")    # tokens by classes: other pieces of K
    assert_rows_close(f64(dW), orc.weight_grad(f64(dY), f64(Zi), f64(Ui), f64(Qi), ci), 1e-2, "dW")
    # the fit: X is copied to aligned rows for the Gram matrix, everything after that is the same
    bf, bp = api.Basis(d, k, r, torch.bfloat16), api.Basis(d, k, r, torch.bfloat16)
    bf.fit(X, seed=31, draw_counter=1)
    bp.fit(Xp, seed=31, draw_counter=1)
    assert bf.status() == api.PRAC_OK and torch.equal(bf.projection()[0], bp.projection()[0])
    assert torch.equal(bf.gram(X), bp.gram(Xp))
    check_basis(api, bf, f64(X), k, r, 31, 1)


def test_full_size_fit_energy_and_draw(api):
    # the fit at the benchmark's size (N = 32768, d = 2048, k = r = 256, outlier channels):
    # captured energy against the exact top-k subspace, orthonormality, and Q column by column
    w = inputs.WORKLOADS["llama1b"]
    N, d, k, r = w.N, w.d, 256, 256
    Xd = _padded(inputs.workload_activation(w, d, seed=0, device="cuda", N=N), torch.bfloat16)
    b = api.Basis(d, k, r, torch.bfloat16)
    b.fit(Xd, seed=77, draw_counter=2)
    assert b.status() == api.PRAC_OK
    check_basis(api, b, f64(Xd), k, r, 77, 2)


def test_linears_sharing_an_input_in_one_call(api):
    # q/k/v (or up/gate) read the same X, hence the same Z: their weight gradients are the row
    # blocks of one product over their output gradients side by side
    N, d, k, r = 3000, 512, 64, 64
    widths = [384, 200, 333]
    X = inputs.make_activation(N, d, seed=41, dtype="bf16")
    U, Q = random_orthonormal_pair(d, k, r, 42)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(dev(X, torch.bfloat16))
    dYs = [inputs.make_grad(N, wd, seed=50 + j, dtype="bf16") for j, wd in enumerate(widths)]
    total = sum(widths)
    side_by_side = torch.zeros(N, inputs.pad64(total), dtype=torch.bfloat16, device="cuda")
    c0 = 0
    for g, wd in zip(dYs, widths):
        side_by_side[:, c0:c0 + wd] = g.to("cuda", torch.bfloat16)
        c0 += wd
    dW = b.weight_grad(side_by_side[:, :total], Z)
    assert dW.shape == (total, d) and b.status() == api.PRAC_OK
    c0 = 0
    for g, wd in zip(dYs, widths):
        want = orc.weight_grad(f64(g), f64(Z), f64(U), f64(Q), c)
        assert orc.rel_fro(f64(dW[c0:c0 + wd]), want) <= 1e-2
        c0 += wd


@pytest.mark.parametrize("shape", [(3000, 512, 64, 64, 384, 0), (1500, 520, 72, 40, 333, 8), (130, 256, 32, 32, 256, 0),
                                   (100, 256, 32, 32, 96, 0)])
def test_linear_forward_reads_x_once_and_matches_both_products(api, shape):
    # Algorithm 2 forward: Y = X W^T and Z = X [U|Q] from one launch (bf16, N > 128) or from
    # the two products in turn; each against the oracle, and Z identical to prac_compress
    N, d, k, r, d_out, pad = shape
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=61, dtype="bf16")
    W = inputs.make_grad(d_out, d, seed=62, dtype="bf16") * 0.05
    W = W.to(torch.bfloat16).to(torch.float32)
    U, Q = random_orthonormal_pair(d, k, r, 63)
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), (d - k) / r)
    Xd = dev(X, torch.bfloat16, d + pad if pad else None)
    Wd = dev(W, torch.bfloat16, d + pad if pad else None)
    before = api.kernel_launches()
    Y, Z = b.linear_forward(Xd, Wd)
    launches = api.kernel_launches() - before
    assert launches == (1 if N > 128 else 2)
    assert b.status() == api.PRAC_OK
    Y0, Z0 = orc.linear_forward(f64(X), f64(W), f64(U), f64(Q))
    assert Y.shape == (N, d_out) and Z.shape == (N, k + r)
    assert orc.rel_fro(f64(Y), Y0) <= 1e-2
    assert orc.rel_fro(f64(Z), Z0) <= 1e-2
    assert torch.equal(Z, b.compress(Xd))
    Y1, none = b.linear_forward(Xd, Wd, want_z=False)
    assert none is None and orc.rel_fro(f64(Y1), Y0) <= 1e-2


def test_linear_forward_fp32_and_full_size(api):
    # fp32 storage takes the general path
    N, d, k, r, d_out = 700, 192, 16, 16, 100
    X = inputs.make_activation(N, d, seed=64, dtype="f32")
    W = inputs.make_grad(d_out, d, seed=65, dtype="f32") * 0.05
    U, Q = random_orthonormal_pair(d, k, r, 66)
    b = api.Basis(d, k, r, torch.float32)
    b.set(U.cuda(), Q.cuda(), (d - k) / r)
    Y, Z = b.linear_forward(X.cuda(), W.cuda())
    Y0, Z0 = orc.linear_forward(f64(X), f64(W), f64(U), f64(Q))
    assert orc.rel_fro(f64(Y), Y0) <= 1e-5 and orc.rel_fro(f64(Z), Z0) <= 1e-5
    # LLaMA-1B mlp-in -> up projection at the benchmark's token count and layout, every element
    w = inputs.WORKLOADS["llama1b"]
    N, d, d_out, k, r = w.N, 2048, 5461, 256, 256
    Xd = _padded(inputs.workload_activation(w, d, seed=5, device="cuda", N=N), torch.bfloat16)
    Wd = _padded(inputs.make_grad(d_out, d, seed=6, device="cuda", dtype="bf16") * 0.02, torch.bfloat16)
    U, Q = random_orthonormal_pair(d, k, r, 67)
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), (d - k) / r)
    Yb = torch.empty(N, inputs.pad64(d_out), dtype=torch.bfloat16, device="cuda")[:, :d_out]
    Y, Z = b.linear_forward(Xd, Wd, out_y=Yb)
    assert b.status() == api.PRAC_OK
    W64, U64, Q64 = f64(Wd), f64(U), f64(Q)
    chk_y, chk_z = BlockwiseCheck(1e-2, "Y"), BlockwiseCheck(1e-2, "Z")
    for i0, i1 in row_blocks(N):
        Y0, Z0 = orc.linear_forward(f64(Xd[i0:i1]), W64, U64, Q64)
        chk_y.add(f64(Y[i0:i1]), Y0)
        chk_z.add(f64(Z[i0:i1]), Z0)
    chk_y.finish(N)
    chk_z.finish(N)
    assert torch.equal(Z, b.compress(Xd))


def test_linear_forward_outputs_with_different_row_alignment(api):
    # Y with rows that are not 16-byte aligned (leading dimension 333) beside a Z with aligned
    # rows: the two store paths may not meet in one launch, so the products run in turn (two
    # launches); many short-K tiles, every element of both outputs compared
    N, d, k, r, d_out = 20000, 128, 56, 56, 333
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=68, device="cuda", dtype="bf16").to(torch.bfloat16)
    W = (inputs.make_grad(d_out, d, seed=69, device="cuda", dtype="bf16") * 0.05).to(torch.bfloat16)
    U, Q = random_orthonormal_pair(d, k, r, 70)
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), (d - k) / r)
    Yb = torch.full((N, d_out), float("nan"), dtype=torch.bfloat16, device="cuda")     # ld = 333
    Zb = torch.full((N, k + r), float("nan"), dtype=torch.bfloat16, device="cuda")     # ld = 112
    before = api.kernel_launches()
    Y, Z = b.linear_forward(X, W, out_y=Yb, out_z=Zb)
    assert api.kernel_launches() - before == 2 and b.status() == api.PRAC_OK
    Y0, Z0 = orc.linear_forward(f64(X), f64(W), f64(U), f64(Q))
    assert_rows_close(f64(Y), Y0, 1e-2, "Y")
    assert_rows_close(f64(Z), Z0, 1e-2, "Z")
    # the mirrored case: aligned Y, Z rows off the 16-byte grid
    Yb2 = torch.full((N, 336), float("nan"), dtype=torch.bfloat16, device="cuda")[:, :d_out]
    Zb2 = torch.full((N, k + r + 1), float("nan"), dtype=torch.bfloat16, device="cuda")[:, :k + r]
    Y2, Z2 = b.linear_forward(X, W, out_y=Yb2, out_z=Zb2)
    assert b.status() == api.PRAC_OK
    assert_rows_close(f64(Y2), Y0, 1e-2, "Y")
    assert_rows_close(f64(Z2), Z0, 1e-2, "Z")


@pytest.mark.parametrize("act", ["silu", "gelu"])
@pytest.mark.parametrize("dtype,shape", [(torch.bfloat16, (3000, 512, 96, 96)), (torch.bfloat16, (777, 328, 40, 24)),
                                         (torch.bfloat16, (100, 64, 8, 8)), (torch.float32, (900, 200, 24, 16))])
def test_activation_backward_on_the_rebuilt_input(api, act, dtype, shape):
    # Section 5.1, non-linear layers: dX = dY * f'(X^) with X^ rebuilt from Z (never stored in bf16)
    N, d, k, r = shape
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    X = inputs.make_activation(N, d, p=0.6, noise=5e-2, seed=81, dtype=name) * 40.0   # pre-activations of order 1
    dY = inputs.make_grad(N, d, seed=82, dtype=name)
    U, Q = random_orthonormal_pair(d, k, r, 83)
    c = (d - k) / r
    b = api.Basis(d, k, r, dtype)
    b.set(U.cuda(), Q.cuda(), c)
    Xd = dev(X.to(dtype).to(torch.float32), dtype)
    Z = b.compress(Xd)
    dYd = dev(dY, dtype)
    dX = b.activation_backward(Z, dYd, act)
    assert dX.shape == (N, d) and dX.dtype == dtype and b.status() == api.PRAC_OK
    want = orc.activation_backward(f64(dY), f64(Z), f64(U), f64(Q), c, act)
    assert float(np.abs(want).max()) > 0.1
    assert orc.rel_fro(f64(dX), want) <= (2e-2 if dtype == torch.bfloat16 else 1e-5)


def test_activation_backward_full_size_every_element(api):
    # the SiLU of a LLaMA-1B MLP: its input is the gate projection's output (N x 5461); rank 0.2 n each
    w = inputs.WORKLOADS["llama1b"]
    N, d = w.N, w.ffn
    k = r = int(0.2 * d)
    Xd = _padded(inputs.workload_activation(w, d, seed=7, device="cuda", N=N) * 30.0, torch.bfloat16)
    dYd = _padded(inputs.make_grad(N, d, seed=8, device="cuda", dtype="bf16"), torch.bfloat16)
    U, Q = random_orthonormal_pair(d, k, r, 84)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(Xd)
    out = torch.empty(N, inputs.pad64(d), dtype=torch.bfloat16, device="cuda")[:, :d]
    dX = b.activation_backward(Z, dYd, "silu", out=out)
    assert b.status() == api.PRAC_OK
    U64, Q64 = f64(U), f64(Q)
    chk = BlockwiseCheck(2e-2, "dX")
    for i0, i1 in row_blocks(N):
        chk.add(f64(dX[i0:i1]), orc.activation_backward(f64(dYd[i0:i1]), f64(Z[i0:i1]), U64, Q64, c, "silu"))
    chk.finish(N)


def test_new_entry_points_reject_bad_calls(api):
    d, k, r, N = 256, 32, 32, 300
    b = api.Basis(d, k, r, torch.bfloat16)
    Z = torch.zeros(N, k + r, dtype=torch.bfloat16, device="cuda")
    dY = torch.zeros(N, d, dtype=torch.bfloat16, device="cuda")
    X = torch.zeros(N, d, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64, d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.PracError) as e:           # no basis yet
        b.activation_backward(Z, dY, "silu")
    assert e.value.code == api.PRAC_ESTATE
    with pytest.raises(api.PracError) as e:
        b.linear_forward(X, W)
    assert e.value.code == api.PRAC_ESTATE
    Y, none = b.linear_forward(X, W, want_z=False)    # the plain linear needs no basis
    assert none is None and Y.shape == (N, 64)
    U, Q = random_orthonormal_pair(d, k, r, 5)
    b.set(U.cuda(), Q.cuda(), (d - k) / r)
    with pytest.raises(KeyError):
        b.activation_backward(Z, dY, "relu")
    lib = api.lib
    bad = lib.prac_activation_backward(b.handle, Z.data_ptr(), k + r, dY.data_ptr(), d, N, 7, dY.data_ptr(), d, None, 0, None)
    assert bad == api.PRAC_EINVAL
    # bf16 rows that do not start on 16-byte boundaries are turned away, not served slowly
    odd = torch.zeros(N, d + 1, dtype=torch.bfloat16, device="cuda")[:, :d]
    with pytest.raises(api.PracError) as e:
        b.activation_backward(Z, odd, "gelu")
    assert e.value.code == api.PRAC_EALIGN
    # fp32 needs its workspace
    bf = api.Basis(64, 8, 8, torch.float32)
    Uf, Qf = random_orthonormal_pair(64, 8, 8, 6)
    bf.set(Uf.cuda(), Qf.cuda(), 7.0)
    Zf = torch.zeros(10, 16, device="cuda"); dYf = torch.zeros(10, 64, device="cuda")
    rc = lib.prac_activation_backward(bf.handle, Zf.data_ptr(), 16, dYf.data_ptr(), 64, 10, 0, dYf.data_ptr(), 64, None, 0, None)
    assert rc == api.PRAC_EWORKSPACE
    assert bf.activation_backward(Zf, dYf, "silu").abs().max().item() == 0.0


@pytest.mark.parametrize("dtype,shape", [(torch.bfloat16, (3000, 512, 96, 96)), (torch.bfloat16, (777, 328, 40, 24)),
                                         (torch.bfloat16, (129, 136, 16, 16)), (torch.float32, (500, 200, 24, 16))])
def test_rmsnorm_backward_on_the_rebuilt_input(api, dtype, shape):
    # Section 5.1, non-linear layers: RMSNorm's backward with the input rebuilt from Z; the row
    # statistic rstd comes from the true input and is kept exactly
    N, d, k, r = shape
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    X = inputs.make_activation(N, d, p=0.6, noise=5e-2, seed=91, dtype=name) * 40.0
    dY = inputs.make_grad(N, d, seed=92, dtype=name)
    g = torch.Generator().manual_seed(93)
    gain = (1.0 + 0.2 * torch.randn(d, generator=g)).to(torch.float32)
    rstd = (1.0 / torch.sqrt((X.double() ** 2).mean(dim=1) + 1e-6)).to(torch.float32)
    U, Q = random_orthonormal_pair(d, k, r, 94)
    c = (d - k) / r
    b = api.Basis(d, k, r, dtype)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(dev(X.to(dtype).to(torch.float32), dtype))
    dX, dgain = b.rmsnorm_backward(Z, dev(dY, dtype), rstd.cuda(), gain.cuda())
    assert dX.shape == (N, d) and dX.dtype == dtype and dgain.shape == (d,) and b.status() == api.PRAC_OK
    dX0, dg0 = orc.rmsnorm_backward(f64(dY), f64(Z), f64(U), f64(Q), c, f64(rstd), f64(gain))
    tol = 2e-2 if dtype == torch.bfloat16 else 1e-5
    assert orc.rel_fro(f64(dX), dX0) <= tol
    assert orc.rel_fro(f64(dgain), dg0) <= (1e-2 if dtype == torch.bfloat16 else 1e-5)
    # twice the same: the reductions have a fixed order
    dX2, dgain2 = b.rmsnorm_backward(Z, dev(dY, dtype), rstd.cuda(), gain.cuda())
    assert torch.equal(dX, dX2) and torch.equal(dgain, dgain2)


@pytest.mark.parametrize("norm", ["rms", "layer"])
def test_norm_backward_full_size_every_element(api, norm):
    # the pre-attention normalisation of a LLaMA-1B block: N x 2048, rank 0.2 n each; every element
    # of dX and every entry of dgain (and dbias) against the oracle
    w = inputs.WORKLOADS["llama1b"]
    N, d = w.N, w.d
    k = r = int(0.2 * d)
    X = inputs.workload_activation(w, d, seed=9, device="cuda", N=N) * 30.0 + (0.25 if norm == "layer" else 0.0)
    Xd = _padded(X, torch.bfloat16)
    dYd = _padded(inputs.make_grad(N, d, seed=10, device="cuda", dtype="bf16"), torch.bfloat16)
    Xw = Xd.double()
    if norm == "rms":
        mean = None
        rstd = (1.0 / torch.sqrt((Xw ** 2).mean(dim=1) + 1e-6)).float().contiguous()
    else:
        mean = Xw.mean(dim=1).float().contiguous()
        rstd = (1.0 / torch.sqrt(Xw.var(dim=1, unbiased=False) + 1e-6)).float().contiguous()
    del Xw
    gain = (1.0 + 0.1 * torch.randn(d, device="cuda", generator=torch.Generator(device="cuda").manual_seed(4))).float()
    U, Q = random_orthonormal_pair(d, k, r, 95)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(Xd)
    if norm == "rms":
        dX, dgain = b.rmsnorm_backward(Z, dYd, rstd, gain)
        dX0, dg0 = orc.rmsnorm_backward(f64(dYd), f64(Z), f64(U), f64(Q), c, f64(rstd), f64(gain))
    else:
        dX, dgain, dbias = b.layernorm_backward(Z, dYd, mean, rstd, gain)
        dX0, dg0, db0 = orc.layernorm_backward(f64(dYd), f64(Z), f64(U), f64(Q), c, f64(mean), f64(rstd), f64(gain))
        assert orc.rel_fro(f64(dbias), db0) <= 1e-5
    assert b.status() == api.PRAC_OK
    assert_rows_close(f64(dX), dX0, 2e-2, "dX")
    assert orc.rel_fro(f64(dgain), dg0) <= 1e-2
    assert float(np.max(np.abs(f64(dgain) - dg0))) <= 5e-2 * float(np.sqrt(np.mean(dg0 ** 2)))


@pytest.mark.parametrize("shape", [(1024, 333, 40), (4096, 1001, 96), (2048, 1002, 64), (32768, 5461, 128)])
def test_fused_consumers_on_contiguous_rows_of_odd_width(api, shape):
    # dY and dX as a framework hands them over for an odd feature count: N x d contiguous, rows off the
    # 16-byte grid (d = 5461: the gate projection's output of the LLaMA-1B MLP).  The activation
    # backward gives the bits of the padded layout (same products, same element-wise step); the
    # norm backwards agree with it up to the order in which the row sums are added; all of them,
    # every element, against the oracle.
    N, d, k = shape
    r = k
    X = inputs.make_activation(N, d, p=0.6, noise=5e-2, seed=151, device="cuda", dtype="bf16").to(torch.bfloat16) * 40.0
    dY = inputs.make_grad(N, d, seed=152, device="cuda", dtype="bf16").to(torch.bfloat16).contiguous()
    assert dY.stride(0) == d and (2 * d) % 16 != 0
    dYp = _padded(dY, torch.bfloat16)
    U, Q = random_orthonormal_pair(d, k, r, 153)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(_padded(X, torch.bfloat16))
    U64, Q64, Z64, dY64 = f64(U), f64(Q), f64(Z), f64(dY)
    dXu = torch.full((N, d), 7.0, dtype=torch.bfloat16, device="cuda")        # contiguous: ld = d
    for act in ("silu", "gelu"):
        dXu.fill_(7.0)
        b.activation_backward(Z, dY, act, out=dXu)
        dXp = b.activation_backward(Z, dYp, act)
        assert b.status() == api.PRAC_OK and torch.equal(dXu, dXp)
        chk = BlockwiseCheck(2e-2, "dX " + act)
        for i0, i1 in row_blocks(N):
            chk.add(f64(dXu[i0:i1]), orc.activation_backward(dY64[i0:i1], Z64[i0:i1], U64, Q64, c, act))
        chk.finish(N)
    Xw = X.double()
    mean = Xw.mean(dim=1).float().contiguous()
    rstd = (1.0 / torch.sqrt(Xw.var(dim=1, unbiased=False) + 1e-6)).float().contiguous()
    gain = (1.0 + 0.1 * torch.randn(d, device="cuda", generator=torch.Generator(device="cuda").manual_seed(4))).float()
    dXu.fill_(7.0)
    _, dgain = b.rmsnorm_backward(Z, dY, rstd, gain, out=dXu)
    dXp, dgp = b.rmsnorm_backward(Z, dYp, rstd, gain)
    assert b.status() == api.PRAC_OK
    dX0, dg0 = orc.rmsnorm_backward(dY64, Z64, U64, Q64, c, f64(rstd), f64(gain))
    assert_rows_close(f64(dXu), dX0, 2e-2, "dX rms")
    assert_rows_close(f64(dXu), f64(dXp), 1e-2, "dX rms, contiguous against padded")
    assert orc.rel_fro(f64(dgain), dg0) <= 1e-2 and orc.rel_fro(f64(dgain), f64(dgp)) <= 1e-5
    dXu.fill_(7.0)
    _, dgain, dbias = b.layernorm_backward(Z, dY, mean, rstd, gain, out=dXu)
    assert b.status() == api.PRAC_OK
    dX0, dg0, db0 = orc.layernorm_backward(dY64, Z64, U64, Q64, c, f64(mean), f64(rstd), f64(gain))
    assert_rows_close(f64(dXu), dX0, 2e-2, "dX layer")
    assert orc.rel_fro(f64(dgain), dg0) <= 1e-2 and orc.rel_fro(f64(dbias), db0) <= 1e-5


def test_llama7b_shapes_every_element_and_fit(api):
    # the largest configuration (N = 16384, d = 4096 -> 11008, k = r = 512): every element of Z and
    # of dW, then the fit's captured energy (against the oracle's exact top-k basis) and
    # orthonormality at that rank
    w = inputs.WORKLOADS["llama7b"]
    N, d, d_out, k, r = w.N, w.d, w.ffn, 512, 512
    Xd = _padded(inputs.workload_activation(w, d, seed=11, device="cuda", N=N), torch.bfloat16)
    dYd = _padded(inputs.make_grad(N, d_out, seed=12, device="cuda", dtype="bf16"), torch.bfloat16)
    U, Q = random_orthonormal_pair(d, k, r, 96)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(Xd)
    dW = b.weight_grad(dYd, Z)
    assert b.status() == api.PRAC_OK
    X64 = f64(Xd)
    assert_rows_close(f64(Z), orc.compress(X64, f64(U), f64(Q)), 1e-2, "Z")
    assert_rows_close(f64(dW), orc.weight_grad(f64(dYd), f64(Z), f64(U), f64(Q), c), 1e-2, "dW")
    del dYd, dW
    b.fit(Xd, seed=5, draw_counter=1)
    assert b.status() == api.PRAC_OK
    Uf, Qf, cf = b.get()
    assert cf == orc.scale_factor(d, k, r)
    U64, Q64 = f64(Uf), f64(Qf)
    U0 = orc.principal_basis(X64, k)
    assert np.linalg.norm(X64 @ U64) ** 2 >= (1 - 1e-3) * np.linalg.norm(X64 @ U0) ** 2
    eye = np.eye(k)
    # fp32 storage of an orthonormal d x 512 matrix is itself off by about k * 2^-24 * O(1)
    assert np.linalg.norm(U64.T @ U64 - eye) <= 2e-5
    assert np.linalg.norm(Q64.T @ Q64 - eye) <= 2e-5
    assert np.linalg.norm(U64.T @ Q64) <= 2e-5
    Q0 = orc.random_basis(U64, orc.gaussian_draw(5, 1, d, r))
    assert np.linalg.norm(Q64 - Q0) / math.sqrt(r) <= 1e-4


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_token_shards_sum_to_the_full_batch(api, dtype):
    # the per-rank parts of a token-sharded batch, computed one after the other on this GPU and
    # summed here in place of the collective: same subspace and same gradient as the whole batch
    from paper_2602_23111_b200.sharded import ShardedCompressor, shard_rows
    N, d, k, r, d_out = 4100, 384, 32, 32, 200
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    X = inputs.make_planted(N, d, k, gap=4.0, seed=101, dtype=name)
    dY = inputs.make_grad(N, d_out, seed=102, dtype=name)
    Xd, dYd = dev(X, dtype), dev(dY, dtype)
    whole = api.Basis(d, k, r, dtype)
    whole.fit(Xd, seed=21, draw_counter=3)
    parts = api.Basis(d, k, r, dtype)
    C = torch.zeros(d, d, device="cuda")
    for rank in range(3):
        b0, b1 = shard_rows(N, 3, rank)
        C += parts.gram(Xd[b0:b1])
    assert torch.equal(C, C.T)
    C0 = f64(X).T @ f64(X)
    assert orc.rel_fro(f64(C), C0) <= 1e-5            # the inputs are exact in either dtype, the sums are fp32
    parts.fit_principal_gram(C, seed=21, draw_counter=3)
    parts.draw_random(seed=21, draw_counter=3)
    Uw, Qw, cw = whole.get()
    Up, Qp, cp = parts.get()
    assert cw == cp
    assert orc.projector_distance(f64(Up), f64(Uw)) <= 1e-3
    U0 = orc.principal_basis(f64(X), k)
    lam = np.linalg.eigvalsh(C0)[::-1]
    if lam[k - 1] / lam[k] >= 2.0:                     # a gap: the subspace itself is pinned
        assert orc.projector_distance(f64(Up), U0) <= 1e-3
    # gradient: parts of M summed, then finished, against the one-call path and the oracle
    Z = parts.compress(Xd)
    M = torch.zeros(d_out, k + r, device="cuda")
    for rank in range(3):
        b0, b1 = shard_rows(N, 3, rank)
        M += parts.weight_grad_partial(dYd[b0:b1], Z[b0:b1])
    dW = parts.weight_grad_finish(M)
    want = orc.weight_grad(f64(dY), f64(Z), f64(Up), f64(Qp), cp)
    assert orc.rel_fro(f64(dW), want) <= TOL[dtype]
    assert orc.rel_fro(f64(dW), f64(parts.weight_grad(dYd, Z))) <= TOL[dtype]
    # the driver itself with a group of one (no collective issued)
    sc = ShardedCompressor(api.Basis(d, k, r, dtype))
    sc.fit(Xd, seed=21, draw_counter=3)
    assert sc.bytes_reduced == 0
    assert orc.projector_distance(f64(sc.basis.get()[0]), f64(Uw)) <= 1e-3
    dW1 = sc.weight_grad(dYd, sc.compress(Xd))
    U1, Q1, c1 = sc.basis.get()
    assert orc.rel_fro(f64(dW1), orc.weight_grad(f64(dY), f64(sc.compress(Xd)), f64(U1), f64(Q1), c1)) <= TOL[dtype]
    assert parts.status() == api.PRAC_OK and sc.basis.status() == api.PRAC_OK


@pytest.mark.parametrize("dtype,shape", [(torch.bfloat16, (3000, 512, 96, 96)), (torch.bfloat16, (777, 328, 40, 24)),
                                         (torch.bfloat16, (129, 136, 16, 16)), (torch.float32, (500, 200, 24, 16))])
def test_layernorm_backward_on_the_rebuilt_input(api, dtype, shape):
    N, d, k, r = shape
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    X = inputs.make_activation(N, d, p=0.6, noise=5e-2, seed=111, dtype=name) * 40.0 + 0.5
    X = X.to(dtype).to(torch.float32)
    dY = inputs.make_grad(N, d, seed=112, dtype=name)
    g = torch.Generator().manual_seed(113)
    gain = (1.0 + 0.2 * torch.randn(d, generator=g)).to(torch.float32)
    mean = X.double().mean(dim=1).to(torch.float32)
    rstd = (1.0 / torch.sqrt(X.double().var(dim=1, unbiased=False) + 1e-6)).to(torch.float32)
    U, Q = random_orthonormal_pair(d, k, r, 114)
    c = (d - k) / r
    b = api.Basis(d, k, r, dtype)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(dev(X, dtype))
    dX, dgain, dbias = b.layernorm_backward(Z, dev(dY, dtype), mean.cuda(), rstd.cuda(), gain.cuda())
    assert dX.shape == (N, d) and dX.dtype == dtype and b.status() == api.PRAC_OK
    dX0, dg0, db0 = orc.layernorm_backward(f64(dY), f64(Z), f64(U), f64(Q), c, f64(mean), f64(rstd), f64(gain))
    assert orc.rel_fro(f64(dX), dX0) <= (2e-2 if dtype == torch.bfloat16 else 1e-5)
    assert orc.rel_fro(f64(dgain), dg0) <= (1e-2 if dtype == torch.bfloat16 else 1e-5)
    assert orc.rel_fro(f64(dbias), db0) <= 1e-5
    dX2, dgain2, dbias2 = b.layernorm_backward(Z, dev(dY, dtype), mean.cuda(), rstd.cuda(), gain.cuda())
    assert torch.equal(dX, dX2) and torch.equal(dgain, dgain2) and torch.equal(dbias, dbias2)
