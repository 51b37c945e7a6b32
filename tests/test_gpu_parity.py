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
    assert orc.rel_fro(f64(Z), Z0) <= TOL[dtype]

    # gradient from the GPU's own Z (stage-wise), fp32 output
    dW = b.weight_grad(dYd, Z)
    dW0 = orc.weight_grad(f64(dY), f64(Z), f64(U), f64(Q), c)
    assert dW.shape == (d_out, d)
    assert orc.rel_fro(f64(dW), dW0) <= TOL[dtype]
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
    assert orc.rel_fro(f64(Xh), Xh0) <= 1e-5
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
    st = b.status()
    assert st in (api.PRAC_OK, api.PRAC_ENUMERIC)
    check_basis(api, b, f64(X), k, r, 4, 0)


def test_edge_rank_deficient_input(api):
    # rank(X) = 4 < k = 8: U must still be orthonormal and contain the row space of X
    N, d, k, r = 512, 96, 8, 8
    X = inputs.make_planted(N, d, 4, seed=14, dtype="f32", exact_rank=True)
    b = api.Basis(d, k, r, torch.float32)
    b.fit(X.cuda(), seed=6)
    b.status()
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


@pytest.mark.parametrize("d_in,d_out", [(2048, 5461), (5461, 2048)])
def test_full_size_launch_sampled_parity(api, d_in, d_out):
    # LLaMA-1B shapes at the benchmark's token count, rank and memory layout: the kernels run in
    # the launch configuration that is timed; the oracle checks sampled rows of Z and of dW.
    w = inputs.WORKLOADS["llama1b"]
    N, k, r = w.N, 256, 256
    s = k + r
    Xd = _padded(inputs.workload_activation(w, d_in, seed=3, device="cuda", N=N), torch.bfloat16)
    dYd = _padded(inputs.make_grad(N, d_out, seed=4, device="cuda", dtype="bf16"), torch.bfloat16)
    U, Q = random_orthonormal_pair(d_in, k, r, 9)
    c = (d_in - k) / r
    b = api.Basis(d_in, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(Xd)
    dW = b.weight_grad(dYd, Z)
    assert b.status() == api.PRAC_OK
    g = torch.Generator().manual_seed(1)
    rows = torch.randint(0, N, (48,), generator=g)
    rows[0], rows[1] = 0, N - 1
    P64 = np.concatenate([f64(U), f64(Q)], axis=1)
    Z_rows = f64(Xd[rows.cuda()]) @ P64
    assert orc.rel_fro(f64(Z[rows.cuda()]), Z_rows) <= 1e-2
    outs = torch.randint(0, d_out, (24,), generator=g)
    outs[0], outs[1] = 0, d_out - 1
    Z64 = f64(Z)
    dW_rows = orc.weight_grad(f64(dYd[:, outs.cuda()]), Z64, f64(U), f64(Q), c)   # rows `outs` of dW
    assert orc.rel_fro(f64(dW[outs.cuda()]), dW_rows) <= 1e-2


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


def test_linear_forward_fp32_and_full_size_sampled(api):
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
    # LLaMA-1B mlp-in -> up projection at the benchmark's token count and layout, sampled rows
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
    g = torch.Generator().manual_seed(2)
    rows = torch.randint(0, N, (40,), generator=g)
    rows[0], rows[1] = 0, N - 1
    Y0, Z0 = orc.linear_forward(f64(Xd[rows.cuda()]), f64(Wd), f64(U), f64(Q))
    assert orc.rel_fro(f64(Y[rows.cuda()]), Y0) <= 1e-2
    assert orc.rel_fro(f64(Z[rows.cuda()]), Z0) <= 1e-2
    assert torch.equal(Z, b.compress(Xd))


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


def test_activation_backward_full_size_sampled(api):
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
    g = torch.Generator().manual_seed(3)
    rows = torch.randint(0, N, (32,), generator=g)
    rows[0], rows[1] = 0, N - 1
    want = orc.activation_backward(f64(dYd[rows.cuda()]), f64(Z[rows.cuda()]), f64(U), f64(Q), c, "silu")
    assert orc.rel_fro(f64(dX[rows.cuda()]), want) <= 2e-2


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


def test_rmsnorm_backward_full_size_sampled(api):
    # the pre-attention RMSNorm of a LLaMA-1B block: N x 2048, rank 0.2 n each
    w = inputs.WORKLOADS["llama1b"]
    N, d = w.N, w.d
    k = r = int(0.2 * d)
    X = inputs.workload_activation(w, d, seed=9, device="cuda", N=N) * 30.0
    Xd = _padded(X, torch.bfloat16)
    dYd = _padded(inputs.make_grad(N, d, seed=10, device="cuda", dtype="bf16"), torch.bfloat16)
    rstd = (1.0 / torch.sqrt((Xd.double() ** 2).mean(dim=1) + 1e-6)).float().contiguous()
    gain = (1.0 + 0.1 * torch.randn(d, device="cuda", generator=torch.Generator(device="cuda").manual_seed(4))).float()
    U, Q = random_orthonormal_pair(d, k, r, 95)
    c = (d - k) / r
    b = api.Basis(d, k, r, torch.bfloat16)
    b.set(U.cuda(), Q.cuda(), c)
    Z = b.compress(Xd)
    dX, dgain = b.rmsnorm_backward(Z, dYd, rstd, gain)
    assert b.status() == api.PRAC_OK
    g = torch.Generator().manual_seed(5)
    rows = torch.randint(0, N, (32,), generator=g)
    rows[0], rows[1] = 0, N - 1
    rc = rows.cuda()
    dX0, _ = orc.rmsnorm_backward(f64(dYd[rc]), f64(Z[rc]), f64(U), f64(Q), c, f64(rstd[rc]), f64(gain))
    assert orc.rel_fro(f64(dX[rc]), dX0) <= 2e-2
    # dgain needs every token: against the definition on sampled features, X^ from the oracle
    feats = torch.randint(0, d, (16,), generator=g)
    Xh = orc.reconstruct(f64(Z), f64(U)[feats.numpy()], f64(Q)[feats.numpy()], c)   # those columns of X^
    want = np.sum(f64(dYd[:, feats.cuda()]) * Xh * f64(rstd).reshape(-1, 1), axis=0)
    assert orc.rel_fro(f64(dgain[feats.cuda()]), want) <= 1e-2


def test_llama7b_shapes_sampled_parity_and_fit(api):
    # the largest configuration (N = 16384, d = 4096 -> 11008, k = r = 512): compress and the weight
    # gradient on sampled rows, then the fit's captured energy and orthonormality at that rank
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
    g = torch.Generator().manual_seed(6)
    rows = torch.randint(0, N, (32,), generator=g)
    rows[0], rows[1] = 0, N - 1
    assert orc.rel_fro(f64(Z[rows.cuda()]), orc.compress(f64(Xd[rows.cuda()]), f64(U), f64(Q))) <= 1e-2
    outs = torch.randint(0, d_out, (16,), generator=g)
    outs[0], outs[1] = 0, d_out - 1
    want = orc.weight_grad(f64(dYd[:, outs.cuda()]), f64(Z), f64(U), f64(Q), c)
    assert orc.rel_fro(f64(dW[outs.cuda()]), want) <= 1e-2
    # fit: energy against the exact top-k eigenvalues (float64 on the device is only the yardstick)
    b.fit(Xd, seed=5, draw_counter=1)
    assert b.status() == api.PRAC_OK
    Uf, Qf, cf = b.get()
    assert cf == (d - k) / r
    X64 = Xd.double()
    C = X64.T @ X64
    top = torch.linalg.eigvalsh(C)[-k:].sum().item()
    got = torch.trace(Uf.double().T @ C @ Uf.double()).item()
    assert got / top >= 1 - 1e-3
    eye = torch.eye(k, device="cuda", dtype=torch.float64)
    # fp32 storage of an orthonormal d x 512 matrix is itself off by about k * 2^-24 * O(1)
    assert torch.linalg.norm(Uf.double().T @ Uf.double() - eye).item() <= 2e-5
    assert torch.linalg.norm(Qf.double().T @ Qf.double() - eye).item() <= 2e-5
    assert torch.linalg.norm(Uf.double().T @ Qf.double()).item() <= 2e-5


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
