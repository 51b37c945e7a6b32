"""The bounds-checking build (libprac_dbg.so, -DPRAC_DEBUG_BOUNDS): the same sources with every
self-computed global-memory index checked against the extent of its buffer.  It is run here over
tiny and odd shapes (the ones where a wrong tail or leading dimension would step outside) and must
count no violation while giving the oracle's results; it stands in for a memory checker."""
import importlib.util
import os

import numpy as np
import pytest
import torch

from oracle import prac_oracle as orc
from paper_2602_23111_b200 import inputs

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def f64(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


@pytest.fixture(scope="module")
def dbg():
    """The Python binding bound to the bounds-checking library instead of the normal one."""
    from paper_2602_23111_b200 import build
    path = build.build(debug_bounds=True)
    src = open(os.path.join(ROOT, "paper_2602_23111_b200", "api.py")).read()
    assert 'os.path.join(_HERE, "libprac.so")' in src
    spec = importlib.util.spec_from_loader("api_dbg", loader=None)
    mod = importlib.util.module_from_spec(spec)
    mod.__file__ = os.path.join(ROOT, "paper_2602_23111_b200", "api.py")
    exec(compile(src.replace('os.path.join(_HERE, "libprac.so")', repr(path)), "api_dbg", "exec"), mod.__dict__)
    return mod


def test_normal_build_has_no_counter():
    from paper_2602_23111_b200 import api
    assert api.lib.prac_debug_bounds_violations() == -1


SHAPES = [  # N, d, k, r, d_out, extra leading-dimension elements, dtype
    (64, 32, 4, 4, 24, 0, torch.float32),
    (513, 100, 10, 6, 50, 3, torch.float32),
    (300, 136, 8, 8, 72, 0, torch.bfloat16),       # tensor-core path with ragged tiles and the split-K reduction
    (513, 100, 10, 6, 50, 3, torch.bfloat16),      # bf16 rows off the 16-byte grid, too small for tiles: general kernels
    (1000, 333, 104, 88, 301, 0, torch.bfloat16),  # plain-load operand path
    (48, 128, 8, 8, 40, 0, torch.float32),         # fewer tokens than features
]


@pytest.mark.parametrize("shape", SHAPES)
def test_tiny_and_odd_shapes_stay_inside_their_buffers(dbg, shape):
    N, d, k, r, d_out, pad, dtype = shape
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    before = dbg.lib.prac_debug_bounds_violations()
    assert before >= 0
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=1, dtype=name)
    dY = inputs.make_grad(N, d_out, seed=2, dtype=name)

    def dev(x, ld):
        buf = torch.zeros(x.shape[0], ld, device="cuda", dtype=dtype)
        buf[:, :x.shape[1]] = x.to("cuda", dtype)
        return buf[:, :x.shape[1]]

    Xd, dYd = dev(X, d + pad), dev(dY, d_out + pad)
    b = dbg.Basis(d, k, r, dtype)
    b.fit(Xd, seed=3, draw_counter=1)
    assert b.status() == dbg.PRAC_OK
    U, Q, c = b.get()
    U64, Q64 = f64(U), f64(Q)
    assert np.linalg.norm(U64.T @ U64 - np.eye(k)) <= 1e-5 and np.linalg.norm(U64.T @ Q64) <= 1e-5
    Q0 = orc.random_basis(U64, orc.gaussian_draw(3, 1, d, r))
    assert np.linalg.norm(Q64 - Q0) / np.sqrt(r) <= 1e-4
    tol = 1e-2 if dtype == torch.bfloat16 else 1e-5
    Z = b.compress(Xd)
    assert orc.rel_fro(f64(Z), orc.compress(f64(X), U64, Q64)) <= tol
    for out_dtype in (torch.float32, dtype):
        dW = b.weight_grad(dYd, Z, out_dtype=out_dtype)
        assert orc.rel_fro(f64(dW), orc.weight_grad(f64(dY), f64(Z), U64, Q64, c)) <= 1e-2
    acc = b.weight_grad(dYd, Z, out=b.weight_grad(dYd, Z), accumulate=True)
    assert orc.rel_fro(f64(acc), 2.0 * orc.weight_grad(f64(dY), f64(Z), U64, Q64, c)) <= tol
    assert orc.rel_fro(f64(b.reconstruct(Z)), orc.reconstruct(f64(Z), U64, Q64, c)) <= 1e-5
    # the consumers of the rebuilt input that run on the general kernels (fp32 storage)
    if dtype == torch.float32:
        dYx = inputs.make_grad(N, d, seed=4, dtype=name).cuda()
        rstd = torch.rand(N, device="cuda") + 0.5
        mean = torch.randn(N, device="cuda") * 0.1
        gain = torch.rand(d, device="cuda") + 0.5
        b.activation_backward(Z, dYx, "gelu")
        b.rmsnorm_backward(Z, dYx, rstd, gain)
        b.layernorm_backward(Z, dYx, mean, rstd, gain)
    # token-sharded entry points and the refresh
    C = b.gram(Xd)
    b.fit_principal_gram(C, seed=3, draw_counter=1)
    b.draw_random(seed=3, draw_counter=1)
    b.weight_grad_finish(b.weight_grad_partial(dYd, Z))
    b.refresh_principal(Xd, seed=3, draw_counter=2)
    b.draw_random(seed=3, draw_counter=2)
    assert b.status() == dbg.PRAC_OK
    assert dbg.lib.prac_debug_bounds_violations() == before       # nothing stepped outside
