"""prac_weight_grad_static: the weight gradient for callers that cannot allocate device memory
or pass a workspace.  It must give what prac_weight_grad gives, call after call (the calls share
one fixed scratch array inside the library, which keeps the previous call's contents), and must
turn away problems too large for that array.  Collected last on purpose."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import prac_oracle as orc
from paper_2602_23111_b200 import inputs

pytestmark = pytest.mark.gpu


def f64(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def test_static_scratch_gradient_matches_workspace_gradient_twice():
    from paper_2602_23111_b200 import api
    assert api.lib.prac_static_scratch_bytes() == 32 << 20
    N, d, k, r = 2048 + 40, 512, 64, 64
    X = inputs.make_activation(N, d, p=0.8, noise=1e-2, seed=31, dtype="bf16").to("cuda", torch.bfloat16)
    b = api.Basis(d, k, r, torch.bfloat16)
    b.fit(X, seed=5)
    Z = b.compress(X)
    U, Q, c = b.get()
    # two calls in a row with different shapes: the second starts from the first one's leftovers
    for d_out, seed in ((768, 1), (200, 2)):
        dY = inputs.make_grad(N, d_out, seed=seed, dtype="bf16").to("cuda", torch.bfloat16)
        want = b.weight_grad(dY, Z)
        got = torch.full((d_out, d), float("nan"), dtype=torch.float32, device="cuda")
        b.weight_grad_static(dY, Z, out=got)
        assert b.status() == api.PRAC_OK
        assert orc.rel_fro(f64(got), f64(want)) <= 1e-2
        assert torch.equal(got, want)          # same kernels, same order of operations
        ref = orc.weight_grad(f64(dY), f64(Z), f64(U), f64(Q), c)
        assert orc.rel_fro(f64(got), ref) <= 1e-2
    # accumulate into an existing gradient, fp32 path as well
    Xf = inputs.make_activation(300, 96, seed=3, dtype="f32").cuda()
    bf = api.Basis(96, 8, 8, torch.float32)
    bf.fit(Xf, seed=1)
    Zf = bf.compress(Xf)
    dYf = inputs.make_grad(300, 40, seed=4).cuda()
    want = bf.weight_grad(dYf, Zf)
    got = want.clone()
    bf.weight_grad_static(dYf, Zf, out=got, accumulate=True)
    assert orc.rel_fro(f64(got), 2.0 * f64(want)) <= 1e-5


def test_static_scratch_rejects_oversized_problems():
    from paper_2602_23111_b200 import api
    d, k, r, d_out, N = 4096, 1024, 1024, 8192, 4096
    b = api.Basis(d, k, r, torch.bfloat16)
    assert b.grad_workspace_bytes(N, d_out) > api.lib.prac_static_scratch_bytes()
    P = torch.zeros(d, k + r, device="cuda")
    b.set(P[:, :k], P[:, k:], 1.0)
    dY = torch.zeros(N, d_out, dtype=torch.bfloat16, device="cuda")
    Z = torch.zeros(N, k + r, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(d_out, d, device="cuda")
    before = api.kernel_launches()
    with pytest.raises(api.PracError) as e:
        b.weight_grad_static(dY, Z, out=out)
    assert e.value.code == api.PRAC_EWORKSPACE
    assert api.kernel_launches() == before      # nothing was launched
    assert api.lib.prac_weight_grad_static(None, None, 1, 1, None, 1, 1, ctypes.c_double(0.0), None, 1, 1, 0,
                                           None) == api.PRAC_EINVAL
