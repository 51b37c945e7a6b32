"""Algorithm 1's lazy update schedule (refresh U every T1 steps, Q every T2 steps) and the
warm-started refresh of U."""
import numpy as np
import pytest
import torch

from oracle import prac_oracle as orc
from paper_2602_23111_b200 import inputs


def test_schedule_actions_table():
    from paper_2602_23111_b200.api import schedule_actions
    # first use always fits and draws, whatever t is
    assert schedule_actions(7, 4, 2, False) == ("fit", True)
    got = [schedule_actions(t, 4, 2, True) for t in range(9)]
    want = [("refresh", True), (None, False), (None, True), (None, False),
            ("refresh", True), (None, False), (None, True), (None, False), ("refresh", True)]
    assert got == want
    # T2 not a divisor of T1: a refresh of U still forces a new Q
    assert schedule_actions(4, 4, 3, True) == ("refresh", True)
    assert schedule_actions(3, 4, 3, True) == (None, True)
    with pytest.raises(ValueError):
        schedule_actions(0, 0, 1, True)


def f64(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


@pytest.mark.gpu
def test_warm_refresh_tracks_a_moving_subspace():
    from paper_2602_23111_b200 import api
    N, d, k, r = 2048, 512, 64, 64
    X0 = inputs.make_planted(N, d, k, gap=4.0, seed=21, dtype="bf16")
    b = api.Basis(d, k, r, torch.bfloat16)
    X0d = X0.to("cuda", torch.bfloat16)
    with pytest.raises(api.PracError) as e:
        b.refresh_principal(X0d)                     # nothing to start from yet
    assert e.value.code == api.PRAC_ESTATE
    b.fit(X0d, seed=3)
    # the activations drift: a perturbation of a few percent rotates the principal subspace
    g = torch.Generator().manual_seed(5)
    X1 = inputs.round_to(X0 + 0.03 * X0.std() * torch.randn(N, d, generator=g), "bf16")
    X1d = X1.to("cuda", torch.bfloat16)
    U_old = f64(b.get()[0])
    U1 = orc.principal_basis(f64(X1), k)
    assert orc.projector_distance(U_old, U1) > 1e-2          # the old basis is measurably off
    launches = api.kernel_launches()
    b.refresh_principal(X1d, seed=3, draw_counter=1, iters=2)
    warm_launches = api.kernel_launches() - launches
    with pytest.raises(api.PracError) as e:                   # Q is stale until redrawn
        b.compress(X1d)
    assert e.value.code == api.PRAC_ESTATE
    b.draw_random(seed=3, draw_counter=1)
    assert b.status() == api.PRAC_OK
    U, Q, c = b.get()
    U64, Q64 = f64(U), f64(Q)
    assert orc.projector_distance(U64, U1) <= 1e-3
    assert np.linalg.norm(U64.T @ U64 - np.eye(k)) <= 1e-5
    assert np.linalg.norm(U64.T @ Q64) <= 1e-5
    # two iterations instead of four: fewer launches than the cold fit
    launches = api.kernel_launches()
    b.fit_principal(X1d, seed=3, draw_counter=2)
    assert warm_launches < api.kernel_launches() - launches


@pytest.mark.gpu
def test_lazy_compressor_follows_algorithm_1():
    from paper_2602_23111_b200 import api
    N, d, k, r = 1024, 256, 16, 16
    X = inputs.make_planted(N, d, k, seed=8, dtype="bf16").to("cuda", torch.bfloat16)
    b = api.Basis(d, k, r, torch.bfloat16)
    lazy = api.LazyCompressor(b, T1=4, T2=2, seed=9)
    Us, Qs = [], []
    for t in range(6):
        Z = lazy.compress(t, X)
        U, Q, c = b.get()
        Us.append(U); Qs.append(Q)
        assert orc.rel_fro(f64(Z), orc.compress(f64(X), f64(U), f64(Q))) <= 1e-2
        assert np.linalg.norm(f64(U).T @ f64(Q)) <= 1e-5
    assert [a for (_, a, _) in lazy.log] == ["fit", None, None, None, "refresh", None]
    assert [dr for (_, _, dr) in lazy.log] == [True, False, True, False, True, False]
    same = lambda a, b_: torch.equal(a, b_)
    assert same(Us[0], Us[1]) and same(Us[1], Us[3]) and same(Us[4], Us[5])
    assert same(Qs[0], Qs[1]) and not same(Qs[1], Qs[2]) and same(Qs[2], Qs[3]) and not same(Qs[3], Qs[4])
    # each Q is the draw of its step: reproducible from (seed, t)
    Q2 = orc.random_basis(f64(Us[2]), orc.gaussian_draw(9, 2, d, r))
    assert np.linalg.norm(f64(Qs[2]) - Q2) / np.sqrt(r) <= 1e-4
    assert b.status() == api.PRAC_OK
