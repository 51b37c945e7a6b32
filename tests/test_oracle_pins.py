"""Pins for the CPU oracle: every function is checked against something other than
itself -- published known-answer vectors, a different library routine, brute force on
tiny inputs, closed forms and the paper's expectation identities."""
import math
import os

import numpy as np
import pytest

from oracle import prac_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _orthonormal(d, k, seed):
    q, _ = np.linalg.qr(_rng(seed).standard_normal((d, k)))
    return q


def _spectrum_matrix(N, d, sig, seed):
    A, _ = np.linalg.qr(_rng(seed).standard_normal((N, d)))
    V = _orthonormal(d, d, seed + 1)
    return (A * sig[None, :]) @ V.T, V


# ------------------------------------------------------------------ Philox / Gaussian

def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        w = [int(x, 16) for x in row]
        out = orc.philox4x32_10(np.array(w[0:4], dtype=np.uint64), np.array(w[4:6], dtype=np.uint64))
        assert [int(x) for x in out] == w[6:10]


def test_draw_words_counter_layout():
    seed, dc = 0x0123456789ABCDEF, 0xFEDCBA9876543210
    n = 37
    words = orc.draw_words(seed, dc, n)
    assert words.dtype == np.uint32 and words.shape == (n,)
    for e in (0, 1, 2, 3, 4, 17, 36):
        blk = e >> 2
        ctr = np.array([blk & 0xFFFFFFFF, blk >> 32, dc & 0xFFFFFFFF, dc >> 32], dtype=np.uint64)
        key = np.array([seed & 0xFFFFFFFF, seed >> 32], dtype=np.uint64)
        assert int(words[e]) == int(orc.philox4x32_10(ctr, key)[e & 3])
    # a different draw counter or seed gives a different stream; same inputs the same one
    assert not np.array_equal(words, orc.draw_words(seed, dc + 1, n))
    assert not np.array_equal(words, orc.draw_words(seed + 1, dc, n))
    assert np.array_equal(words, orc.draw_words(seed, dc, n))
    # prefix property: a longer draw starts with the shorter one
    assert np.array_equal(orc.draw_words(seed, dc, 64)[:n], words)


def test_uniform_open_interval_and_exactness():
    w = np.array([0, 511, 512, 0xFFFFFFFF, 0x80000000], dtype=np.uint32)
    u = orc.words_to_uniform(w)
    assert u.min() > 0.0 and u.max() < 1.0
    assert u[0] == 2.0 ** -24 and u[1] == 2.0 ** -24 and u[2] == 3.0 * 2.0 ** -24
    assert u[3] == 1.0 - 2.0 ** -24 and u[4] == 0.5 + 2.0 ** -24
    allw = orc.words_to_uniform(np.arange(0, 2 ** 32, 2 ** 9, dtype=np.uint64).astype(np.uint32))
    assert abs(allw.mean() - 0.5) < 1e-12 and np.all(np.diff(allw) == 2.0 ** -23)
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)  # exact in binary32


def test_gaussian_moments_and_pair_structure():
    d, r = 2048, 1000
    G = orc.gaussian_draw(7, 3, d, r)
    z = G.reshape(-1)
    n = z.size
    assert abs(z.mean()) < 4.0 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 4.0 * math.sqrt(2.0 / n)
    assert abs((z ** 4).mean() - 3.0) < 4.0 * math.sqrt(96.0 / n)
    assert abs((z ** 3).mean()) < 4.0 * math.sqrt(15.0 / n)
    # Box-Muller: z_even^2 + z_odd^2 = -2 ln u_a, angle = 2 pi u_b
    u = orc.words_to_uniform(orc.draw_words(7, 3, n))
    assert np.allclose(z[0::2] ** 2 + z[1::2] ** 2, -2.0 * np.log(u[0::2]), rtol=1e-12)
    ang = np.mod(np.arctan2(z[1::2], z[0::2]), 2 * np.pi)
    assert np.allclose(ang, 2 * np.pi * u[1::2], atol=1e-9)
    # independence across the pair and across neighbours
    assert abs(np.mean(z[0::2] * z[1::2])) < 4.0 / math.sqrt(n / 2)
    assert abs(np.mean(z[:-2] * z[2:])) < 4.0 / math.sqrt(n)
    # row-major element order: entry (i, j) is element i*r + j
    assert G[5, 7] == z[5 * r + 7]


def test_gaussian_ragged_size():
    a = orc.gaussian_draw(1, 0, 3, 5)       # 15 entries: last block partly used
    b = orc.gaussian_draw(1, 0, 4, 4).reshape(-1)[:15]
    assert np.array_equal(a.reshape(-1), b)


# ------------------------------------------------------------------ principal basis

def test_principal_basis_matches_svd_and_eckart_young():
    N, d, k = 96, 24, 5
    sig = np.array([10.0, 8.0, 6.5, 5.0, 4.0] + [1.0 / (i + 1) for i in range(d - 5)])
    X, V = _spectrum_matrix(N, d, sig, 0)
    U = orc.principal_basis(X, k)
    assert U.shape == (d, k)
    assert np.linalg.norm(U.T @ U - np.eye(k)) < 1e-12
    # a different routine (one-sided SVD of X itself)
    _, s, Vt = np.linalg.svd(X, full_matrices=False)
    assert orc.projector_distance(U, Vt[:k].T) < 1e-10
    # the planted right singular vectors
    assert orc.projector_distance(U, V[:, :k]) < 1e-10
    # PAC error = tail energy (Section 4.2)
    err = np.linalg.norm(X - X @ U @ U.T) ** 2
    assert abs(err - np.sum(s[k:] ** 2)) < 1e-10 * np.sum(s ** 2)
    assert abs(err - np.sum(sig[k:] ** 2)) < 1e-10 * np.sum(sig ** 2)
    # columns ordered by decreasing singular value
    assert np.allclose(np.linalg.norm(X @ U, axis=0), s[:k], rtol=1e-10)


def test_principal_basis_brute_force_power_iteration():
    # tiny case: deflated power iteration written out with loops
    N, d, k = 20, 6, 2
    sig = np.array([5.0, 3.0, 1.0, 0.5, 0.2, 0.1])
    X, _ = _spectrum_matrix(N, d, sig, 3)
    C = X.T @ X
    vecs = []
    for _ in range(k):
        v = np.ones(d) / math.sqrt(d)
        for _ in range(2000):
            w = C @ v
            for u in vecs:
                w = w - u * (u @ w)
            v = w / np.linalg.norm(w)
        vecs.append(v)
    assert orc.projector_distance(orc.principal_basis(X, k), np.stack(vecs, 1)) < 1e-9


def test_planted_exact_low_rank_is_reconstructed_for_every_seed():
    N, d, k, r = 64, 20, 4, 3
    sig = np.zeros(d)
    sig[:k] = [4.0, 3.0, 2.0, 1.0]
    X, V = _spectrum_matrix(N, d, sig, 5)
    for seed in range(5):
        U, Q, c = orc.fit_basis(X, k, r, seed)
        assert orc.projector_distance(U, V[:, :k]) < 1e-10
        Xh = orc.reconstruct(orc.compress(X, U, Q), U, Q, c)
        assert np.linalg.norm(Xh - X) < 1e-10 * np.linalg.norm(X)


# ------------------------------------------------------------------ random basis

def test_random_basis_matches_gram_schmidt_brute_force():
    d, k, r = 9, 2, 4
    U = _orthonormal(d, k, 11)
    S = orc.gaussian_draw(2, 0, d, r)
    Q = orc.random_basis(U, S)
    # modified Gram-Schmidt against [U | previous q], positive normalisation
    cols = [U[:, j].copy() for j in range(k)]
    out = []
    for j in range(r):
        v = S[:, j].copy()
        for _ in range(2):
            for b in cols:
                v = v - b * float(b @ v)
        v = v / math.sqrt(float(v @ v))
        cols.append(v)
        out.append(v)
    Qgs = np.stack(out, axis=1)
    assert np.allclose(Q, Qgs, atol=1e-12)
    # diag(R) > 0: q_j has positive inner product with the projected column
    So = S - U @ (U.T @ S)
    assert np.all(np.sum(Q * So, axis=0) > 0)


def test_construction_invariants_and_scale():
    N, d, k, r = 80, 30, 6, 5
    X = _rng(0).standard_normal((N, d)) @ np.diag(np.arange(1, d + 1) ** -1.0)
    U, Q, c = orc.fit_basis(X, k, r, seed=9, draw_counter=2)
    assert c == (d - k) / r
    assert np.linalg.norm(U.T @ U - np.eye(k)) < 1e-12
    assert np.linalg.norm(Q.T @ Q - np.eye(r)) < 1e-12
    assert np.linalg.norm(U.T @ Q) < 1e-12
    assert orc.scale_factor(100, 0, 25) == 4.0          # RAC: n / r_2
    assert orc.scale_factor(2048, 256, 256) == 7.0


def test_full_rank_budget_is_exact():
    # k + r = d: c = 1 and [U | Q] is an orthogonal matrix, so X~ = X and dW = dY^T X
    N, d, k, dout = 40, 12, 5, 7
    r = d - k
    X = _rng(1).standard_normal((N, d))
    dY = _rng(2).standard_normal((N, dout))
    for seed in range(3):
        U, Q, c = orc.fit_basis(X, k, r, seed)
        assert c == 1.0
        Z = orc.compress(X, U, Q)
        assert np.allclose(orc.reconstruct(Z, U, Q, c), X, atol=1e-12)
        assert np.allclose(orc.weight_grad(dY, Z, U, Q, c), dY.T @ X, atol=1e-11)


def test_pac_and_rac_edge_cases():
    N, d = 50, 10
    X = _rng(4).standard_normal((N, d))
    # PAC: r = 0
    U, Q, c = orc.fit_basis(X, 3, 0, seed=0)
    assert Q.shape == (d, 0)
    Z = orc.compress(X, U, Q)
    assert Z.shape == (N, 3)
    assert np.allclose(orc.reconstruct(Z, U, Q, c), X @ U @ U.T, atol=1e-12)
    # RAC: k = 0
    U, Q, c = orc.fit_basis(X, 0, 4, seed=0)
    assert U.shape == (d, 0) and c == d / 4
    assert np.linalg.norm(Q.T @ Q - np.eye(4)) < 1e-12
    # Q equals the positive-diagonal QR factor of the raw draw
    S = orc.gaussian_draw(0, 0, d, 4)
    Qn, R = np.linalg.qr(S)
    assert np.allclose(Q, Qn * np.sign(np.diag(R))[None, :], atol=1e-12)


# ------------------------------------------------------------------ compress / gradient

def test_compress_and_gradient_by_explicit_loops():
    N, d, k, r, dout = 7, 6, 2, 2, 3
    X = _rng(6).standard_normal((N, d))
    dY = _rng(7).standard_normal((N, dout))
    U, Q, c = orc.fit_basis(X, k, r, seed=1)
    P = [[U[i, j] if j < k else Q[i, j - k] for j in range(k + r)] for i in range(d)]
    Z = orc.compress(X, U, Q)
    for t in range(N):
        for j in range(k + r):
            assert abs(Z[t, j] - sum(X[t, i] * P[i][j] for i in range(d))) < 1e-12
    dW = orc.weight_grad(dY, Z, U, Q, c)
    assert dW.shape == (dout, d)
    for o in range(dout):
        for i in range(d):
            # dW[o, i] = sum_t dY[t, o] * X~[t, i]
            acc = 0.0
            for t in range(N):
                xh = sum(Z[t, j] * P[i][j] * (1.0 if j < k else c) for j in range(k + r))
                acc += dY[t, o] * xh
            assert abs(dW[o, i] - acc) < 1e-10
    assert np.allclose(dW, orc.weight_grad_materialised(dY, Z, U, Q, c), rtol=0, atol=1e-11)


def test_linear_forward_by_explicit_loops_and_gradient_orientation():
    N, d, k, r, dout = 5, 6, 2, 3, 4
    X = _rng(16).standard_normal((N, d))
    W = _rng(17).standard_normal((dout, d))
    U, Q, c = orc.fit_basis(X, k, r, seed=2)
    Y, Z = orc.linear_forward(X, W, U, Q)
    assert Y.shape == (N, dout) and Z.shape == (N, k + r)
    for t in range(N):
        for o in range(dout):
            assert abs(Y[t, o] - sum(X[t, i] * W[o, i] for i in range(d))) < 1e-12
    assert np.array_equal(Z, orc.compress(X, U, Q))
    # orientation: with the full budget k + r = d the estimated gradient is the exact one, i.e. the
    # derivative of sum(dY * Y) with respect to W, checked by finite differences on one entry
    dY = _rng(18).standard_normal((N, dout))
    Uf, Qf, cf = orc.fit_basis(X, 3, 3, seed=2)
    dW = orc.weight_grad(dY, orc.compress(X, Uf, Qf), Uf, Qf, cf)
    W2 = W.copy()
    W2[1, 4] += 1e-6
    Y2, _ = orc.linear_forward(X, W2, Uf, Qf)
    fd = (np.sum(dY * Y2) - np.sum(dY * Y)) / 1e-6
    assert abs(fd - dW[1, 4]) < 1e-5 * max(1.0, abs(dW[1, 4]))


def test_activation_derivatives_against_differences_and_known_values():
    xs = np.concatenate([np.linspace(-9.0, 9.0, 73), [-30.0, -2.4, 0.0, 1e-3, 30.0]])
    h = 1e-5
    f = {"silu": lambda x: x / (1.0 + np.exp(-x)),
         "gelu": lambda x: np.array([0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in np.atleast_1d(x)])}
    for kind in ("silu", "gelu"):
        d = orc.activation_derivative(xs, kind)
        fd = (f[kind](xs + h) - f[kind](xs - h)) / (2 * h)
        assert np.max(np.abs(d - fd)) < 1e-8
        assert abs(orc.activation_derivative(np.array([0.0]), kind)[0] - 0.5) < 1e-15
        assert abs(orc.activation_derivative(np.array([40.0]), kind)[0] - 1.0) < 1e-12
        assert abs(orc.activation_derivative(np.array([-40.0]), kind)[0]) < 1e-12
    # the dip of SiLU's derivative below zero, and GeLU's overshoot above one
    assert abs(orc.activation_derivative(np.array([-2.3994]), "silu")[0] + 0.0998) < 1e-3
    assert orc.activation_derivative(np.array([1.5]), "gelu")[0] > 1.1
    with pytest.raises(ValueError):
        orc.activation_derivative(xs, "relu6")


def test_activation_backward_by_loops_and_exact_at_full_budget():
    N, d, k, r = 6, 5, 2, 2
    X = _rng(21).standard_normal((N, d))
    dY = _rng(22).standard_normal((N, d))
    U, Q, c = orc.fit_basis(X, k, r, seed=4)
    Z = orc.compress(X, U, Q)
    for kind in ("silu", "gelu"):
        dX = orc.activation_backward(dY, Z, U, Q, c, kind)
        for t in range(N):
            for i in range(d):
                xh = sum(Z[t, j] * U[i, j] for j in range(k)) + c * sum(Z[t, k + j] * Q[i, j] for j in range(r))
                want = dY[t, i] * orc.activation_derivative(np.array([xh]), kind)[0]
                assert abs(dX[t, i] - want) < 1e-12
        # k + r = d: the stored copy is exact, so the result is the uncompressed layer's backward
        Uf, Qf, cf = orc.fit_basis(X, 3, 2, seed=4)
        exact = dY * orc.activation_derivative(X, kind)
        got = orc.activation_backward(dY, orc.compress(X, Uf, Qf), Uf, Qf, cf, kind)
        assert np.max(np.abs(got - exact)) < 1e-10


def test_rmsnorm_backward_against_differences_of_the_forward_at_full_budget():
    # k + r = d: X~ = X, so the formulas must be the derivative of the RMSNorm forward itself
    N, d, eps = 5, 6, 1e-6
    X = _rng(31).standard_normal((N, d))
    g = _rng(32).standard_normal(d)
    dY = _rng(33).standard_normal((N, d))
    U, Q, c = orc.fit_basis(X, 4, 2, seed=5)
    Z = orc.compress(X, U, Q)

    def forward(Xv, gv):
        rs = 1.0 / np.sqrt(np.mean(Xv * Xv, axis=1, keepdims=True) + eps)
        return gv * Xv * rs, rs

    Y, rstd = forward(X, g)
    dX, dg = orc.rmsnorm_backward(dY, Z, U, Q, c, rstd, g)
    loss = lambda Xv, gv: float(np.sum(dY * forward(Xv, gv)[0]))
    h = 1e-6
    for (t, i) in [(0, 0), (2, 3), (4, 5), (1, 2)]:
        Xp, Xm = X.copy(), X.copy()
        Xp[t, i] += h; Xm[t, i] -= h
        assert abs((loss(Xp, g) - loss(Xm, g)) / (2 * h) - dX[t, i]) < 1e-6
    for i in range(d):
        gp, gm = g.copy(), g.copy()
        gp[i] += h; gm[i] -= h
        assert abs((loss(X, gp) - loss(X, gm)) / (2 * h) - dg[i]) < 1e-6
    # the gradient of a scale-invariant function is orthogonal to its argument (eps -> 0)
    _, rstd0 = forward(X, g)
    dX0, _ = orc.rmsnorm_backward(dY, Z, U, Q, c, 1.0 / np.sqrt(np.mean(X * X, axis=1)), g)
    assert np.max(np.abs(np.sum(dX0 * X, axis=1))) < 1e-9


def test_rmsnorm_backward_by_explicit_loops_on_a_compressed_input():
    N, d, k, r = 4, 6, 2, 2
    X = _rng(34).standard_normal((N, d))
    g = _rng(35).standard_normal(d)
    dY = _rng(36).standard_normal((N, d))
    rstd = 1.0 / np.sqrt(np.mean(X * X, axis=1) + 1e-6)
    U, Q, c = orc.fit_basis(X, k, r, seed=6)
    Z = orc.compress(X, U, Q)
    Xh = orc.reconstruct(Z, U, Q, c)
    dX, dg = orc.rmsnorm_backward(dY, Z, U, Q, c, rstd, g)
    for i in range(d):
        assert abs(dg[i] - sum(dY[t, i] * Xh[t, i] * rstd[t] for t in range(N))) < 1e-12
    for t in range(N):
        u = sum(g[i] * dY[t, i] * Xh[t, i] for i in range(d))
        for i in range(d):
            want = rstd[t] * g[i] * dY[t, i] - rstd[t] ** 3 / d * u * Xh[t, i]
            assert abs(dX[t, i] - want) < 1e-12


def test_layernorm_backward_against_differences_of_the_forward_at_full_budget():
    N, d, eps = 5, 6, 1e-6
    X = _rng(41).standard_normal((N, d)) + 0.7
    g = _rng(42).standard_normal(d)
    beta = _rng(43).standard_normal(d)
    dY = _rng(44).standard_normal((N, d))
    U, Q, c = orc.fit_basis(X, 4, 2, seed=7)          # k + r = d: X~ = X
    Z = orc.compress(X, U, Q)

    def forward(Xv, gv, bv):
        mu = Xv.mean(axis=1, keepdims=True)
        rs = 1.0 / np.sqrt(((Xv - mu) ** 2).mean(axis=1, keepdims=True) + eps)
        return gv * (Xv - mu) * rs + bv, mu, rs

    _, mu, rs = forward(X, g, beta)
    dX, dg, db = orc.layernorm_backward(dY, Z, U, Q, c, mu, rs, g)
    loss = lambda Xv, gv, bv: float(np.sum(dY * forward(Xv, gv, bv)[0]))
    h = 1e-6
    for (t, i) in [(0, 0), (2, 3), (4, 5), (1, 2)]:
        Xp, Xm = X.copy(), X.copy()
        Xp[t, i] += h; Xm[t, i] -= h
        assert abs((loss(Xp, g, beta) - loss(Xm, g, beta)) / (2 * h) - dX[t, i]) < 1e-6
    for i in range(d):
        gp, gm = g.copy(), g.copy(); gp[i] += h; gm[i] -= h
        assert abs((loss(X, gp, beta) - loss(X, gm, beta)) / (2 * h) - dg[i]) < 1e-6
        bp, bm = beta.copy(), beta.copy(); bp[i] += h; bm[i] -= h
        assert abs((loss(X, g, bp) - loss(X, g, bm)) / (2 * h) - db[i]) < 1e-6
    # the layer ignores a shift and (for eps -> 0) a scaling of its input row: dX_t sums to zero
    # and is orthogonal to the normalised row
    mu0 = X.mean(axis=1); rs0 = 1.0 / np.sqrt(((X - mu0[:, None]) ** 2).mean(axis=1))
    dX0, _, _ = orc.layernorm_backward(dY, Z, U, Q, c, mu0, rs0, g)
    assert np.max(np.abs(dX0.sum(axis=1))) < 1e-10
    assert np.max(np.abs(np.sum(dX0 * (X - mu0[:, None]), axis=1))) < 1e-9


def test_layernorm_backward_by_explicit_loops_on_a_compressed_input():
    N, d, k, r = 4, 6, 2, 2
    X = _rng(45).standard_normal((N, d)) - 0.3
    g = _rng(46).standard_normal(d)
    dY = _rng(47).standard_normal((N, d))
    mu = X.mean(axis=1)
    rs = 1.0 / np.sqrt(X.var(axis=1) + 1e-6)
    U, Q, c = orc.fit_basis(X, k, r, seed=8)
    Z = orc.compress(X, U, Q)
    Xh = orc.reconstruct(Z, U, Q, c)
    dX, dg, db = orc.layernorm_backward(dY, Z, U, Q, c, mu, rs, g)
    for i in range(d):
        assert abs(db[i] - sum(dY[t, i] for t in range(N))) < 1e-12
        assert abs(dg[i] - sum(dY[t, i] * (Xh[t, i] - mu[t]) * rs[t] for t in range(N))) < 1e-12
    for t in range(N):
        xn = [(Xh[t, i] - mu[t]) * rs[t] for i in range(d)]
        a = [g[i] * dY[t, i] for i in range(d)]
        ma = sum(a) / d
        mb = sum(a[i] * xn[i] for i in range(d)) / d
        for i in range(d):
            assert abs(dX[t, i] - rs[t] * (a[i] - ma - xn[i] * mb)) < 1e-12


# ------------------------------------------------------------------ expectation identities

def _mean_projector(U, d, r, seeds):
    k = U.shape[1]
    c = orc.scale_factor(d, k, r)
    acc = np.zeros((d, d))
    for s in seeds:
        Q = orc.random_basis(U, orc.gaussian_draw(s, 0, d, r))
        acc += c * (Q @ Q.T)
    return U @ U.T + acc / len(seeds)


def test_unbiased_projector_converges_at_monte_carlo_rate():
    # mean over draws of U U^T + c Q Q^T -> I (the lemma E[Q_2 Q_2^T] = r_2/(n-r_1) (I - Q_1 Q_1^T)
    # and the unbiased-reconstruction theorem); error ~ 1/sqrt(S)
    d, k, r = 12, 3, 3
    U = _orthonormal(d, k, 21)
    errs = []
    for S in (64, 256, 1024):
        errs.append(np.linalg.norm(_mean_projector(U, d, r, range(S)) - np.eye(d)))
    assert errs[2] < 0.25
    assert 1.5 < errs[0] / errs[1] < 2.7 and 1.5 < errs[1] / errs[2] < 2.7
    # a wrong scale (sqrt(c) or 1) leaves a bias that does not shrink
    acc = np.zeros((d, d))
    for s in range(256):
        Q = orc.random_basis(U, orc.gaussian_draw(s, 0, d, r))
        acc += Q @ Q.T
    biased = U @ U.T + acc / 256
    assert np.linalg.norm(biased - np.eye(d)) > 1.0


def test_variance_equality_for_any_orthonormal_U():
    # E ||X~ - X||_F^2 = (c - 1) ||X - X U U^T||_F^2  (the equality derived in the proof
    # of the variance theorem); it holds for any orthonormal U, fitted or not.
    N, d, k, r = 30, 14, 4, 5
    X = _rng(8).standard_normal((N, d)) @ np.diag(np.arange(1, d + 1) ** -0.7)
    for U in (orc.principal_basis(X, k), _orthonormal(d, k, 33)):
        c = orc.scale_factor(d, k, r)
        S = 3000
        tot = 0.0
        mean_hat = np.zeros_like(X)
        for s in range(S):
            Q = orc.random_basis(U, orc.gaussian_draw(s, 1, d, r))
            Xh = orc.reconstruct(orc.compress(X, U, Q), U, Q, c)
            tot += np.linalg.norm(Xh - X) ** 2
            mean_hat += Xh
        want = (c - 1.0) * np.linalg.norm(X - X @ U @ U.T) ** 2
        assert abs(tot / S - want) < 0.05 * want
        assert np.linalg.norm(mean_hat / S - X) < 0.06 * np.linalg.norm(X)


def test_rac_special_case():
    # k = 0: E[Q Q^T] = (r/d) I, variance (d/r - 1) ||X||_F^2
    N, d, r = 10, 8, 2
    X = _rng(9).standard_normal((N, d))
    U = np.zeros((d, 0))
    c = orc.scale_factor(d, 0, r)
    S = 4000
    acc = np.zeros((d, d))
    tot = 0.0
    for s in range(S):
        Q = orc.random_basis(U, orc.gaussian_draw(s, 0, d, r))
        acc += Q @ Q.T
        tot += np.linalg.norm(orc.reconstruct(orc.compress(X, U, Q), U, Q, c) - X) ** 2
    assert np.linalg.norm(acc / S - (r / d) * np.eye(d)) < 0.05
    want = (d / r - 1.0) * np.linalg.norm(X) ** 2
    assert abs(tot / S - want) < 0.05 * want


def test_gradient_estimator_is_unbiased():
    # mean over draws of dW -> dY^T X (gradient-estimator lemma, Section 3.2)
    N, d, k, r, dout = 16, 10, 2, 4, 5
    X = _rng(12).standard_normal((N, d))
    dY = _rng(13).standard_normal((N, dout))
    U = orc.principal_basis(X, k)
    c = orc.scale_factor(d, k, r)
    S = 4000
    acc = np.zeros((dout, d))
    for s in range(S):
        Q = orc.random_basis(U, orc.gaussian_draw(s, 0, d, r))
        acc += orc.weight_grad(dY, orc.compress(X, U, Q), U, Q, c)
    exact = dY.T @ X
    assert np.linalg.norm(acc / S - exact) < 0.05 * np.linalg.norm(exact)


def test_memory_ratio():
    # stored elements (k + r) per token instead of d (Table "Memory comparison", FFN rows)
    N, d, k, r = 32, 20, 3, 3
    X = _rng(0).standard_normal((N, d))
    U, Q, _ = orc.fit_basis(X, k, r, 0)
    assert orc.compress(X, U, Q).size / X.size == (k + r) / d


def test_comparison_helpers_against_explicit_forms():
    A, B = _orthonormal(15, 4, 1), _orthonormal(15, 4, 2)
    assert abs(orc.projector_distance(A, B) - np.linalg.norm(A @ A.T - B @ B.T)) < 1e-12
    assert orc.projector_distance(A, A @ _orthonormal(4, 4, 3)) < 1e-14   # rotation-invariant
    a, b = _rng(0).standard_normal((3, 4)), _rng(1).standard_normal((3, 4))
    assert abs(orc.rel_fro(a, b) - np.sqrt(((a - b) ** 2).sum() / (b ** 2).sum())) < 1e-15
