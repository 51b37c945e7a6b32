"""CPU oracle for the PRAC per-linear-layer activation compression path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, double-precision statement of what
the CUDA library must compute.  It is imported by the tests, by the smoke check and by
the benchmark's CPU-baseline leg; the product path never imports it, and it imports
nothing from the product.  It shares no code, table or constant generator with the
CUDA sources.

Notation (paper -> here): activation X is N x d ("(b*s) x n"); principal rank r_1 -> k;
random rank r_2 -> r; Q_1 -> U (d x k); Q_2 -> Q (d x r); the paper's scale factor
"k = (n - r_1)/r_2" -> c.  Stored compressed activations are Z = X [U | Q] without the
scale; c is applied once when the gradient (or the reconstruction) is formed, which
gives the same reconstruction as Algorithm 1's "X_2 = k X Q_2" (Section 5.1, the
identity X P P^T = X Q_1 Q_1^T + k X Q_2 Q_2^T).

Everything is float64.  Library primitives used as single steps: matmul, symmetric
eigendecomposition (for "top-r_1 right singular vectors"), Householder QR.

Pins (tests/test_oracle_*.py): Philox known-answer vectors of the published generator,
SVD-vs-Gram agreement, Eckart-Young tail energy, planted low-rank recovery, the
k+r=d identity, Monte-Carlo checks of the appendix lemma E[Q_2 Q_2^T] =
r_2/(n-r_1) (I - Q_1 Q_1^T), of the theorems "Unbiased Reconstruction of PRAC" and
"Variance Bound of PRAC" (the equality its proof derives), of the gradient-estimator
lemma of Section 3.2 (E[dW] = dY^T X), and of the RAC special case.
The paper prints no numeric value of any U, Q, Z or dW, so those values are pinned only
through the identities above ("parity unpinned" against printed numbers: there are none).
"""
from __future__ import annotations

import math

import numpy as np

# --------------------------------------------------------------------------------------
# Random draw S ~ N(0,1)^{d x r}  (Eq. "S_o = (I - Q_1 Q_1^T) S", Algorithm 1 "Sample S")
# The paper fixes no generator.  This build defines the draw as Philox4x32-10 (Salmon,
# Moraes, Dror, Shaw, SC'11) words -> 23-bit uniforms -> Box-Muller, as documented below.
# --------------------------------------------------------------------------------------

_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)
_PHILOX_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter, key):
    """Philox4x32 with 10 rounds, vectorised.

    counter: array (..., 4) of 32-bit words, key: array (..., 2) (broadcastable).
    Returns uint32 array (..., 4).  One round maps (c0,c1,c2,c3) to
    (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)); the key is bumped by the
    Weyl constants between rounds.
    """
    c = np.asarray(counter, dtype=np.uint64) & _MASK32
    k = np.asarray(key, dtype=np.uint64) & _MASK32
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0 = np.broadcast_to(k[..., 0], c0.shape).copy()
    k1 = np.broadcast_to(k[..., 1], c0.shape).copy()
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PHILOX_W0) & _MASK32
            k1 = (k1 + _PHILOX_W1) & _MASK32
        p0 = _PHILOX_M0 * c0          # < 2^64, exact in uint64
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def draw_words(seed: int, draw_counter: int, n_elems: int) -> np.ndarray:
    """The uint32 word assigned to each of the n_elems entries of a draw.

    Entry e (row-major index into the d x r matrix) takes output lane e&3 of the block
    with counter (lo32(e>>2), hi32(e>>2), lo32(draw_counter), hi32(draw_counter)) and
    key (lo32(seed), hi32(seed)).
    """
    n_blocks = (n_elems + 3) // 4
    blk = np.arange(n_blocks, dtype=np.uint64)
    dc = np.uint64(draw_counter & 0xFFFFFFFFFFFFFFFF)
    sd = np.uint64(seed & 0xFFFFFFFFFFFFFFFF)
    counter = np.stack(
        [blk & _MASK32, blk >> np.uint64(32),
         np.full(n_blocks, dc & _MASK32, dtype=np.uint64),
         np.full(n_blocks, dc >> np.uint64(32), dtype=np.uint64)], axis=-1)
    key = np.array([sd & _MASK32, sd >> np.uint64(32)], dtype=np.uint64)
    return philox4x32_10(counter, key).reshape(-1)[:n_elems]


def words_to_uniform(words: np.ndarray) -> np.ndarray:
    """u = (2 (w >> 9) + 1) * 2^-24: the midpoints of 2^23 equal cells of (0, 1); never
    0 or 1, and exact in binary32 as well as binary64 (odd numerator below 2^24)."""
    return (2.0 * (words.astype(np.uint64) >> np.uint64(9)).astype(np.float64) + 1.0) * 2.0 ** -24


def gaussian_draw(seed: int, draw_counter: int, d: int, r: int) -> np.ndarray:
    """S (d x r), S_ij ~ N(0,1), by Box-Muller on lane pairs (0,1) and (2,3) of a block:
    z_even = sqrt(-2 ln u_a) cos(2 pi u_b),  z_odd = sqrt(-2 ln u_a) sin(2 pi u_b),
    with u_a from the even lane and u_b from the odd lane."""
    n = d * r
    n_pad = 4 * ((n + 3) // 4)
    u = words_to_uniform(draw_words(seed, draw_counter, n_pad))
    ua, ub = u[0::2], u[1::2]
    rad = np.sqrt(-2.0 * np.log(ua))
    z = np.empty(n_pad, dtype=np.float64)
    z[0::2] = rad * np.cos(2.0 * np.pi * ub)
    z[1::2] = rad * np.sin(2.0 * np.pi * ub)
    return z[:n].reshape(d, r)


# --------------------------------------------------------------------------------------
# Projection construction (Section 4.3; Algorithm 1)
# --------------------------------------------------------------------------------------

def principal_basis(X: np.ndarray, k: int) -> np.ndarray:
    """Q_1: the top-k right singular vectors of X (Section 4.2 "PAC"; Algorithm 1,
    "top-r_1 right singular vectors of X"), as a d x k matrix with orthonormal columns.

    Right singular vectors of X are eigenvectors of X^T X; the k largest eigenvalues are
    taken.  Only the spanned subspace is defined (signs, and rotations inside repeated
    singular values, are free).
    """
    X = np.asarray(X, dtype=np.float64)
    d = X.shape[1]
    if k == 0:
        return np.zeros((d, 0))
    evals, evecs = np.linalg.eigh(X.T @ X)        # ascending
    return np.ascontiguousarray(evecs[:, ::-1][:, :k])


def scale_factor(d: int, k: int, r: int) -> float:
    """The unbiasedness scale (n - r_1)/r_2 (Theorem "Unbiased Reconstruction of PRAC";
    Algorithm 1, first statement).  For k = 0 this is RAC's n/r_2."""
    return (d - k) / r if r > 0 else 1.0


def random_basis(U: np.ndarray, S: np.ndarray) -> np.ndarray:
    """Q_2: the Q factor of the thin QR of S_o = (I - Q_1 Q_1^T) S (Eq. "so_prac"), with
    the sign convention diag(R) > 0 that the appendix lemma on the thin QR of a Gaussian
    matrix assumes (it makes the factor unique)."""
    S = np.asarray(S, dtype=np.float64)
    if S.shape[1] == 0:
        return np.zeros((S.shape[0], 0))
    So = S - U @ (U.T @ S)
    Qf, R = np.linalg.qr(So, mode="reduced")
    sgn = np.where(np.diag(R) < 0.0, -1.0, 1.0)
    return Qf * sgn[None, :]


def fit_basis(X: np.ndarray, k: int, r: int, seed: int, draw_counter: int = 0):
    """Algorithm 1 up to (not including) the compression line: (U, Q, c)."""
    d = X.shape[1]
    U = principal_basis(X, k)
    Q = random_basis(U, gaussian_draw(seed, draw_counter, d, r))
    return U, Q, scale_factor(d, k, r)


# --------------------------------------------------------------------------------------
# Compression, recovery and the weight gradient (Algorithm 1 last step; Algorithm 2)
# --------------------------------------------------------------------------------------

def compress(X: np.ndarray, U: np.ndarray, Q: np.ndarray) -> np.ndarray:
    """Z = X [U | Q]  (N x (k+r)); Algorithm 1's X_1 = X Q_1 and X_2 / k = X Q_2."""
    return np.asarray(X, dtype=np.float64) @ np.concatenate([U, Q], axis=1)


def linear_forward(X: np.ndarray, W: np.ndarray, U: np.ndarray, Q: np.ndarray):
    """Algorithm 2 forward of one linear layer: the layer output Y = X W^T (W is d_out x d, the
    orientation of the weight whose gradient weight_grad returns) and the tensor saved for the
    backward pass, Z = X [U | Q], instead of X."""
    X = np.asarray(X, dtype=np.float64)
    return X @ np.asarray(W, dtype=np.float64).T, compress(X, U, Q)


def reconstruct(Z: np.ndarray, U: np.ndarray, Q: np.ndarray, c: float) -> np.ndarray:
    """X~ = X_1 Q_1^T + X_2 Q_2^T with X_2 = c Z[:, k:]  (Algorithm 2, "Reconstruct input
    approximation"; the transposes are the ones Section 5.1's identity shows)."""
    k = U.shape[1]
    Z = np.asarray(Z, dtype=np.float64)
    return Z[:, :k] @ U.T + c * (Z[:, k:] @ Q.T)


_erf = np.vectorize(math.erf, otypes=[np.float64])


def activation_derivative(x: np.ndarray, kind: str) -> np.ndarray:
    """f'(x) for the element-wise activations Section 5.1 ("Layer-Wise Design", non-linear layers)
    names: SiLU f(x) = x sigma(x), and GeLU f(x) = x Phi(x) with the normal distribution function Phi."""
    x = np.asarray(x, dtype=np.float64)
    if kind == "silu":
        sg = 1.0 / (1.0 + np.exp(-x))
        return sg * (1.0 + x * (1.0 - sg))
    if kind == "gelu":
        Phi = 0.5 * (1.0 + _erf(x / math.sqrt(2.0)))
        phi = np.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)
        return Phi + x * phi
    raise ValueError(kind)


def activation_backward(dY, Z, U, Q, c, kind: str) -> np.ndarray:
    """Backward of y = f(x) when x was stored compressed (Algorithm 2 applied to a non-linear layer,
    Section 5.1): rebuild X~ from Z, then the layer's ordinary backward dX = dY * f'(X~)."""
    return np.asarray(dY, dtype=np.float64) * activation_derivative(reconstruct(Z, U, Q, c), kind)


def rmsnorm_backward(dY, Z, U, Q, c, rstd, gain):
    """Backward of y_t = gain * x_t * rstd_t (RMSNorm) when x was stored compressed (Section 5.1,
    non-linear layers; the per-token statistic rstd_t = (mean_i x_ti^2 + eps)^-1/2 is kept exactly,
    as the paper keeps the normalisation layers' means and variances).  With X~ rebuilt from Z:
        dgain_i = sum_t dY_ti X~_ti rstd_t
        dX_t    = rstd_t (gain * dY_t) - (rstd_t^3 / d) X~_t sum_i gain_i dY_ti X~_ti
    Returns (dX, dgain)."""
    dY = np.asarray(dY, dtype=np.float64)
    rstd = np.asarray(rstd, dtype=np.float64).reshape(-1, 1)
    gain = np.asarray(gain, dtype=np.float64).reshape(1, -1)
    Xh = reconstruct(Z, U, Q, c)
    d = Xh.shape[1]
    a = dY * gain
    u = np.sum(a * Xh, axis=1, keepdims=True)
    dX = rstd * a - (rstd ** 3 / d) * u * Xh
    dgain = np.sum(dY * Xh * rstd, axis=0)
    return dX, dgain


def layernorm_backward(dY, Z, U, Q, c, mean, rstd, gain):
    """Backward of y_t = gain * (x_t - mean_t) * rstd_t + bias (LayerNorm) when x was stored
    compressed (Section 5.1, non-linear layers; the per-token mean and rstd come from the true
    input and stay uncompressed).  With X~ rebuilt from Z and xn_t = (X~_t - mean_t) rstd_t:
        dbias_i = sum_t dY_ti            dgain_i = sum_t dY_ti xn_ti
        dX_t    = rstd_t [a_t - mean_i(a_t) - xn_t mean_i(a_ti xn_ti)],   a_t = gain * dY_t
    Returns (dX, dgain, dbias)."""
    dY = np.asarray(dY, dtype=np.float64)
    mean = np.asarray(mean, dtype=np.float64).reshape(-1, 1)
    rstd = np.asarray(rstd, dtype=np.float64).reshape(-1, 1)
    gain = np.asarray(gain, dtype=np.float64).reshape(1, -1)
    xn = (reconstruct(Z, U, Q, c) - mean) * rstd
    a = dY * gain
    dX = rstd * (a - a.mean(axis=1, keepdims=True) - xn * (a * xn).mean(axis=1, keepdims=True))
    return dX, np.sum(dY * xn, axis=0), np.sum(dY, axis=0)


def weight_grad_materialised(dY, Z, U, Q, c) -> np.ndarray:
    """Algorithm 2 as printed: rebuild X~, then the ordinary linear backward
    grad_W = dY^T X~  (d_out x d_in; the gradient-estimator lemma's X~^T grad_Y,
    transposed to the weight-is-(d_out x d_in) orientation)."""
    return np.asarray(dY, dtype=np.float64).T @ reconstruct(Z, U, Q, c)


def weight_grad(dY, Z, U, Q, c) -> np.ndarray:
    """The same gradient without X~: (dY^T Z) diag(1_k, c 1_r) [U | Q]^T."""
    k = U.shape[1]
    M = np.asarray(dY, dtype=np.float64).T @ np.asarray(Z, dtype=np.float64)
    M[:, k:] *= c
    return M @ np.concatenate([U, Q], axis=1).T


# --------------------------------------------------------------------------------------
# Comparison helpers used by parity tests (no method arithmetic)
# --------------------------------------------------------------------------------------

def projector_distance(A: np.ndarray, B: np.ndarray) -> float:
    """|| A A^T - B B^T ||_F for matrices with orthonormal columns, without forming the
    d x d projectors and without cancellation:
    ||AA^T - BB^T||_F^2 = ||(I - BB^T) A||_F^2 + ||(I - AA^T) B||_F^2."""
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    ra = A - B @ (B.T @ A)
    rb = B - A @ (A.T @ B)
    return float(np.sqrt(np.sum(ra * ra) + np.sum(rb * rb)))


def rel_fro(a: np.ndarray, b: np.ndarray) -> float:
    """|| a - b ||_F / || b ||_F."""
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(np.asarray(a, dtype=np.float64) - b) / (nb if nb > 0 else 1.0))
