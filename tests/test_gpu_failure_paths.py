"""Failure paths of the CUDA library, provoked without faulting the GPU: a grid barrier made to
give up through the poll-limit hook, the decoding of the device status word, and numerical
breakdown of the orthonormalisation on rank-deficient input (a numeric condition, nothing traps).
Every case ends with a normal call on the same basis, which must succeed."""
import numpy as np
import pytest
import torch

from oracle import prac_oracle as orc
from paper_2602_23111_b200 import inputs

pytestmark = pytest.mark.gpu

DEV_CHOL_PIVOT, DEV_JACOBI_NOCONV, DEV_WAIT_EXPIRED = 1, 2, 4      # bits of the device status word


@pytest.fixture(scope="module")
def api():
    from paper_2602_23111_b200 import api as _api
    return _api


def f64(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def test_grid_barrier_gives_up_reports_timeout_and_the_basis_stays_usable(api):
    # panel of 96 columns: the Cholesky kernel runs on 3 CTAs and the eigen-solver on 4, so their
    # grid barriers really wait; with a poll limit of 1 the first CTA to arrive gives up at once
    N, d, k, r = 2048, 512, 64, 64
    X = inputs.make_planted(N, d, k, gap=4.0, seed=201, dtype="bf16")
    Xd = X.to("cuda", torch.bfloat16)
    b = api.Basis(d, k, r, torch.bfloat16)
    api.lib.prac_debug_set_barrier_poll_limit(1)
    try:
        b.fit(Xd, seed=3, draw_counter=1)            # every kernel leaves through its normal exit
        assert b.status() == api.PRAC_ETIMEOUT
        assert b.status() == api.PRAC_OK             # the word is cleared when read
    finally:
        api.lib.prac_debug_set_barrier_poll_limit(0)
    b.fit(Xd, seed=3, draw_counter=1)
    assert b.status() == api.PRAC_OK
    U, Q, c = b.get()
    assert orc.projector_distance(f64(U), orc.principal_basis(f64(X), k)) <= 1e-3
    Q0 = orc.random_basis(f64(U), orc.gaussian_draw(3, 1, d, r))
    assert np.linalg.norm(f64(Q) - Q0) / np.sqrt(r) <= 1e-4


def test_status_word_decoding(api):
    # the first four bytes of the basis storage are the device status word; written here from the
    # host side (a plain copy) to check how prac_device_status maps its bits and that it clears them.
    # (The mbarrier waits of the tensor-core kernels raise the same WAIT_EXPIRED bit; they are not
    # made to expire on the GPU, where copies could still be in flight when a CTA gives up.)
    b = api.Basis(64, 8, 8, torch.float32)
    word = b.storage[:4].view(torch.int32)
    for bits, want in ((DEV_WAIT_EXPIRED, api.PRAC_ETIMEOUT), (DEV_CHOL_PIVOT, api.PRAC_ENUMERIC),
                       (DEV_JACOBI_NOCONV, api.PRAC_ENUMERIC), (DEV_WAIT_EXPIRED | DEV_CHOL_PIVOT, api.PRAC_ETIMEOUT)):
        word.fill_(bits)
        assert b.status() == want
        assert int(word.item()) == 0 and b.status() == api.PRAC_OK
    assert api.status_string(api.PRAC_ETIMEOUT) == "bounded device wait expired"


def test_zero_input_breaks_down_and_is_reported(api):
    # X = 0: every Gram matrix of the iteration is zero, the extra orthonormalisation pass cannot
    # help either, and the fit says so instead of handing back a basis that is not orthonormal
    N, d, k, r = 256, 128, 8, 8
    b = api.Basis(d, k, r, torch.float32)
    b.fit(torch.zeros(N, d, device="cuda"), seed=1)
    assert b.status() == api.PRAC_ENUMERIC
    X = inputs.make_planted(N, d, k, seed=202, dtype="f32")
    b.fit(X.cuda(), seed=1)                        # the same basis object afterwards
    assert b.status() == api.PRAC_OK
    assert orc.projector_distance(f64(b.get()[0]), orc.principal_basis(f64(X), k)) <= 1e-3


@pytest.mark.parametrize("case", ["rank_below_k", "fewer_tokens_than_panel_columns"])
def test_rank_deficient_input_is_completed_to_an_orthonormal_basis(api, case):
    # rank(X) < k, or fewer tokens than panel columns: the panel of the subspace iteration is rank
    # deficient, its guarded pivots leave amplified rounding noise in the spare columns, and the
    # extra pass turns that into orthonormal directions: PRAC_OK, U orthonormal and containing the
    # row space of X (any completion is a valid basis there)
    if case == "rank_below_k":
        N, d, k, r, rank = 512, 96, 8, 8, 4
        X = inputs.make_planted(N, d, rank, seed=14, dtype="f32", exact_rank=True)
    else:
        N, d, k, r, rank = 20, 128, 8, 8, 20
        X = inputs.make_activation(N, d, seed=13, dtype="f32")
    b = api.Basis(d, k, r, torch.float32)
    b.fit(X.cuda(), seed=6)
    assert b.status() == api.PRAC_OK
    U, Q, c = b.get()
    U64, Q64, X64 = f64(U), f64(Q), f64(X)
    assert np.linalg.norm(U64.T @ U64 - np.eye(k)) <= 1e-5
    assert np.linalg.norm(Q64.T @ Q64 - np.eye(r)) <= 1e-5
    assert np.linalg.norm(U64.T @ Q64) <= 1e-5
    if rank <= k:
        assert np.linalg.norm(X64 - X64 @ U64 @ U64.T) <= 1e-4 * np.linalg.norm(X64)
    else:
        e, e0 = np.linalg.norm(X64 @ U64) ** 2, np.linalg.norm(X64 @ orc.principal_basis(X64, k)) ** 2
        assert e >= (1.0 - 1e-3) * e0
