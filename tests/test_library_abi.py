"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every function
declared in include/prac.h, and its host-only queries validate their arguments."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    from paper_2602_23111_b200 import build
    build.build()
    from paper_2602_23111_b200 import api as _api
    return _api


def declared_functions():
    text = open(os.path.join(ROOT, "include", "prac.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(prac_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(api):
    names = declared_functions()
    assert len(names) >= 18
    raw = ctypes.CDLL(api.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
    assert set(api.EXPORTS) <= set(names)


def test_version_and_status_strings(api):
    assert api.lib.prac_version() >= 1000
    seen = {api.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert api.status_string(99) == "unknown status"


def test_size_queries_validate_params(api):
    P = api.PracParams
    ok = P(2048, 256, 256, api.PRAC_BF16, 0, 0, 0)
    nb = api.lib.prac_basis_bytes(ctypes.byref(ok))
    # fp32 P + two bf16 copies + status word, each region 256-byte aligned
    assert nb >= 2048 * 512 * (4 + 2 + 2) and nb % 256 == 0
    assert api.lib.prac_fit_workspace_bytes(ctypes.byref(ok), 32768) > 2048 * 2048 * 4
    assert api.lib.prac_grad_workspace_bytes(ctypes.byref(ok), 32768, 2048) >= 2048 * 512 * 2
    for bad in (P(64, 40, 40, 0, 0, 0, 0), P(64, 0, 0, 0, 0, 0, 0), P(0, 0, 1, 0, 0, 0, 0),
                P(64, -1, 8, 0, 0, 0, 0), P(64, 8, 8, 5, 0, 0, 0), P(64, 8, 8, 0, -1, 0, 0),
                P(64, 8, 8, 0, 0, 0, 1)):
        assert api.lib.prac_basis_bytes(ctypes.byref(bad)) == 0
        assert api.lib.prac_fit_workspace_bytes(ctypes.byref(bad), 128) == 0
        assert api.lib.prac_grad_workspace_bytes(ctypes.byref(bad), 128, 64) == 0
    assert api.lib.prac_fit_workspace_bytes(ctypes.byref(ok), 0) == 0
    assert api.lib.prac_grad_workspace_bytes(ctypes.byref(ok), 128, 0) == 0


def test_workspaces_have_room_for_operands_taken_by_row_classes(api):
    # An output width that is not a multiple of 8 means a contiguous dY has rows off the 16-byte grid,
    # which the weight gradient takes as one piece of K per class of rows: the size query leaves room
    # for one partial product per class (8 classes for an odd width, 4 and 2 for widths that are 2 and
    # 4 modulo 8), never less than the aligned layout needs; the norm backward's query covers the
    # extra row and column partials of that layout too.
    P = api.PracParams
    p = P(2048, 256, 256, api.PRAC_BF16, 0, 0, 0)
    N = 32768
    grad = lambda d_out: api.lib.prac_grad_workspace_bytes(ctypes.byref(p), N, d_out)
    tile = 256 * 256 * 4
    aligned = grad(5464)
    for d_out, classes in ((5461, 8), (5462, 4), (5460, 2)):
        need = grad(d_out)
        assert need >= aligned - 8 * tile                     # (5464 has at most a few columns more)
        tiles = ((d_out + 7 + 255) // 256) * 2                # row tiles of the offset output x two column tiles
        assert need >= classes * tiles * tile
    q = P(5461, 256, 256, api.PRAC_BF16, 0, 0, 0)
    rms = api.lib.prac_rmsnorm_workspace_bytes(ctypes.byref(q), N)
    parts = 2 * ((5461 + 7 + 255) // 256)
    assert rms >= parts * N * 4 + (N // 32 + 8) * 5461 * 4 + N * 4


def test_null_and_misaligned_arguments_are_rejected_before_any_launch(api):
    P = api.PracParams
    ok = P(64, 8, 8, api.PRAC_F32, 0, 0, 0)
    h = ctypes.c_void_p()
    assert api.lib.prac_basis_create(ctypes.byref(h), ctypes.byref(ok), None, 1 << 20) == api.PRAC_EINVAL
    assert api.lib.prac_basis_create(None, ctypes.byref(ok), None, 0) == api.PRAC_EINVAL
    assert api.lib.prac_basis_create(ctypes.byref(h), ctypes.byref(ok), 0x1001, 1 << 20) == api.PRAC_EALIGN
    assert api.lib.prac_basis_create(ctypes.byref(h), ctypes.byref(ok), 0x1000, 16) == api.PRAC_EWORKSPACE
    assert h.value is None
    for fn, args in (("prac_compress", (None, None, 1, 1, None, 1, None)),
                     ("prac_activation_backward", (None, None, 1, None, 1, 1, 0, None, 1, None, 0, None)),
                     ("prac_rmsnorm_backward", (None, None, 1, None, 1, 1, None, None, None, 1, None, None, 0, None)),
                     ("prac_gram", (None, None, 1, 1, None, 1, None, 0, None)),
                     ("prac_fit_principal_gram", (None, None, 1, 0, 0, None, 0, None)),
                     ("prac_weight_grad_partial", (None, None, 1, 1, None, 1, 1, None, 1, None, 0, None)),
                     ("prac_weight_grad_finish", (None, None, 1, 1, 0.0, None, 1, 0, 0, None, 0, None)),
                     ("prac_layernorm_backward", (None, None, 1, None, 1, 1, None, None, None, None, 1, None, None, None, 0, None)),
                     ("prac_linear_forward", (None, None, 1, 1, None, 1, 1, None, 1, None, 1, None)),
                     ("prac_reconstruct", (None, None, 1, 1, None, 1, None)),
                     ("prac_draw_random", (None, 0, 0, None, 0, None)),
                     ("prac_device_status", (None, None))):
        assert getattr(api.lib, fn)(*args) == api.PRAC_EINVAL
    assert api.lib.prac_philox_words(0, 0, -1, None, None) == api.PRAC_EINVAL
    assert api.lib.prac_gaussian(0, 0, 4, 4, None, 2, None) == api.PRAC_EINVAL
    api.lib.prac_basis_destroy(None)


def test_missing_library_fails_loudly(api, tmp_path, monkeypatch):
    import importlib.util
    spec = importlib.util.spec_from_file_location("api_copy", os.path.join(ROOT, "paper_2602_23111_b200", "api.py"))
    mod = importlib.util.module_from_spec(spec)
    src = open(os.path.join(ROOT, "paper_2602_23111_b200", "api.py")).read()
    code = compile(src.replace('os.path.join(_HERE, "libprac.so")', repr(str(tmp_path / "absent.so"))), "api_copy", "exec")
    with pytest.raises(RuntimeError, match="no fallback"):
        exec(code, mod.__dict__)
