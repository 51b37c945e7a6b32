"""ctypes binding of libprac.so: argument marshalling only.

Every function below forwards to the C entry point of the same name (include/prac.h);
`Basis` bundles a handle with the torch-allocated device storage it lives in.  PyTorch is
used for device memory and streams, nothing else.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libprac.so")

PRAC_OK, PRAC_EINVAL, PRAC_EWORKSPACE, PRAC_EALIGN, PRAC_ENUMERIC, PRAC_ETIMEOUT, PRAC_ECUDA, PRAC_ESTATE = range(8)
PRAC_BF16, PRAC_F32 = 0, 1


class PracParams(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int64), ("k", ctypes.c_int64), ("r", ctypes.c_int64),
                ("dtype", ctypes.c_int32), ("oversample", ctypes.c_int32),
                ("iters", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class PracFitInfo(ctypes.Structure):
    _fields_ = [("panel_cols", ctypes.c_int32), ("iterations", ctypes.c_int32), ("eig_size", ctypes.c_int32),
                ("window_first", ctypes.c_int32), ("jacobi_sweeps", ctypes.c_int32), ("reserved", ctypes.c_int32 * 3)]


class PracError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} failed: {code} ({status_string(code)})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2602_23111_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, u64, i32, dbl, sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64, ctypes.c_int32,
                                  ctypes.c_double, ctypes.c_size_t)
    pp = ctypes.POINTER(PracParams)
    sigs = {
        "prac_version": (ctypes.c_int, []),
        "prac_kernel_launches": (ctypes.c_uint64, []),
        "prac_debug_set_barrier_poll_limit": (None, [ctypes.c_uint32]),
        "prac_debug_bounds_violations": (ctypes.c_int64, []),
        "prac_status_string": (ctypes.c_char_p, [ctypes.c_int]),
        "prac_basis_bytes": (sz, [pp]),
        "prac_fit_workspace_bytes": (sz, [pp, i64]),
        "prac_grad_workspace_bytes": (sz, [pp, i64, i64]),
        "prac_basis_create": (ctypes.c_int, [ctypes.POINTER(vp), pp, vp, sz]),
        "prac_basis_destroy": (None, [vp]),
        "prac_fit_basis": (ctypes.c_int, [vp, vp, i64, i64, u64, u64, vp, sz, vp]),
        "prac_fit_principal": (ctypes.c_int, [vp, vp, i64, i64, u64, u64, vp, sz, vp]),
        "prac_refresh_principal": (ctypes.c_int, [vp, vp, i64, i64, u64, u64, i32, vp, sz, vp]),
        "prac_draw_random": (ctypes.c_int, [vp, u64, u64, vp, sz, vp]),
        "prac_set_basis": (ctypes.c_int, [vp, vp, i64, vp, i64, dbl, vp]),
        "prac_basis_get": (ctypes.c_int, [vp, ctypes.POINTER(vp), ctypes.POINTER(i64), ctypes.POINTER(dbl)]),
        "prac_compress": (ctypes.c_int, [vp, vp, i64, i64, vp, i64, vp]),
        "prac_activation_backward": (ctypes.c_int, [vp, vp, i64, vp, i64, i64, ctypes.c_int32, vp, i64, vp, sz, vp]),
        "prac_activation_workspace_bytes": (sz, [pp, i64]),
        "prac_rmsnorm_backward": (ctypes.c_int, [vp, vp, i64, vp, i64, i64, vp, vp, vp, i64, vp, vp, sz, vp]),
        "prac_rmsnorm_workspace_bytes": (sz, [pp, i64]),
        "prac_layernorm_backward": (ctypes.c_int, [vp, vp, i64, vp, i64, i64, vp, vp, vp, vp, i64, vp, vp, vp, sz, vp]),
        "prac_layernorm_workspace_bytes": (sz, [pp, i64]),
        "prac_gram": (ctypes.c_int, [vp, vp, i64, i64, vp, i64, vp, sz, vp]),
        "prac_fit_principal_gram": (ctypes.c_int, [vp, vp, i64, u64, u64, vp, sz, vp]),
        "prac_weight_grad_partial": (ctypes.c_int, [vp, vp, i64, i64, vp, i64, i64, vp, i64, vp, sz, vp]),
        "prac_weight_grad_finish": (ctypes.c_int, [vp, vp, i64, i64, ctypes.c_double, vp, i64, ctypes.c_int32,
                                                   ctypes.c_int32, vp, sz, vp]),
        "prac_linear_forward": (ctypes.c_int, [vp, vp, i64, i64, vp, i64, i64, vp, i64, vp, i64, vp]),
        "prac_weight_grad": (ctypes.c_int, [vp, vp, i64, i64, vp, i64, i64, dbl, vp, i64, i32, i32, vp, sz, vp]),
        "prac_static_scratch_bytes": (sz, []),
        "prac_weight_grad_static": (ctypes.c_int, [vp, vp, i64, i64, vp, i64, i64, dbl, vp, i64, i32, i32, vp]),
        "prac_reconstruct": (ctypes.c_int, [vp, vp, i64, i64, vp, i64, vp]),
        "prac_device_status": (ctypes.c_int, [vp, vp]),
        "prac_fit_report": (ctypes.c_int, [vp, vp, sz, i64, vp, ctypes.POINTER(PracFitInfo)]),
        "prac_philox_words": (ctypes.c_int, [u64, u64, i64, vp, vp]),
        "prac_gaussian": (ctypes.c_int, [u64, u64, i64, i64, vp, i64, vp]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


lib = _load()
EXPORTS = ["prac_version", "prac_kernel_launches", "prac_debug_set_barrier_poll_limit", "prac_debug_bounds_violations", "prac_status_string", "prac_basis_bytes", "prac_fit_workspace_bytes",
           "prac_grad_workspace_bytes", "prac_basis_create", "prac_basis_destroy", "prac_fit_basis",
           "prac_fit_principal", "prac_refresh_principal", "prac_draw_random", "prac_set_basis", "prac_basis_get", "prac_compress", "prac_linear_forward", "prac_activation_backward", "prac_activation_workspace_bytes",
           "prac_rmsnorm_backward", "prac_rmsnorm_workspace_bytes",
           "prac_layernorm_backward", "prac_layernorm_workspace_bytes", "prac_gram", "prac_fit_principal_gram",
           "prac_weight_grad_partial", "prac_weight_grad_finish",
           "prac_weight_grad", "prac_static_scratch_bytes", "prac_weight_grad_static", "prac_reconstruct", "prac_device_status", "prac_fit_report", "prac_philox_words",
           "prac_gaussian"]


def kernel_launches() -> int:
    return int(lib.prac_kernel_launches())


def status_string(code: int) -> str:
    return lib.prac_status_string(int(code)).decode()


def _check(fn: str, code: int) -> None:
    if code != PRAC_OK:
        raise PracError(fn, code)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.bfloat16:
        return PRAC_BF16
    if t == torch.float32:
        return PRAC_F32
    raise TypeError(f"unsupported dtype {t}")


def _torch_dtype(code: int) -> torch.dtype:
    return torch.bfloat16 if code == PRAC_BF16 else torch.float32


def _mat(t: torch.Tensor, name: str) -> Tuple[int, int]:
    """(pointer, leading dimension) of a 2-D row-major CUDA tensor (unit inner stride)."""
    if not t.is_cuda or t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name}: expected a 2-D CUDA tensor with unit inner stride")
    return t.data_ptr(), (t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1]))


def _buffer(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def prac_philox_words(seed: int, draw_counter: int, n: int, device="cuda") -> torch.Tensor:
    out = torch.empty(n, dtype=torch.int32, device=device)
    _check("prac_philox_words", lib.prac_philox_words(seed, draw_counter, n, out.data_ptr(), _stream()))
    return out


def prac_gaussian(seed: int, draw_counter: int, d: int, r: int, device="cuda") -> torch.Tensor:
    out = torch.empty(d, r, dtype=torch.float32, device=device)
    _check("prac_gaussian", lib.prac_gaussian(seed, draw_counter, d, r, out.data_ptr(), r, _stream()))
    return out


class Basis:
    """A fitted (or to-be-fitted) pair U, Q with its scale c, for one saved input."""

    def __init__(self, d: int, k: int, r: int, dtype: torch.dtype = torch.bfloat16,
                 oversample: int = 0, iters: int = 0, device="cuda"):
        self.params = PracParams(d, k, r, _dtype_code(dtype), oversample, iters, 0)
        self.d, self.k, self.r, self.s = d, k, r, k + r
        self.dtype = dtype
        self.device = torch.device(device)
        nbytes = lib.prac_basis_bytes(ctypes.byref(self.params))
        if nbytes == 0:
            raise PracError("prac_basis_bytes", PRAC_EINVAL)
        self.storage = _buffer(nbytes, self.device)
        handle = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check("prac_basis_create",
                   lib.prac_basis_create(ctypes.byref(handle), ctypes.byref(self.params),
                                         self.storage.data_ptr(), self.storage.numel()))
        self.handle = handle
        self._ws: Optional[torch.Tensor] = None

    def __del__(self):
        h = getattr(self, "handle", None)
        if h and lib is not None:       # at interpreter shutdown the module globals may be gone already
            lib.prac_basis_destroy(h)
            self.handle = None

    # -- workspaces -------------------------------------------------------------------
    def _workspace(self, nbytes: int) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = _buffer(nbytes, self.device)
        return self._ws

    def fit_workspace_bytes(self, N: int) -> int:
        return lib.prac_fit_workspace_bytes(ctypes.byref(self.params), N)

    def grad_workspace_bytes(self, N: int, d_out: int) -> int:
        return lib.prac_grad_workspace_bytes(ctypes.byref(self.params), N, d_out)

    # -- Algorithm 1 ------------------------------------------------------------------
    def fit(self, X: torch.Tensor, seed: int, draw_counter: int = 0, ws: Optional[torch.Tensor] = None):
        ptr, ld = _mat(X, "X")
        ws = ws if ws is not None else self._workspace(self.fit_workspace_bytes(X.shape[0]))
        _check("prac_fit_basis", lib.prac_fit_basis(self.handle, ptr, X.shape[0], ld, seed, draw_counter,
                                                    ws.data_ptr(), ws.numel(), _stream()))

    def fit_principal(self, X: torch.Tensor, seed: int = 0, draw_counter: int = 0,
                      ws: Optional[torch.Tensor] = None):
        ptr, ld = _mat(X, "X")
        ws = ws if ws is not None else self._workspace(self.fit_workspace_bytes(X.shape[0]))
        _check("prac_fit_principal", lib.prac_fit_principal(self.handle, ptr, X.shape[0], ld, seed, draw_counter,
                                                            ws.data_ptr(), ws.numel(), _stream()))

    def refresh_principal(self, X: torch.Tensor, seed: int = 0, draw_counter: int = 0, iters: int = 2,
                          ws: Optional[torch.Tensor] = None):
        ptr, ld = _mat(X, "X")
        ws = ws if ws is not None else self._workspace(self.fit_workspace_bytes(X.shape[0]))
        _check("prac_refresh_principal",
               lib.prac_refresh_principal(self.handle, ptr, X.shape[0], ld, seed, draw_counter, iters,
                                          ws.data_ptr(), ws.numel(), _stream()))

    def draw_random(self, seed: int, draw_counter: int = 0, ws: Optional[torch.Tensor] = None):
        ws = ws if ws is not None else self._workspace(self.fit_workspace_bytes(1))
        _check("prac_draw_random", lib.prac_draw_random(self.handle, seed, draw_counter, ws.data_ptr(),
                                                        ws.numel(), _stream()))

    def set(self, U: Optional[torch.Tensor], Q: Optional[torch.Tensor], c: float):
        up, uld = _mat(U, "U") if U is not None and self.k > 0 else (None, 0)
        qp, qld = _mat(Q, "Q") if Q is not None and self.r > 0 else (None, 0)
        _check("prac_set_basis", lib.prac_set_basis(self.handle, up, uld, qp, qld, float(c), _stream()))

    def get(self) -> Tuple[torch.Tensor, torch.Tensor, float]:
        """Copies of U (d x k), Q (d x r) as fp32 tensors, and c."""
        P, c = self.projection()
        return P[:, :self.k].clone(), P[:, self.k:].clone(), c

    def projection(self) -> Tuple[torch.Tensor, float]:
        """A view of the library-owned fp32 P = [U | Q] (d x (k+r)), and c."""
        p = ctypes.c_void_p()
        ld = ctypes.c_int64()
        c = ctypes.c_double()
        _check("prac_basis_get", lib.prac_basis_get(self.handle, ctypes.byref(p), ctypes.byref(ld), ctypes.byref(c)))
        off = p.value - self.storage.data_ptr()
        view = self.storage[off:off + self.d * ld.value * 4].view(torch.float32).view(self.d, ld.value)
        return view[:, :self.s], c.value

    @property
    def c(self) -> float:
        return self.projection()[1]

    # -- Algorithm 1 "Compression", Algorithm 2 backward --------------------------------
    def compress(self, X: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        ptr, ld = _mat(X, "X")
        N = X.shape[0]
        if out is None:
            ldz = (self.s + 7) // 8 * 8
            out = torch.empty(N, ldz, dtype=self.dtype, device=X.device)[:, :self.s]
        zp, ldz = _mat(out, "Z")
        _check("prac_compress", lib.prac_compress(self.handle, ptr, N, ld, zp, ldz, _stream()))
        return out

    def linear_forward(self, X: torch.Tensor, W: torch.Tensor, out_y: Optional[torch.Tensor] = None,
                       out_z: Optional[torch.Tensor] = None, want_z: bool = True):
        """Algorithm 2 forward of one linear: (Y, Z) = (X W^T, X [U|Q]) with X read once.
        want_z=False computes Y only and returns (Y, None)."""
        xp, ldx = _mat(X, "X")
        wp, ldw = _mat(W, "W")
        N, d_out = X.shape[0], W.shape[0]
        if out_y is None:
            ldy = (d_out + 7) // 8 * 8
            out_y = torch.empty(N, ldy, dtype=self.dtype, device=X.device)[:, :d_out]
        if out_z is None and want_z:
            ldz = (self.s + 7) // 8 * 8
            out_z = torch.empty(N, ldz, dtype=self.dtype, device=X.device)[:, :self.s]
        yp, ldy = _mat(out_y, "Y")
        zp, ldz = _mat(out_z, "Z") if want_z else (None, 0)
        _check("prac_linear_forward",
               lib.prac_linear_forward(self.handle, xp, N, ldx, wp, ldw, d_out, yp, ldy, zp, ldz, _stream()))
        return out_y, (out_z if want_z else None)

    def activation_backward(self, Z: torch.Tensor, dY: torch.Tensor, act: str = "silu",
                            out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Section 5.1, non-linear layers: dX = dY * f'(X^) for f = "silu" or "gelu", X^ rebuilt from Z."""
        zp, ldz = _mat(Z, "Z")
        yp, ldy = _mat(dY, "dY")
        N = dY.shape[0]
        if out is None:
            ldx = (self.d + 7) // 8 * 8
            out = torch.empty(N, ldx, dtype=self.dtype, device=dY.device)[:, :self.d]
        xp, ldx = _mat(out, "dX")
        nbytes = lib.prac_activation_workspace_bytes(ctypes.byref(self.params), N)
        if nbytes and ws is None:
            ws = self._workspace(nbytes)
        _check("prac_activation_backward",
               lib.prac_activation_backward(self.handle, zp, ldz, yp, ldy, N, {"silu": 0, "gelu": 1}[act], xp, ldx,
                                            ws.data_ptr() if ws is not None else None,
                                            ws.numel() if ws is not None else 0, _stream()))
        return out

    # -- token-sharded batches: per-rank parts and the steps that follow their sum -----------
    def gram(self, X: torch.Tensor, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
        """C = X^T X (d x d fp32) of this rank's tokens."""
        ptr, ld = _mat(X, "X")
        N = X.shape[0]
        C = torch.empty(self.d, self.d, dtype=torch.float32, device=X.device)
        ws = ws if ws is not None else self._workspace(self.fit_workspace_bytes(N))
        _check("prac_gram", lib.prac_gram(self.handle, ptr, N, ld, C.data_ptr(), self.d, ws.data_ptr(), ws.numel(), _stream()))
        return C

    def fit_principal_gram(self, C: torch.Tensor, seed: int = 0, draw_counter: int = 0,
                           ws: Optional[torch.Tensor] = None) -> None:
        if C.dtype != torch.float32 or C.shape != (self.d, self.d) or C.stride(1) != 1:
            raise ValueError("C must be a d x d float32 matrix with contiguous rows")
        ws = ws if ws is not None else self._workspace(self.fit_workspace_bytes(1))
        _check("prac_fit_principal_gram",
               lib.prac_fit_principal_gram(self.handle, C.data_ptr(), C.stride(0), seed, draw_counter,
                                           ws.data_ptr(), ws.numel(), _stream()))

    def weight_grad_partial(self, dY: torch.Tensor, Z: torch.Tensor, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
        """M = dY^T Z (d_out x (k+r) fp32, unscaled) of this rank's tokens."""
        yp, ldy = _mat(dY, "dY")
        zp, ldz = _mat(Z, "Z")
        N, d_out = dY.shape
        M = torch.empty(d_out, self.s, dtype=torch.float32, device=dY.device)
        ws = ws if ws is not None else self._workspace(self.grad_workspace_bytes(N, d_out))
        _check("prac_weight_grad_partial",
               lib.prac_weight_grad_partial(self.handle, yp, ldy, d_out, zp, ldz, N, M.data_ptr(), self.s,
                                            ws.data_ptr(), ws.numel(), _stream()))
        return M

    def weight_grad_finish(self, M: torch.Tensor, out: Optional[torch.Tensor] = None,
                           out_dtype: torch.dtype = torch.float32, accumulate: bool = False,
                           c: float = math.nan, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
        if M.dtype != torch.float32 or M.shape[1] != self.s or M.stride(1) != 1:
            raise ValueError("M must be d_out x (k+r) float32 with contiguous rows")
        d_out = M.shape[0]
        if out is None:
            out = torch.empty(d_out, self.d, dtype=out_dtype, device=M.device)
        wp, ldw = _mat(out, "dW")
        ws = ws if ws is not None else self._workspace(d_out * ((self.s + 7) // 8 * 8) * 2 + 256)
        _check("prac_weight_grad_finish",
               lib.prac_weight_grad_finish(self.handle, M.data_ptr(), M.stride(0), d_out, float(c), wp, ldw,
                                           _dtype_code(out.dtype), int(accumulate), ws.data_ptr(), ws.numel(), _stream()))
        return out

    def rmsnorm_backward(self, Z: torch.Tensor, dY: torch.Tensor, rstd: torch.Tensor, gain: torch.Tensor,
                         out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None):
        """Section 5.1, non-linear layers: (dX, dgain) of y = gain * x * rstd with x rebuilt from Z."""
        zp, ldz = _mat(Z, "Z")
        yp, ldy = _mat(dY, "dY")
        N = dY.shape[0]
        if rstd.dtype != torch.float32 or gain.dtype != torch.float32 or not rstd.is_contiguous() or not gain.is_contiguous():
            raise ValueError("rstd and gain must be contiguous float32")
        if rstd.numel() != N or gain.numel() != self.d:
            raise ValueError("rstd has one entry per token, gain one per feature")
        if out is None:
            ldx = (self.d + 7) // 8 * 8
            out = torch.empty(N, ldx, dtype=self.dtype, device=dY.device)[:, :self.d]
        xp, ldx = _mat(out, "dX")
        dgain = torch.empty(self.d, dtype=torch.float32, device=dY.device)
        nbytes = lib.prac_rmsnorm_workspace_bytes(ctypes.byref(self.params), N)
        ws = ws if ws is not None else self._workspace(nbytes)
        _check("prac_rmsnorm_backward",
               lib.prac_rmsnorm_backward(self.handle, zp, ldz, yp, ldy, N, rstd.data_ptr(), gain.data_ptr(), xp, ldx,
                                         dgain.data_ptr(), ws.data_ptr(), ws.numel(), _stream()))
        return out, dgain

    def layernorm_backward(self, Z: torch.Tensor, dY: torch.Tensor, mean: torch.Tensor, rstd: torch.Tensor,
                           gain: torch.Tensor, out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None):
        """Section 5.1, non-linear layers: (dX, dgain, dbias) of LayerNorm with x rebuilt from Z."""
        zp, ldz = _mat(Z, "Z")
        yp, ldy = _mat(dY, "dY")
        N = dY.shape[0]
        for v, n, what in ((mean, N, "mean"), (rstd, N, "rstd"), (gain, self.d, "gain")):
            if v.dtype != torch.float32 or not v.is_contiguous() or v.numel() != n:
                raise ValueError(f"{what} must be contiguous float32 of length {n}")
        if out is None:
            ldx = (self.d + 7) // 8 * 8
            out = torch.empty(N, ldx, dtype=self.dtype, device=dY.device)[:, :self.d]
        xp, ldx = _mat(out, "dX")
        dgain = torch.empty(self.d, dtype=torch.float32, device=dY.device)
        dbias = torch.empty(self.d, dtype=torch.float32, device=dY.device)
        nbytes = lib.prac_layernorm_workspace_bytes(ctypes.byref(self.params), N)
        ws = ws if ws is not None else self._workspace(nbytes)
        _check("prac_layernorm_backward",
               lib.prac_layernorm_backward(self.handle, zp, ldz, yp, ldy, N, mean.data_ptr(), rstd.data_ptr(),
                                           gain.data_ptr(), xp, ldx, dgain.data_ptr(), dbias.data_ptr(),
                                           ws.data_ptr(), ws.numel(), _stream()))
        return out, dgain, dbias

    def weight_grad(self, dY: torch.Tensor, Z: torch.Tensor, out: Optional[torch.Tensor] = None,
                    out_dtype: torch.dtype = torch.float32, accumulate: bool = False,
                    c: float = math.nan, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
        yp, ldy = _mat(dY, "dY")
        zp, ldz = _mat(Z, "Z")
        N, d_out = dY.shape
        if out is None:
            out = torch.empty(d_out, self.d, dtype=out_dtype, device=dY.device)
        wp, ldw = _mat(out, "dW")
        ws = ws if ws is not None else self._workspace(self.grad_workspace_bytes(N, d_out))
        _check("prac_weight_grad",
               lib.prac_weight_grad(self.handle, yp, ldy, d_out, zp, ldz, N, float(c), wp, ldw,
                                    _dtype_code(out.dtype), int(accumulate), ws.data_ptr(), ws.numel(), _stream()))
        return out

    def weight_grad_static(self, dY: torch.Tensor, Z: torch.Tensor, out: torch.Tensor,
                           accumulate: bool = False, c: float = math.nan) -> torch.Tensor:
        """prac_weight_grad_static: same gradient, scratch taken from the library's fixed device
        array instead of a workspace (for callers that cannot allocate).  `out` must exist: this
        wrapper allocates nothing either."""
        yp, ldy = _mat(dY, "dY")
        zp, ldz = _mat(Z, "Z")
        wp, ldw = _mat(out, "dW")
        N, d_out = dY.shape
        _check("prac_weight_grad_static",
               lib.prac_weight_grad_static(self.handle, yp, ldy, d_out, zp, ldz, N, float(c), wp, ldw,
                                           _dtype_code(out.dtype), int(accumulate), _stream()))
        return out

    def reconstruct(self, Z: torch.Tensor) -> torch.Tensor:
        zp, ldz = _mat(Z, "Z")
        N = Z.shape[0]
        out = torch.empty(N, self.d, dtype=torch.float32, device=Z.device)
        _check("prac_reconstruct", lib.prac_reconstruct(self.handle, zp, ldz, N, out.data_ptr(), self.d, _stream()))
        return out

    def fit_report(self, N: int, ws: Optional[torch.Tensor] = None) -> dict:
        """prac_fit_report for the workspace of the last fit (default: this object's own)."""
        ws = ws if ws is not None else self._ws
        info = PracFitInfo()
        _check("prac_fit_report", lib.prac_fit_report(self.handle, ws.data_ptr() if ws is not None else None,
                                                      ws.numel() if ws is not None else 0, N, _stream(),
                                                      ctypes.byref(info)))
        return {f: getattr(info, f) for f, _ in PracFitInfo._fields_ if f != "reserved"}

    def status(self) -> int:
        """Waits for the current stream; returns the (cleared) device status code."""
        return lib.prac_device_status(self.handle, _stream())


def schedule_actions(t: int, T1: int, T2: int, fitted: bool) -> Tuple[Optional[str], bool]:
    """What Algorithm 1's lazy update does at training step t, as (principal, draw):
    principal = "fit" (first use: no U yet), "refresh" (t a multiple of T1: warm-started update of
    U) or None; draw = whether Q is redrawn (t a multiple of T2, and always when U changed, because
    a Q drawn against the old U is not orthogonal to the new one)."""
    if T1 < 1 or T2 < 1:
        raise ValueError("update intervals must be >= 1")
    principal = "fit" if not fitted else ("refresh" if t % T1 == 0 else None)
    draw = principal is not None or t % T2 == 0
    return principal, draw


class LazyCompressor:
    """Algorithm 1 as a stateful wrapper around one Basis: `compress(t, X)` refreshes U every T1
    steps and Q every T2 steps, then stores Z = X [U | Q].  The draw counter is the step number, so
    a run is reproducible from (seed, t)."""

    def __init__(self, basis: Basis, T1: int, T2: int, seed: int, warm_iters: int = 2):
        schedule_actions(0, T1, T2, False)
        self.basis, self.T1, self.T2, self.seed, self.warm_iters = basis, T1, T2, seed, warm_iters
        self.fitted = False
        self.log = []          # (t, principal action, drew) per call

    def compress(self, t: int, X: torch.Tensor, out: Optional[torch.Tensor] = None,
                 ws: Optional[torch.Tensor] = None) -> torch.Tensor:
        principal, draw = schedule_actions(t, self.T1, self.T2, self.fitted)
        if principal == "fit":
            self.basis.fit_principal(X, seed=self.seed, draw_counter=t, ws=ws)
            self.fitted = True
        elif principal == "refresh":
            self.basis.refresh_principal(X, seed=self.seed, draw_counter=t, iters=self.warm_iters, ws=ws)
        if draw:
            self.basis.draw_random(seed=self.seed, draw_counter=t, ws=ws)
        self.log.append((t, principal, draw))
        return self.basis.compress(X, out=out)
