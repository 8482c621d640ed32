"""Python binding of ``libslope.so`` -- argument marshalling only.

Each function has the name of the C entry point it calls (``include/slope.h``), takes
torch CUDA tensors (bf16 / uint8 / int16 / float32 storage, contiguous) and launches
on torch's current stream.  Nothing is computed here; if the library is missing the
import of this module's functions fails loudly -- there is no fallback.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional

import torch

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libslope.so"
_lib: Optional[ctypes.CDLL] = None

SLOPE_OK = 0
STATUS_NAMES = {0: "SLOPE_OK", 1: "SLOPE_ERR_INVALID_ARG", 2: "SLOPE_ERR_SHAPE", 3: "SLOPE_ERR_ALIGNMENT",
                4: "SLOPE_ERR_UNSUPPORTED_ARCH", 5: "SLOPE_ERR_CUDA", 6: "SLOPE_ERR_TIMEOUT"}

# every symbol include/slope.h declares
EXPORTS = (
    "slope_values_bytes", "slope_meta_bytes", "slope_mask_bytes",
    "slope_prune_24", "slope_double_prune", "slope_linear_fwd", "slope_linear_bwd_dx",
    "slope_linear_bwd_dw_masked", "slope_adapter_workspace_bytes", "slope_adapter_fwd_bwd",
    "slope_meta_to_canonical", "slope_poll_status", "slope_launch_count", "slope_status_string",
    "slope_adapter_dl_noalloc", "slope_adapter_dl_noalloc_max_scratch_bytes",
    "slope_sparse_add", "slope_update_sparse_matrix", "slope_selftest_wait_timeout",
    "slope_prune_nm", "slope_double_prune_nm", "slope_apply_mask",
    "slope_dense_linear_fwd", "slope_dense_linear_bwd_dx", "slope_dense_linear_bwd_dw", "slope_mask_difference",
    "slope_linear_fwd_adapter", "slope_prune_24_double",
    "slope_bwd_dw_adapter_workspace_bytes", "slope_linear_bwd_dw_adapter", "slope_kernel_clock_mhz",
)


class SlopeError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        super().__init__(f"{call} returned {STATUS_NAMES.get(status, status)}")


def lib() -> ctypes.CDLL:
    """Load libslope.so (built by ``build.build()``); raises if it is not there."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2608_24070_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(str(_LIB_PATH))
        vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        for name in ("slope_values_bytes", "slope_meta_bytes", "slope_mask_bytes"):
            getattr(L, name).restype = sz
            getattr(L, name).argtypes = [ci, ci]
        L.slope_prune_24.argtypes = [vp, ci, ci, vp, vp, vp, vp]
        L.slope_double_prune.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp]
        L.slope_prune_24_double.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp, vp, vp]
        L.slope_prune_24_double.restype = ci
        L.slope_bwd_dw_adapter_workspace_bytes.restype = sz
        L.slope_bwd_dw_adapter_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.slope_linear_bwd_dw_adapter.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, vp, vp, vp, sz, vp]
        L.slope_linear_bwd_dw_adapter.restype = ci
        L.slope_linear_fwd.argtypes = [vp, ci, vp, vp, ci, ci, vp, vp, ci, vp, vp]
        L.slope_linear_bwd_dx.argtypes = [vp, ci, vp, vp, ci, ci, vp, vp, ci, vp, vp]
        L.slope_linear_fwd_adapter.argtypes = [vp, ci, vp, vp, ci, ci, vp, vp, ci, vp, vp, vp]
        L.slope_linear_fwd_adapter.restype = ci
        L.slope_linear_bwd_dw_masked.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp]
        L.slope_adapter_workspace_bytes.restype = sz
        L.slope_adapter_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.slope_adapter_fwd_bwd.argtypes = [ci, vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, vp, vp, vp, sz, vp]
        L.slope_meta_to_canonical.argtypes = [vp, ci, ci, vp, vp]
        L.slope_adapter_dl_noalloc.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        L.slope_adapter_dl_noalloc.restype = ci
        L.slope_adapter_dl_noalloc_max_scratch_bytes.restype = sz
        L.slope_adapter_dl_noalloc_max_scratch_bytes.argtypes = []
        L.slope_sparse_add.argtypes = [vp, vp, ctypes.c_float, ctypes.c_float, ci, ci, vp, vp]
        L.slope_sparse_add.restype = ci
        L.slope_update_sparse_matrix.argtypes = [vp, vp, vp, ci, ci, vp, vp]
        L.slope_update_sparse_matrix.restype = ci
        L.slope_dense_linear_fwd.argtypes = [vp, ci, vp, ci, ci, vp, vp]
        L.slope_dense_linear_bwd_dx.argtypes = [vp, ci, vp, ci, ci, vp, vp]
        L.slope_dense_linear_bwd_dw.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        for name in ("slope_dense_linear_fwd", "slope_dense_linear_bwd_dx", "slope_dense_linear_bwd_dw"):
            getattr(L, name).restype = ci
        L.slope_mask_difference.argtypes = [vp, vp, ci, ci, vp, vp]
        L.slope_mask_difference.restype = ci
        L.slope_prune_nm.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp]
        L.slope_prune_nm.restype = ci
        L.slope_double_prune_nm.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp, vp]
        L.slope_double_prune_nm.restype = ci
        L.slope_apply_mask.argtypes = [vp, vp, ci, ci, vp, vp]
        L.slope_apply_mask.restype = ci
        L.slope_selftest_wait_timeout.argtypes = [ctypes.c_uint, vp, vp]
        L.slope_selftest_wait_timeout.restype = ci
        L.slope_poll_status.argtypes = [vp]
        L.slope_kernel_clock_mhz.argtypes = [ci, vp, ctypes.POINTER(ctypes.c_double)]
        L.slope_kernel_clock_mhz.restype = ci
        L.slope_launch_count.restype = ctypes.c_ulonglong
        L.slope_status_string.restype = ctypes.c_char_p
        L.slope_status_string.argtypes = [ci]
        for name in ("slope_prune_24", "slope_double_prune", "slope_linear_fwd", "slope_linear_bwd_dx",
                     "slope_linear_bwd_dw_masked", "slope_adapter_fwd_bwd", "slope_meta_to_canonical",
                     "slope_poll_status"):
            getattr(L, name).restype = ci
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    """Device address as a plain int (the argtypes make a void* of it); None stays NULL."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return t.data_ptr()


# torch's raw-stream getter skips building a Stream object (about 1.5 us per call, which is a
# sixth of a whole small-layer call); the public API is the fallback where it is missing.
_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream():
    if _raw_stream is not None:
        return _raw_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


def _check(call: str, status: int):
    if status != SLOPE_OK:
        raise SlopeError(call, status)


def slope_values_bytes(rows: int, cols: int) -> int:
    return int(lib().slope_values_bytes(rows, cols))


def slope_meta_bytes(rows: int, cols: int) -> int:
    return int(lib().slope_meta_bytes(rows, cols))


def slope_mask_bytes(rows: int, cols: int) -> int:
    return int(lib().slope_mask_bytes(rows, cols))


def slope_prune_24(W, Wc_vals, Wc_meta, mask1_bits=None):
    d_out, d_in = W.shape
    _check("slope_prune_24", lib().slope_prune_24(_ptr(W), d_out, d_in, _ptr(Wc_vals), _ptr(Wc_meta),
                                                  _ptr(mask1_bits), _stream()))


def slope_double_prune(W, mask1_bits, WTc_vals, WTc_meta, mask2_bits=None):
    d_out, d_in = W.shape
    _check("slope_double_prune", lib().slope_double_prune(_ptr(W), _ptr(mask1_bits), d_out, d_in, _ptr(WTc_vals),
                                                          _ptr(WTc_meta), _ptr(mask2_bits), _stream()))


def slope_prune_24_double(W, Wc_vals, Wc_meta, mask1_bits, WTc_vals, WTc_meta, mask2_bits=None):
    d_out, d_in = W.shape
    _check("slope_prune_24_double", lib().slope_prune_24_double(_ptr(W), d_out, d_in, _ptr(Wc_vals), _ptr(Wc_meta),
                                                                _ptr(mask1_bits), _ptr(WTc_vals), _ptr(WTc_meta),
                                                                _ptr(mask2_bits), _stream()))


def slope_linear_fwd(X, Wc_vals, Wc_meta, d_out, Y, T=None, R=None):
    b, d_in = X.shape
    r = 0 if T is None else T.shape[1]
    _check("slope_linear_fwd", lib().slope_linear_fwd(_ptr(X), b, _ptr(Wc_vals), _ptr(Wc_meta), d_out, d_in,
                                                      _ptr(T), _ptr(R), r, _ptr(Y), _stream()))


def slope_linear_fwd_adapter(X, Wc_vals, Wc_meta, d_out, L, R, T, Y):
    """T = X L and Y = X (W^R)^T + T R in one call (a fused pair of launches at inference sizes)."""
    b, d_in = X.shape
    _check("slope_linear_fwd_adapter", lib().slope_linear_fwd_adapter(
        _ptr(X), b, _ptr(Wc_vals), _ptr(Wc_meta), d_out, d_in, _ptr(L), _ptr(R), L.shape[1], _ptr(T), _ptr(Y),
        _stream()))


def slope_linear_bwd_dx(dY, WTc_vals, WTc_meta, d_in, dX, dT=None, L=None):
    b, d_out = dY.shape
    r = 0 if dT is None else dT.shape[1]
    _check("slope_linear_bwd_dx", lib().slope_linear_bwd_dx(_ptr(dY), b, _ptr(WTc_vals), _ptr(WTc_meta), d_out, d_in,
                                                            _ptr(dT), _ptr(L), r, _ptr(dX), _stream()))


def slope_linear_bwd_dw_masked(dY, X, mask1_bits, dWc_vals):
    b, d_out = dY.shape
    d_in = X.shape[1]
    _check("slope_linear_bwd_dw_masked", lib().slope_linear_bwd_dw_masked(_ptr(dY), _ptr(X), b, d_out, d_in,
                                                                          _ptr(mask1_bits), _ptr(dWc_vals), _stream()))


def slope_bwd_dw_adapter_workspace_bytes(b: int, d_out: int, d_in: int, r: int) -> int:
    return int(lib().slope_bwd_dw_adapter_workspace_bytes(b, d_out, d_in, r))


def slope_linear_bwd_dw_adapter(dY, X, T, dT, mask1_bits, dWc_vals, dL, dR, workspace):
    b, d_out = dY.shape
    d_in, r = X.shape[1], T.shape[1]
    _check("slope_linear_bwd_dw_adapter", lib().slope_linear_bwd_dw_adapter(
        _ptr(dY), _ptr(X), _ptr(T), _ptr(dT), b, d_out, d_in, r, _ptr(mask1_bits), _ptr(dWc_vals), _ptr(dL), _ptr(dR),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()))


def slope_kernel_clock_mhz(kind: int) -> float:
    """Mean SM clock (MHz) inside the sparse (kind 0) / dense CTA-pair (kind 1) tile-kernel launches
    since the previous call for that kind."""
    mhz = ctypes.c_double(0.0)
    _check("slope_kernel_clock_mhz", lib().slope_kernel_clock_mhz(int(kind), _stream(), ctypes.byref(mhz)))
    return float(mhz.value)


def slope_adapter_workspace_bytes(b: int, d_out: int, d_in: int, r: int) -> int:
    return int(lib().slope_adapter_workspace_bytes(b, d_out, d_in, r))


def slope_adapter_fwd_bwd(phase, X, dY, L, R, b, d_out, d_in, r, T=None, dT=None, dL=None, dR=None, workspace=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("slope_adapter_fwd_bwd", lib().slope_adapter_fwd_bwd(
        phase, _ptr(X), _ptr(dY), _ptr(L), _ptr(R), b, d_out, d_in, r, _ptr(T), _ptr(dT), _ptr(dL), _ptr(dR),
        _ptr(workspace), ws_bytes, _stream()))


def slope_adapter_dl_noalloc(X, dT, dL):
    """dL = X^T dT with the split-K scratch in the library's fixed device array (no allocation,
    no workspace argument).  For callers that are not allowed to allocate GPU memory."""
    b, d_in = X.shape
    r = dT.shape[1]
    _check("slope_adapter_dl_noalloc", lib().slope_adapter_dl_noalloc(_ptr(X), _ptr(dT), b, d_in, r, _ptr(dL),
                                                                      _stream()))


def slope_adapter_dl_noalloc_max_scratch_bytes() -> int:
    return int(lib().slope_adapter_dl_noalloc_max_scratch_bytes())


def slope_sparse_add(A_vals, B_vals, beta, gamma, out_vals):
    rows, half = A_vals.shape
    _check("slope_sparse_add", lib().slope_sparse_add(_ptr(A_vals), _ptr(B_vals), float(beta), float(gamma), rows,
                                                      half * 2, _ptr(out_vals), _stream()))


def slope_update_sparse_matrix(Wc_vals, mask1_bits, WTc_meta, WTc_vals):
    d_out, half = Wc_vals.shape
    _check("slope_update_sparse_matrix", lib().slope_update_sparse_matrix(
        _ptr(Wc_vals), _ptr(mask1_bits), _ptr(WTc_meta), d_out, half * 2, _ptr(WTc_vals), _stream()))


def slope_dense_linear_fwd(X, W, Y):
    (b, d_in), d_out = X.shape, W.shape[0]
    _check("slope_dense_linear_fwd", lib().slope_dense_linear_fwd(_ptr(X), b, _ptr(W), d_out, d_in, _ptr(Y), _stream()))


def slope_dense_linear_bwd_dx(dY, W, dX):
    (b, d_out), d_in = dY.shape, W.shape[1]
    _check("slope_dense_linear_bwd_dx", lib().slope_dense_linear_bwd_dx(_ptr(dY), b, _ptr(W), d_out, d_in, _ptr(dX),
                                                                        _stream()))


def slope_dense_linear_bwd_dw(dY, X, dW):
    (b, d_out), d_in = dY.shape, X.shape[1]
    _check("slope_dense_linear_bwd_dw", lib().slope_dense_linear_bwd_dw(_ptr(dY), _ptr(X), b, d_out, d_in, _ptr(dW),
                                                                        _stream()))


def slope_mask_difference(mask_a, mask_b, count_out):
    rows, mrow = mask_a.shape
    _check("slope_mask_difference", lib().slope_mask_difference(_ptr(mask_a), _ptr(mask_b), rows, mrow * 8,
                                                                _ptr(count_out), _stream()))


def slope_prune_nm(W, n, m, W_R, mask1_bits=None):
    d_out, d_in = W.shape
    _check("slope_prune_nm", lib().slope_prune_nm(_ptr(W), d_out, d_in, int(n), int(m), _ptr(W_R), _ptr(mask1_bits),
                                                  _stream()))


def slope_double_prune_nm(W, mask1_bits, n, m, W_RC, mask2_bits=None):
    d_out, d_in = W.shape
    _check("slope_double_prune_nm", lib().slope_double_prune_nm(_ptr(W), _ptr(mask1_bits), d_out, d_in, int(n), int(m),
                                                                _ptr(W_RC), _ptr(mask2_bits), _stream()))


def slope_apply_mask(G, mask_bits, out):
    d_out, d_in = G.shape
    _check("slope_apply_mask", lib().slope_apply_mask(_ptr(G), _ptr(mask_bits), d_out, d_in, _ptr(out), _stream()))


def slope_meta_to_canonical(meta_hw, rows, cols, meta_canon):
    _check("slope_meta_to_canonical", lib().slope_meta_to_canonical(_ptr(meta_hw), rows, cols, _ptr(meta_canon),
                                                                    _stream()))


def slope_selftest_wait_timeout(limit_us: int, gave_up_flag):
    _check("slope_selftest_wait_timeout", lib().slope_selftest_wait_timeout(int(limit_us), _ptr(gave_up_flag), _stream()))


def slope_poll_status() -> int:
    return int(lib().slope_poll_status(_stream()))


def slope_launch_count() -> int:
    return int(lib().slope_launch_count())


def slope_status_string(status: int) -> str:
    return lib().slope_status_string(status).decode()


# ------------------------------------------------------------------ small conveniences (allocation only)
def alloc_compressed(rows: int, cols: int, device="cuda"):
    """Caller-owned buffers of the compressed format of a [rows x cols] matrix."""
    vals = torch.empty((rows, cols // 2), dtype=torch.bfloat16, device=device)
    meta = torch.empty(slope_meta_bytes(rows, cols), dtype=torch.uint8, device=device)
    mask = torch.empty((rows, cols // 8), dtype=torch.uint8, device=device)
    return vals, meta, mask


def bf16_from_bits(bits, device="cuda") -> torch.Tensor:
    """numpy uint16 bit patterns -> torch bf16 tensor on `device` (bit copy)."""
    import numpy as np

    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device)
    return t.view(torch.bfloat16)


def bits_from_bf16(t: torch.Tensor):
    """torch bf16 tensor -> numpy uint16 bit patterns (bit copy)."""
    import numpy as np

    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
