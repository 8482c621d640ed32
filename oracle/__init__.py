"""CPU oracle for the SLoPe 2:4-sparse linear layer -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``slope_oracle.c`` (plain C, fp64).  Only the
tests, the smoke check and the benchmark's CPU-baseline / reference arm may
import this package; the CUDA library never does, and nothing here imports the
CUDA package.  bf16 tensors are numpy ``uint16`` arrays holding raw bit
patterns; results are ``float64`` (GEMMs) or integer arrays (selection).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "slope_oracle.c"
_LIB = _HERE / "libslope_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (-O2, OpenMP, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-std=c11", "-shared", "-fPIC", "-o", str(tmp), str(_SRC)]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.slope_oracle_max_threads.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 tensors travel as uint16 bit patterns"
    return a


def _u8(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint8
    return a


def _idx(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def max_threads() -> int:
    return int(_load().slope_oracle_max_threads())


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def prune24(W: np.ndarray):
    """O1: returns (vals[d_out,d_in/2] u16, nib[d_out,d_in/4] u8, mask1[d_out,d_in/8] u8)."""
    W = _u16(W)
    d_out, d_in = W.shape
    assert d_in % 8 == 0
    vals = np.empty((d_out, d_in // 2), np.uint16)
    nib = np.empty((d_out, d_in // 4), np.uint8)
    mask = np.empty((d_out, d_in // 8), np.uint8)
    _load().slope_oracle_prune24(_p(W), d_out, d_in, _p(vals), _p(nib), _p(mask))
    return vals, nib, mask


def double_prune(W: np.ndarray, mask1: np.ndarray):
    """O2: returns (valsT[d_in,d_out/2] u16, nibT[d_in,d_out/4] u8, mask2[d_out,d_in/8] u8)."""
    W = _u16(W)
    mask1 = _u8(mask1)
    d_out, d_in = W.shape
    assert d_out % 4 == 0 and mask1.shape == (d_out, d_in // 8)
    valsT = np.empty((d_in, d_out // 2), np.uint16)
    nibT = np.empty((d_in, d_out // 4), np.uint8)
    mask2 = np.empty((d_out, d_in // 8), np.uint8)
    _load().slope_oracle_double_prune(_p(W), _p(mask1), d_out, d_in, _p(valsT), _p(nibT), _p(mask2))
    return valsT, nibT, mask2


def pack_canonical(nib: np.ndarray) -> np.ndarray:
    nib = _u8(nib)
    rows, groups = nib.shape
    assert groups % 4 == 0
    canon = np.empty((rows, groups // 4), np.uint16)
    _load().slope_oracle_pack_canonical(_p(nib), rows, groups * 4, _p(canon))
    return canon


def canonical_to_hw(canon: np.ndarray) -> np.ndarray:
    canon = _u16(canon)
    rows, units = canon.shape
    cols = units * 16
    assert rows % 128 == 0 and cols % 128 == 0
    hw = np.zeros(rows * cols // 8, np.uint8)
    _load().slope_oracle_canonical_to_hw(_p(canon), rows, cols, _p(hw))
    return hw


def decompress(vals: np.ndarray, nib: np.ndarray) -> np.ndarray:
    vals = _u16(vals)
    nib = _u8(nib)
    rows = vals.shape[0]
    cols = vals.shape[1] * 2
    dense = np.empty((rows, cols), np.float64)
    _load().slope_oracle_decompress(_p(vals), _p(nib), rows, cols, _p(dense))
    return dense


def prune_nm(W: np.ndarray, n: int, m: int):
    """O9: general N:M first pass.  Returns (WR[d_out,d_in] u16 dense with +0 at pruned entries, mask1)."""
    W = _u16(W)
    d_out, d_in = W.shape
    assert 0 < n < m <= 64 and d_in % m == 0 and d_in % 8 == 0
    WR = np.empty((d_out, d_in), np.uint16)
    mask = np.empty((d_out, d_in // 8), np.uint8)
    _load().slope_oracle_prune_nm(_p(W), d_out, d_in, n, m, _p(WR), _p(mask))
    return WR, mask


def double_prune_nm(W: np.ndarray, mask1: np.ndarray, n: int, m: int):
    """O10: general N:M second pass along the columns.  Returns (WRC[d_out,d_in] u16 dense, mask2)."""
    W = _u16(W)
    mask1 = _u8(mask1)
    d_out, d_in = W.shape
    assert 0 < n < m <= 64 and d_out % m == 0 and mask1.shape == (d_out, d_in // 8)
    WRC = np.empty((d_out, d_in), np.uint16)
    mask2 = np.empty((d_out, d_in // 8), np.uint8)
    _load().slope_oracle_double_prune_nm(_p(W), _p(mask1), d_out, d_in, n, m, _p(WRC), _p(mask2))
    return WRC, mask2


def mask_difference(mask_a: np.ndarray, mask_b: np.ndarray) -> int:
    """O11: number of element positions in which two bit masks [rows, cols/8] differ."""
    mask_a, mask_b = _u8(mask_a), _u8(mask_b)
    assert mask_a.shape == mask_b.shape
    rows, mrow = mask_a.shape
    fn = _load().slope_oracle_mask_difference
    fn.restype = ctypes.c_longlong
    return int(fn(_p(mask_a), _p(mask_b), rows, mrow * 8))


def mask_to_bool(mask: np.ndarray, cols: int) -> np.ndarray:
    """Bit mask (LSB-first bytes) -> boolean [rows, cols]."""
    return np.unpackbits(np.asarray(mask, np.uint8), axis=1, bitorder="little")[:, :cols].astype(bool)


def _adapter(L, R, d_in, d_out):
    if L is None or R is None:
        z = np.zeros(1, np.uint16)
        return z, z, 0
    L = _u16(L)
    R = _u16(R)
    r = L.shape[1]
    assert L.shape == (d_in, r) and R.shape == (r, d_out)
    return L, R, r


def fwd_rows(X, W, mask1, rows, L=None, R=None) -> np.ndarray:
    """O3 for the listed token rows -> float64 [len(rows), d_out]."""
    X, W, mask1 = _u16(X), _u16(W), _u8(mask1)
    b, d_in = X.shape
    d_out = W.shape[0]
    L, R, r = _adapter(L, R, d_in, d_out)
    rows = _idx(rows)
    Y = np.empty((len(rows), d_out), np.float64)
    _load().slope_oracle_fwd_rows(_p(X), _p(W), _p(mask1), b, d_out, d_in, _p(L), _p(R), r,
                                  _p(rows), len(rows), _p(Y))
    return Y


def dx_rows(dY, W, mask2, rows, L=None, R=None) -> np.ndarray:
    """O4 for the listed token rows -> float64 [len(rows), d_in]."""
    dY, W, mask2 = _u16(dY), _u16(W), _u8(mask2)
    b, d_out = dY.shape
    d_in = W.shape[1]
    L, R, r = _adapter(L, R, d_in, d_out)
    rows = _idx(rows)
    dX = np.empty((len(rows), d_in), np.float64)
    _load().slope_oracle_dx_rows(_p(dY), _p(W), _p(mask2), b, d_out, d_in, _p(L), _p(R), r,
                                 _p(rows), len(rows), _p(dX))
    return dX


def dw_rows(dY, X, mask1, orows) -> np.ndarray:
    """O5 for the listed d_out rows -> float64 [len(orows), d_in/2] (compressed)."""
    dY, X, mask1 = _u16(dY), _u16(X), _u8(mask1)
    b, d_out = dY.shape
    d_in = X.shape[1]
    orows = _idx(orows)
    dWc = np.empty((len(orows), d_in // 2), np.float64)
    _load().slope_oracle_dw_rows(_p(dY), _p(X), _p(mask1), b, d_out, d_in, _p(orows), len(orows), _p(dWc))
    return dWc


def adapter_T_rows(X, L, rows) -> np.ndarray:
    X, L = _u16(X), _u16(L)
    b, d_in = X.shape
    r = L.shape[1]
    rows = _idx(rows)
    T = np.empty((len(rows), r), np.float64)
    _load().slope_oracle_adapter_T_rows(_p(X), _p(L), b, d_in, r, _p(rows), len(rows), _p(T))
    return T


def adapter_dT_rows(dY, R, rows) -> np.ndarray:
    dY, R = _u16(dY), _u16(R)
    b, d_out = dY.shape
    r = R.shape[0]
    rows = _idx(rows)
    dT = np.empty((len(rows), r), np.float64)
    _load().slope_oracle_adapter_dT_rows(_p(dY), _p(R), b, d_out, r, _p(rows), len(rows), _p(dT))
    return dT


def adapter_dL_rows(X, dY, R, jrows) -> np.ndarray:
    X, dY, R = _u16(X), _u16(dY), _u16(R)
    b, d_in = X.shape
    d_out = dY.shape[1]
    r = R.shape[0]
    jrows = _idx(jrows)
    dL = np.empty((len(jrows), r), np.float64)
    _load().slope_oracle_adapter_dL_rows(_p(X), _p(dY), _p(R), b, d_out, d_in, r, _p(jrows), len(jrows), _p(dL))
    return dL


def adapter_dR_cols(X, L, dY, icols) -> np.ndarray:
    X, L, dY = _u16(X), _u16(L), _u16(dY)
    b, d_in = X.shape
    d_out = dY.shape[1]
    r = L.shape[1]
    icols = _idx(icols)
    dR = np.empty((r, len(icols)), np.float64)
    _load().slope_oracle_adapter_dR_cols(_p(X), _p(L), _p(dY), b, d_out, d_in, r, _p(icols), len(icols), _p(dR))
    return dR


def sparse_add(A_vals, B_vals, beta: float, gamma: float) -> np.ndarray:
    """O7: beta*A + gamma*B on compressed value arrays of one pattern -> float64, same shape."""
    A_vals, B_vals = _u16(A_vals), _u16(B_vals)
    assert A_vals.shape == B_vals.shape
    out = np.empty(A_vals.shape, np.float64)
    lib = _load()
    lib.slope_oracle_sparse_add.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_double, ctypes.c_double,
                                            ctypes.c_long, ctypes.c_void_p]
    lib.slope_oracle_sparse_add(_p(A_vals), _p(B_vals), float(beta), float(gamma), A_vals.size, _p(out))
    return out


def update_transposed(Wc_new, mask1, mask2, nibT) -> np.ndarray:
    """O8: values of the compressed transposed double-pruned copy rebuilt from new forward values."""
    Wc_new, mask1, mask2, nibT = _u16(Wc_new), _u8(mask1), _u8(mask2), _u8(nibT)
    d_out, half = Wc_new.shape
    d_in = half * 2
    assert mask1.shape == (d_out, d_in // 8) and mask2.shape == mask1.shape and nibT.shape == (d_in, d_out // 4)
    valsT = np.empty((d_in, d_out // 2), np.uint16)
    _load().slope_oracle_update_transposed(_p(Wc_new), _p(mask1), _p(mask2), _p(nibT), d_out, d_in, _p(valsT))
    return valsT
