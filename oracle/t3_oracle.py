"""ctypes front end of the CPU oracle in ``t3_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by
the bench's CPU-baseline leg; the CUDA path never touches it.

The oracle is the definition of the path's result (paper Sections 2.3 and
2.4): per tensor-parallel slice r the partial product P_r = X_r . W_r over
that slice of the dot-product dimension, summed over r in fp64, viewed as R
reduce-scatter row chunks.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "t3_oracle.c")
_LIB = os.path.join(_HERE, "libt3_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile t3_oracle.c with gcc (OpenMP, no fp contraction)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call([
            "gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
            "-shared", "-fPIC", "-o", tmp, _SRC,
        ])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.t3_oracle_gemm_rs_bf16.argtypes = [p, p, i64, i64, i64, ctypes.c_int, p, i64, p, p]
        lib.t3_oracle_gemm_rs_bf16.restype = ctypes.c_int
        lib.t3_oracle_gemm_rs_f64.argtypes = [p, p, i64, i64, i64, ctypes.c_int, p, i64, p, p]
        lib.t3_oracle_gemm_rs_f64.restype = ctypes.c_int
        lib.t3_oracle_ring_sum_f32.argtypes = [p, i64, i64, ctypes.c_int, p]
        lib.t3_oracle_ring_sum_f32.restype = ctypes.c_int
        lib.t3_oracle_ring_order.argtypes = [ctypes.c_int, ctypes.c_int, p]
        lib.t3_oracle_ring_order.restype = None
        lib.t3_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """OpenMP threads the oracle will use."""
    return int(_load().t3_oracle_threads())


def ring_order(c: int, R: int) -> List[int]:
    """Order in which the ring adds the slices' partials of chunk c
    (Section 4.1/4.4 running example): [c-1, c-2, ..., c-R+1, c] mod R."""
    out = (ctypes.c_int * R)()
    _load().t3_oracle_ring_order(int(c), int(R), out)
    return list(out)


def _rows_arg(rows, M):
    if rows is None:
        return None, M, None
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    assert r.ndim == 1 and (r >= 0).all() and (r < M).all()
    return r, int(r.size), r.ctypes.data


def gemm_rs(x_bits: np.ndarray, w_kn_bits: np.ndarray, R: int,
            rows: Optional[Sequence[int]] = None, return_partials: bool = False):
    """fp64 Y = sum_r X_r . W_r from bf16 bit patterns.

    x_bits [M,K] uint16, w_kn_bits [K,N] uint16 (mathematical layout).
    rows: optional subset of output rows (spot checks at full size).
    Returns Y [n_rows,N] float64 (and P [R,n_rows,N] if asked).
    """
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    w = np.ascontiguousarray(w_kn_bits, dtype=np.uint16)
    M, K = x.shape
    K2, N = w.shape
    assert K == K2
    rkeep, n_rows, rptr = _rows_arg(rows, M)
    Y = np.empty((n_rows, N), dtype=np.float64)
    P = np.empty((R, n_rows, N), dtype=np.float64) if return_partials else None
    rc = _load().t3_oracle_gemm_rs_bf16(x.ctypes.data, w.ctypes.data, M, N, K, int(R), rptr, n_rows,
                                        Y.ctypes.data, P.ctypes.data if P is not None else None)
    if rc != 0:
        raise ValueError(f"oracle rejected arguments (rc={rc}): M={M} N={N} K={K} R={R}")
    return (Y, P) if return_partials else Y


def gemm_rs_f64(x: np.ndarray, w_kn: np.ndarray, R: int,
                rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Same definition on float64 inputs (no input rounding anywhere)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    w = np.ascontiguousarray(w_kn, dtype=np.float64)
    M, K = x.shape
    K2, N = w.shape
    assert K == K2
    rkeep, n_rows, rptr = _rows_arg(rows, M)
    Y = np.empty((n_rows, N), dtype=np.float64)
    rc = _load().t3_oracle_gemm_rs_f64(x.ctypes.data, w.ctypes.data, M, N, K, int(R), rptr, n_rows,
                                       Y.ctypes.data, None)
    if rc != 0:
        raise ValueError(f"oracle rejected arguments (rc={rc})")
    return Y


def ring_sum_f32(P: np.ndarray) -> np.ndarray:
    """Reduction stage alone in device arithmetic: sequential fp32 adds of the
    R partial arrays P [R,M,N] in each row chunk's ring order."""
    P = np.ascontiguousarray(P, dtype=np.float32)
    R, M, N = P.shape
    Y = np.empty((M, N), dtype=np.float32)
    rc = _load().t3_oracle_ring_sum_f32(P.ctypes.data, M, N, R, Y.ctypes.data)
    if rc != 0:
        raise ValueError(f"oracle rejected arguments (rc={rc})")
    return Y


def epilogue(Y: np.ndarray, bias: Optional[np.ndarray] = None, keep: Optional[np.ndarray] = None,
             keep_scale: float = 1.0, residual: Optional[np.ndarray] = None) -> np.ndarray:
    """The element-wise operators that follow the all-reduce, applied to the reduced array (Section 7.6:
    bias, dropout and residual add can run on each device's reduce-scattered chunk before the all-gather):

        out[m][n] = (Y[m][n] + bias[n]) * (keep_scale if keep[m][n] else 0) + residual[m][n]

    in fp64.  The dropout mask is an input (whoever drew it); a missing operand skips its step.
    Y [rows,N]; bias [N]; keep, residual [rows,N] (the same rows as Y)."""
    out = np.array(Y, dtype=np.float64, copy=True)
    if bias is not None:
        out = out + np.asarray(bias, dtype=np.float64)[None, :]
    if keep is not None:
        out = out * np.where(np.asarray(keep) != 0, np.float64(keep_scale), np.float64(0.0))
    if residual is not None:
        out = out + np.asarray(residual, dtype=np.float64)
    return out


def epilogue_f32(S: np.ndarray, bias: Optional[np.ndarray] = None, keep: Optional[np.ndarray] = None,
                 keep_scale: float = 1.0, residual: Optional[np.ndarray] = None) -> np.ndarray:
    """The same three steps in device arithmetic: each one a single fp32 operation rounded to nearest
    (add, multiply, add; nothing fused), on an fp32 sum S.  Lets a test check the fused tail bit for bit
    given the device's own reduced sum."""
    out = np.array(S, dtype=np.float32, copy=True)
    if bias is not None:
        out = (out + np.asarray(bias, dtype=np.float32)[None, :]).astype(np.float32)
    if keep is not None:
        out = (out * np.where(np.asarray(keep) != 0, np.float32(keep_scale), np.float32(0.0))).astype(np.float32)
    if residual is not None:
        out = (out + np.asarray(residual, dtype=np.float32)).astype(np.float32)
    return out


def chunks(Y: np.ndarray, R: int) -> List[np.ndarray]:
    """Reduce-scatter view (Section 2.3): chunk c = rows [c*M/R, (c+1)*M/R),
    the part device c owns after the collective."""
    M = Y.shape[0]
    assert M % R == 0
    cr = M // R
    return [Y[c * cr:(c + 1) * cr] for c in range(R)]


def max_rel_err(y: np.ndarray, y_ref: np.ndarray, rms: Optional[float] = None) -> float:
    """max_ij |y - y_ref| / max(|y_ref|, rms(y_ref)); NaN/Inf anywhere -> inf.

    The floor at the reference's rms keeps the measure defined at zeros and
    meaningful for elements far below the typical magnitude.  Pass `rms` when
    y_ref is only a row sample whose rms should come from elsewhere.
    """
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    if not np.isfinite(y).all():
        return float("inf")
    if rms is None:
        rms = float(np.sqrt(np.mean(y_ref * y_ref)))
    den = np.maximum(np.abs(y_ref), max(rms, 1e-300))
    return float(np.max(np.abs(y - y_ref) / den))
