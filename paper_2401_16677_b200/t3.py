"""ctypes binding of the C-ABI library (declared in include/t3.h).

The build makes ``libt3.so`` and, where its extra source file is present,
``libt3_sf.so`` (same ABI plus the 4-CTA-cluster kernel variant, whose W
fetches are TMA loads multicast to two CTA pairs).  That variant is for
single-process, single-GPU use only: the binding loads it when it exists AND
the process is not part of a multi-process launch (``WORLD_SIZE`` or
``LOCAL_WORLD_SIZE`` above 1); in such a launch it always loads ``libt3.so``,
whatever files exist and whatever ``T3_LIB_PATH`` says about the variant.

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Function names mirror the C names without the ``t3_`` prefix.
There is no fallback: if the shared library is missing or fails to load,
``lib()`` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PORTABLE = os.path.join(_HERE, "libt3.so")
_LIB_SF = os.path.join(_HERE, "libt3_sf.so")


def multi_process_launch(env=None) -> bool:
    """True when this process is one rank of a launch with more than one process."""
    env = os.environ if env is None else env
    for key in ("WORLD_SIZE", "LOCAL_WORLD_SIZE"):
        try:
            if int(env.get(key, "1")) > 1:
                return True
        except ValueError:
            return True          # unreadable: assume the cautious answer
    return False


def choose_lib_path(env=None) -> str:
    """The library this process may load.  The multicast variant is never chosen in a multi-process launch."""
    env = os.environ if env is None else env
    if multi_process_launch(env):
        return _LIB_PORTABLE
    override = env.get("T3_LIB_PATH")
    if override:
        return override
    return _LIB_SF if os.path.exists(_LIB_SF) else _LIB_PORTABLE


LIB_PATH = choose_lib_path()

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_DEVICE, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED, ERR_TOO_LARGE = \
    -1, -2, -3, -4, -5, -6, -7, -8
BF16_OUT_BF16, BF16_OUT_F32 = 0, 1
MODE_FUSED, MODE_SEQUENTIAL, MODE_GEMM_ONLY, MODE_REDUCE_ONLY = 0, 1, 2, 3
PARTIAL_F32, PARTIAL_BF16 = 0, 1
W_NK, W_KN = 0, 1
ORDER_GROUPED, ORDER_STAGGERED = 0, 1
REDUCE_RING, REDUCE_INPLACE = 0, 1
EPI_BF16, EPI_F32 = 0, 1
DEBUG_INFLATE_EXPECTED = 1

EXPORTS = [
    "t3_plan", "t3_gemm_rs", "t3_gemm_rs_mode", "t3_gemm_rs_ex", "t3_gemm_rs_host", "t3_gemm_rs_static", "t3_destroy",
    "t3_plan_info", "t3_plan_status", "t3_plan_tune", "t3_plan_timeline",
    "t3_plan_partials", "t3_plan_ring", "t3_plan_export_partials", "t3_geometry", "t3_schedule", "t3_reduce_schedule", "t3_ring_order",
    "t3_last_error", "t3_strerror", "t3_version", "t3_shared_fetch_available", "t3_abi_sizes",
]


class Chunking(ctypes.Structure):
    _fields_ = [
        ("mode", ctypes.c_int32), ("tile_n", ctypes.c_int32), ("group_tiles", ctypes.c_int32),
        ("reducer_ctas", ctypes.c_int32), ("reducer_warps", ctypes.c_int32), ("reduce_rows", ctypes.c_int32),
        ("stages", ctypes.c_int32), ("timeout_ms", ctypes.c_int32), ("debug_flags", ctypes.c_int32),
        ("max_ctas", ctypes.c_int32), ("ring_slots", ctypes.c_int32), ("cluster_ctas", ctypes.c_int32),
        ("partial_dtype", ctypes.c_int32), ("w_layout", ctypes.c_int32), ("order", ctypes.c_int32),
        ("reduce", ctypes.c_int32), ("split_k", ctypes.c_int32), ("l2_hints", ctypes.c_int32),
        ("reserved", ctypes.c_int32 * 2),
    ]


class Epilogue(ctypes.Structure):
    """t3_epilogue_t: element-wise work fused on the reduced chunk (device pointers; 0 = skip)."""
    _fields_ = [
        ("bias", ctypes.c_void_p), ("residual", ctypes.c_void_p), ("keep", ctypes.c_void_p),
        ("keep_scale", ctypes.c_float), ("bias_dtype", ctypes.c_int32), ("residual_dtype", ctypes.c_int32),
        ("reserved", ctypes.c_int32),
    ]


class Timeline(ctypes.Structure):
    _fields_ = [("total_us", ctypes.c_double), ("produce_us", ctypes.c_double), ("tail_us", ctypes.c_double),
                ("drain_us", ctypes.c_double), ("ctas", ctypes.c_int32), ("reserved", ctypes.c_int32)]

    def as_dict(self) -> dict:
        return {n: getattr(self, n) for n, _ in self._fields_ if n != "reserved"}


class Tune(ctypes.Structure):
    _fields_ = [("n_tried", ctypes.c_int32), ("chosen", ctypes.c_int32),
                ("mode", ctypes.c_int32 * 48), ("ring_slots", ctypes.c_int32 * 48), ("reduce_rows", ctypes.c_int32 * 48),
                ("cluster_ctas", ctypes.c_int32 * 48), ("group_tiles", ctypes.c_int32 * 48), ("us", ctypes.c_float * 48)]

    def candidates(self) -> list:
        return [dict(mode=self.mode[i], ring_slots=self.ring_slots[i], reduce_rows=self.reduce_rows[i],
                     cluster_ctas=self.cluster_ctas[i], group_tiles=self.group_tiles[i], us=float(self.us[i]))
                for i in range(self.n_tried)]


class Info(ctypes.Structure):
    _fields_ = [
        ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
        ("R", ctypes.c_int32), ("K_r", ctypes.c_int32), ("chunk_rows", ctypes.c_int32),
        ("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32),
        ("n_m_tiles", ctypes.c_int32), ("n_n_tiles", ctypes.c_int32),
        ("n_jobs", ctypes.c_int32), ("n_regions", ctypes.c_int32), ("expected", ctypes.c_int32),
        ("group_tiles", ctypes.c_int32), ("ring_slots", ctypes.c_int32),
        ("grid", ctypes.c_int32), ("gemm_ctas", ctypes.c_int32), ("reducer_ctas", ctypes.c_int32),
        ("reducer_warps", ctypes.c_int32),
        ("reduce_rows", ctypes.c_int32), ("n_reduce_items", ctypes.c_int32),
        ("stages", ctypes.c_int32), ("k_blocks", ctypes.c_int32), ("smem_bytes", ctypes.c_int32),
        ("mode", ctypes.c_int32), ("dtype", ctypes.c_int32), ("cluster_ctas", ctypes.c_int32),
        ("partial_dtype", ctypes.c_int32), ("w_layout", ctypes.c_int32), ("order", ctypes.c_int32),
        ("reduce", ctypes.c_int32), ("split_k", ctypes.c_int32), ("tuned", ctypes.c_int32), ("reserved0", ctypes.c_int32),
        ("workspace_bytes", ctypes.c_int64),
        ("flops", ctypes.c_double), ("bytes_gemm", ctypes.c_double), ("bytes_reduce", ctypes.c_double),
        ("bytes_fused", ctypes.c_double),
    ]

    def as_dict(self) -> dict:
        return {n: getattr(self, n) for n, _ in self._fields_}


class Status(ctypes.Structure):
    _fields_ = [("code", ctypes.c_int32), ("where", ctypes.c_int32), ("block", ctypes.c_int32),
                ("detail", ctypes.c_int32)]


class T3Error(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libt3.so (built by paper_2401_16677_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2401_16677_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        i32, i64, p = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
        cp = ctypes.POINTER(Chunking)
        L.t3_plan.argtypes = [i64, i64, i64, i32, i32, cp]
        L.t3_plan.restype = p
        L.t3_gemm_rs.argtypes = [p, p, p, p, p]
        L.t3_gemm_rs.restype = ctypes.c_int
        L.t3_gemm_rs_mode.argtypes = [p, i32, p, p, p, p]
        L.t3_gemm_rs_mode.restype = ctypes.c_int
        L.t3_gemm_rs_ex.argtypes = [p, p, p, p, ctypes.POINTER(Epilogue), p]
        L.t3_gemm_rs_ex.restype = ctypes.c_int
        L.t3_plan_tune.argtypes = [p, p, p, p, p, ctypes.POINTER(Tune)]
        L.t3_plan_tune.restype = ctypes.c_int
        L.t3_plan_timeline.argtypes = [p, ctypes.POINTER(Timeline)]
        L.t3_plan_timeline.restype = ctypes.c_int
        L.t3_plan_ring.argtypes = [p, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_int64)]
        L.t3_plan_ring.restype = ctypes.c_int
        L.t3_gemm_rs_host.argtypes = [p, p, p, p, p]
        L.t3_gemm_rs_host.restype = ctypes.c_int
        L.t3_gemm_rs_static.argtypes = [i64, i64, i64, i32, i32, p, p, p, p]
        L.t3_gemm_rs_static.restype = ctypes.c_int
        L.t3_destroy.argtypes = [p]
        L.t3_destroy.restype = ctypes.c_int
        L.t3_plan_info.argtypes = [p, ctypes.POINTER(Info)]
        L.t3_plan_info.restype = ctypes.c_int
        L.t3_plan_status.argtypes = [p, ctypes.POINTER(Status)]
        L.t3_plan_status.restype = ctypes.c_int
        L.t3_plan_partials.argtypes = [p, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_int64)]
        L.t3_plan_partials.restype = ctypes.c_int
        L.t3_plan_export_partials.argtypes = [p, p, p]
        L.t3_plan_export_partials.restype = ctypes.c_int
        L.t3_geometry.argtypes = [i64, i64, i64, i32, i32, cp, ctypes.POINTER(Info)]
        L.t3_geometry.restype = ctypes.c_int
        L.t3_schedule.argtypes = [i64, i64, i64, i32, i32, cp, p, i64]
        L.t3_schedule.restype = i64
        L.t3_reduce_schedule.argtypes = [i64, i64, i64, i32, i32, cp, p, i64]
        L.t3_reduce_schedule.restype = i64
        L.t3_ring_order.argtypes = [i32, i32, p]
        L.t3_ring_order.restype = ctypes.c_int
        L.t3_last_error.restype = ctypes.c_int
        L.t3_strerror.argtypes = [ctypes.c_int]
        L.t3_strerror.restype = ctypes.c_char_p
        L.t3_abi_sizes.argtypes = [ctypes.POINTER(ctypes.c_int32), i32]
        L.t3_abi_sizes.restype = ctypes.c_int
        sizes = (ctypes.c_int32 * 6)()
        L.t3_abi_sizes(sizes, 6)
        mine = [ctypes.sizeof(c) for c in (Chunking, Info, Status, Epilogue, Timeline, Tune)]
        if list(sizes) != mine:
            raise RuntimeError(f"{LIB_PATH}: struct sizes {list(sizes)} differ from this binding's {mine} (stale library?)")
        L.t3_version.restype = ctypes.c_int
        L.t3_shared_fetch_available.restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().t3_strerror(int(code)).decode()


def last_error() -> int:
    return int(lib().t3_last_error())


def version() -> int:
    return int(lib().t3_version())


def shared_fetch_available() -> bool:
    return bool(lib().t3_shared_fetch_available())


STATIC_SCRATCH_BYTES = (32 << 20) + (64 << 10)


def gemm_rs_static(M: int, N: int, K: int, R: int, dtype: int, X: int, W: int, Y: int, stream: int = 0) -> None:
    """t3_gemm_rs_static: the fused op for callers that may not allocate device memory.  Scratch is a
    static device array inside the library (STATIC_SCRATCH_BYTES); calls that overlap on one GPU race."""
    rc = lib().t3_gemm_rs_static(M, N, K, R, dtype, X, W, Y, stream)
    if rc != OK:
        raise T3Error(rc, "t3_gemm_rs_static")


def epilogue(bias: int = 0, residual: int = 0, keep: int = 0, keep_scale: float = 1.0,
             bias_dtype: int = EPI_BF16, residual_dtype: int = EPI_BF16) -> Epilogue:
    e = Epilogue()
    e.bias, e.residual, e.keep = bias or None, residual or None, keep or None
    e.keep_scale, e.bias_dtype, e.residual_dtype = float(keep_scale), int(bias_dtype), int(residual_dtype)
    return e


def chunking(**kw) -> Chunking:
    c = Chunking()
    for k, v in kw.items():
        if not hasattr(c, k):
            raise TypeError(f"unknown chunking field {k!r}")
        setattr(c, k, int(v))
    return c


def _cptr(c: Optional[Chunking]):
    return ctypes.byref(c) if c is not None else None


def geometry(M: int, N: int, K: int, R: int, dtype: int = BF16_OUT_BF16,
             chunk: Optional[Chunking] = None) -> Info:
    out = Info()
    rc = lib().t3_geometry(M, N, K, R, dtype, _cptr(chunk), ctypes.byref(out))
    if rc != OK:
        raise T3Error(rc, "t3_geometry")
    return out


def schedule(M: int, N: int, K: int, R: int, dtype: int = BF16_OUT_BF16,
             chunk: Optional[Chunking] = None) -> List[Tuple[int, int, int]]:
    n = lib().t3_schedule(M, N, K, R, dtype, _cptr(chunk), None, 0)
    if n < 0:
        raise T3Error(int(n), "t3_schedule")
    buf = (ctypes.c_int32 * (3 * n))()
    n2 = lib().t3_schedule(M, N, K, R, dtype, _cptr(chunk), buf, n)
    assert n2 == n
    return [(buf[3 * j], buf[3 * j + 1], buf[3 * j + 2]) for j in range(n)]


def reduce_schedule(M: int, N: int, K: int, R: int, dtype: int = BF16_OUT_BF16,
                    chunk: Optional[Chunking] = None) -> List[Tuple[int, int, int, int, int, int]]:
    """Reducer items in ticket order: (m_tile, n_tile, row0, n_rows, col0, n_cols)."""
    n = lib().t3_reduce_schedule(M, N, K, R, dtype, _cptr(chunk), None, 0)
    if n < 0:
        raise T3Error(int(n), "t3_reduce_schedule")
    buf = (ctypes.c_int32 * (6 * n))()
    n2 = lib().t3_reduce_schedule(M, N, K, R, dtype, _cptr(chunk), buf, n)
    assert n2 == n
    return [tuple(buf[6 * j + i] for i in range(6)) for j in range(n)]


def ring_order(c: int, R: int) -> List[int]:
    buf = (ctypes.c_int32 * R)()
    rc = lib().t3_ring_order(c, R, buf)
    if rc != OK:
        raise T3Error(rc, "t3_ring_order")
    return list(buf)


class Plan:
    """Owns one t3_plan_t.  Pointers passed to the run calls are raw device
    addresses (e.g. ``tensor.data_ptr()``); ``stream`` is a cudaStream_t value
    (e.g. ``torch.cuda.current_stream().cuda_stream``)."""

    def __init__(self, M: int, N: int, K: int, R: int, dtype: int = BF16_OUT_BF16,
                 chunk: Optional[Chunking] = None):
        self._h = lib().t3_plan(M, N, K, R, dtype, _cptr(chunk))
        if not self._h:
            raise T3Error(last_error(), "t3_plan")

    def info(self) -> Info:
        out = Info()
        rc = lib().t3_plan_info(self._h, ctypes.byref(out))
        if rc != OK:
            raise T3Error(rc, "t3_plan_info")
        return out

    def gemm_rs(self, X: int, W: int, Y: int, stream: int = 0) -> None:
        rc = lib().t3_gemm_rs(self._h, X, W, Y, stream)
        if rc != OK:
            raise T3Error(rc, "t3_gemm_rs")

    def gemm_rs_mode(self, mode: int, X: int, W: int, Y: int, stream: int = 0) -> None:
        rc = lib().t3_gemm_rs_mode(self._h, mode, X, W, Y, stream)
        if rc != OK:
            raise T3Error(rc, "t3_gemm_rs_mode")

    def gemm_rs_ex(self, X: int, W: int, Y: int, epi: Optional[Epilogue], stream: int = 0) -> None:
        """t3_gemm_rs with bias / dropout mask / residual fused on the reduced chunk."""
        rc = lib().t3_gemm_rs_ex(self._h, X, W, Y, ctypes.byref(epi) if epi is not None else None, stream)
        if rc != OK:
            raise T3Error(rc, "t3_gemm_rs_ex")

    def tune(self, X: int, W: int, Y: int, stream: int = 0) -> Tune:
        """t3_plan_tune: short trial on the real operands; keeps the fastest configuration."""
        out = Tune()
        rc = lib().t3_plan_tune(self._h, X, W, Y, stream, ctypes.byref(out))
        if rc != OK:
            raise T3Error(rc, "t3_plan_tune")
        return out

    def timeline(self) -> Timeline:
        """t3_plan_timeline of the last fused call (synchronises)."""
        out = Timeline()
        rc = lib().t3_plan_timeline(self._h, ctypes.byref(out))
        if rc != OK:
            raise T3Error(rc, "t3_plan_timeline")
        return out

    def ring(self) -> Tuple[int, int]:
        """(device address, bytes) of the fused mode's ring of region slots; (0, 0) without a ring."""
        out = ctypes.c_void_p()
        nbytes = ctypes.c_int64()
        rc = lib().t3_plan_ring(self._h, ctypes.byref(out), ctypes.byref(nbytes))
        if rc != OK:
            raise T3Error(rc, "t3_plan_ring")
        return int(out.value or 0), int(nbytes.value)

    def gemm_rs_host(self, X_host: int, W_host: int, Y_host: int, stream: int = 0) -> None:
        """Host-pointer entry: H2D copies, the op, D2H copy, all on `stream`."""
        rc = lib().t3_gemm_rs_host(self._h, X_host, W_host, Y_host, stream)
        if rc != OK:
            raise T3Error(rc, "t3_gemm_rs_host")

    def status(self) -> Status:
        """Synchronises, returns the device status word (code 0 = fine)."""
        out = Status()
        rc = lib().t3_plan_status(self._h, ctypes.byref(out))
        if rc not in (OK, ERR_TIMEOUT):
            raise T3Error(rc, "t3_plan_status")
        return out

    def partials(self) -> Tuple[int, int]:
        """(device address, bytes) of the full partial buffers; the layout is internal."""
        out = ctypes.c_void_p()
        nbytes = ctypes.c_int64()
        rc = lib().t3_plan_partials(self._h, ctypes.byref(out), ctypes.byref(nbytes))
        if rc != OK:
            raise T3Error(rc, "t3_plan_partials")
        return int(out.value), int(nbytes.value)

    def export_partials(self, dst: int, stream: int = 0) -> None:
        """Writes the partial products as row-major fp32 [R][M][N] to device address ``dst``."""
        rc = lib().t3_plan_export_partials(self._h, ctypes.c_void_p(dst), ctypes.c_void_p(stream))
        if rc != OK:
            raise T3Error(rc, "t3_plan_export_partials")

    def destroy(self) -> None:
        if self._h:
            lib().t3_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()
