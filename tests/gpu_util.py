"""Helpers for the GPU tests: device upload of bf16 bit patterns and a
zero-copy torch view of a raw device pointer.  Marshalling only."""
import numpy as np
import torch

from paper_2401_16677_b200 import t3
from paper_2401_16677_b200 import workloads as wl


def to_device_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> cuda bfloat16 tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


class _Raw:
    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = dict(shape=tuple(shape), typestr=typestr, data=(int(ptr), False), version=2)


def view_f32(ptr: int, shape) -> torch.Tensor:
    return torch.as_tensor(_Raw(ptr, shape, "<f4"), device="cuda")


def poison_partials(plan) -> None:
    """Fills the full partial buffers AND the fused mode's ring of region slots with NaN: a reducer that
    reads a tile before it landed shows up.  (Not for update-in-place plans, whose accumulators must be zero.)"""
    ptr, nbytes = plan.partials()
    view_f32(ptr, (nbytes // 4,)).fill_(float("nan"))
    rptr, rbytes = plan.ring()
    if rptr:
        view_f32(rptr, (rbytes // 4,)).fill_(float("nan"))


BAND_BYTES = 4096
BAND_PATTERN = 0xA5


def banded(nbytes: int):
    """A device buffer of nbytes with a 4 KiB guard band of a known byte pattern on each side.
    Returns (whole uint8 tensor, byte offset of the payload)."""
    whole = torch.full((nbytes + 2 * BAND_BYTES,), BAND_PATTERN, dtype=torch.uint8, device="cuda")
    return whole, BAND_BYTES


def bands_intact(whole: torch.Tensor) -> bool:
    """True when both guard bands still hold the pattern (nothing was written outside the payload)."""
    lo, hi = whole[:BAND_BYTES], whole[-BAND_BYTES:]
    return bool((lo == BAND_PATTERN).all()) and bool((hi == BAND_PATTERN).all())


def exported_partials(plan, R, M, N) -> np.ndarray:
    """The partial products of the last sequential / full-buffer run as a row-major [R][M][N] array."""
    dst = torch.empty((R, M, N), dtype=torch.float32, device="cuda")
    plan.export_partials(dst.data_ptr(), stream())
    torch.cuda.synchronize()
    return dst.cpu().numpy()


def stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def out_tensor(M, N, dtype, fill=float("nan")) -> torch.Tensor:
    td = torch.float32 if dtype == t3.BF16_OUT_F32 else torch.bfloat16
    return torch.full((M, N), fill, dtype=td, device="cuda")


def y_bits(Y: torch.Tensor) -> np.ndarray:
    """Raw bits of the output for bitwise comparisons."""
    if Y.dtype == torch.bfloat16:
        return Y.view(torch.int16).cpu().numpy().view(np.uint16)
    return Y.view(torch.int32).cpu().numpy().view(np.uint32)


def run_once(plan, mode, X, W, Y):
    plan.gemm_rs_mode(mode, X.data_ptr(), W.data_ptr(), Y.data_ptr(), stream())
    s = plan.status()
    assert s.code == 0, f"device status {s.code} where={s.where} block={s.block} detail={s.detail}"


def upload(xb, wb_kn):
    return to_device_bf16(xb), to_device_bf16(wl.w_nk(wb_kn))
