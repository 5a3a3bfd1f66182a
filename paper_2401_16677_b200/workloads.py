"""Seeded synthetic inputs for the tensor-parallel sublayer workloads.

This module only *draws numbers and lays them out*.  It contains none of the
method's arithmetic (no product, no partial sum, no reduction), imports
neither the CUDA binding nor the CPU oracle, and is the one piece both sides
share: tests and the bench feed the very same bf16 bit patterns to each.

Shapes follow the paper's sliced sublayers (Section 2.4: a weight sliced
along its dot-product dimension over the tensor-parallel group; Section 5.2
and the model table: token counts of 8K-16K, TP degrees 8/16).  Value
distributions are synthetic stand-ins for trained activations and weights.

Conventions
-----------
M tokens, N output features, K total reduction dim, R tensor-parallel slices,
K_r = K / R.  ``X`` is [M, K]; ``W`` is the *mathematical* [K, N] matrix.
Arrays are returned as ``uint16`` bf16 bit patterns (round-to-nearest-even
from float32).  ``w_nk`` gives the [N, K] K-contiguous storage the device
library takes by default.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field
from typing import Dict, Iterator, List, Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    M: int
    N: int
    K: int
    R: int
    x_dist: str            # "uniform_rsqrtk" | "normal" | "gelu_normal"
    w_dist: str            # "uniform_rsqrtk" | "normal"
    w_std: float = 0.02
    seed: int | None = None  # None -> crc32 of "M,N,K,R"
    out: Tuple[str, ...] = ("bf16",)

    @property
    def K_r(self) -> int:
        return self.K // self.R

    @property
    def chunk_rows(self) -> int:
        return self.M // self.R

    @property
    def flops(self) -> int:
        return 2 * self.M * self.N * self.K

    def resolved_seed(self) -> int:
        if self.seed is not None:
            return self.seed
        return shape_seed(self.M, self.N, self.K, self.R)


def shape_seed(M: int, N: int, K: int, R: int) -> int:
    """seed = crc32 of the ASCII string "M,N,K,R"."""
    return zlib.crc32(f"{M},{N},{K},{R}".encode("ascii")) & 0xFFFFFFFF


# The five benchmark configurations.
C1 = Workload("C1_tiny", M=256, N=512, K=2048, R=2,
              x_dist="uniform_rsqrtk", w_dist="uniform_rsqrtk", seed=0)
C2 = Workload("C2_gpt2xl_fc2", M=8192, N=1600, K=6400, R=8,
              x_dist="gelu_normal", w_dist="normal", w_std=0.02)
C3A = Workload("C3a_megagpt_attn_out", M=4096, N=3072, K=3072, R=8,
               x_dist="normal", w_dist="normal", w_std=0.02)
C3B = Workload("C3b_megagpt_fc2", M=4096, N=3072, K=12288, R=8,
               x_dist="normal", w_dist="normal", w_std=0.02)
C4 = Workload("C4_large_fc2", M=4096, N=8192, K=32768, R=16,
              x_dist="normal", w_dist="normal", w_std=0.01, out=("bf16", "f32"))

CONFIGS: Dict[str, Workload] = {w.name: w for w in (C1, C2, C3A, C3B, C4)}

# Backward-pass sublayers that need the same sliced GEMM + all-reduce (Section 2.4 and the sublayer
# list of Section 5.2): the input-gradient GEMMs of the input projection (K = 3H) and of FC-1
# (K = 4H, the same shape as the forward FC-2), at the Mega-GPT-like width.  Incoming gradients are
# drawn small and zero-mean like activations' gradients.
X_BWD_IP = Workload("X_megagpt_bwd_ip", M=4096, N=3072, K=9216, R=8,
                    x_dist="normal", w_dist="normal", w_std=0.02)
X_BWD_FC1 = Workload("X_megagpt_bwd_fc1", M=4096, N=3072, K=12288, R=8,
                     x_dist="normal", w_dist="normal", w_std=0.02, seed=20240116)
EXTRA: Dict[str, Workload] = {w.name: w for w in (X_BWD_IP, X_BWD_FC1)}


def sweep_points() -> List[Workload]:
    """Config 5: R x M x H grid, K = 4H split evenly over R."""
    pts = []
    for R in (2, 4, 8, 16):
        for M in (1024, 4096, 16384):
            for H in (2048, 4096, 8192):
                pts.append(Workload(f"C5_R{R}_M{M}_H{H}", M=M, N=H, K=4 * H, R=R,
                                    x_dist="normal", w_dist="normal", w_std=0.02))
    return pts


def by_name(name: str) -> Workload:
    if name in CONFIGS:
        return CONFIGS[name]
    if name in EXTRA:
        return EXTRA[name]
    for w in sweep_points():
        if w.name == name:
            return w
    raise KeyError(name)


# ---------------------------------------------------------------------------
# bf16 bit helpers (layout / encoding only)
# ---------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns (finite inputs)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def w_nk(w_kn_bits: np.ndarray) -> np.ndarray:
    """[K, N] mathematical matrix -> [N, K] K-contiguous storage."""
    return np.ascontiguousarray(w_kn_bits.T)


# ---------------------------------------------------------------------------
# generators
# ---------------------------------------------------------------------------

def _draw(rng: np.random.Generator, dist: str, shape, K: int, std: float) -> np.ndarray:
    if dist == "uniform_rsqrtk":
        a = rng.random(shape, dtype=np.float32)
        a *= np.float32(2.0)
        a -= np.float32(1.0)
        a *= np.float32(1.0 / np.sqrt(float(K)))
        return a
    if dist == "normal":
        a = rng.standard_normal(shape, dtype=np.float32)
        if std != 1.0:
            a *= np.float32(std)
        return a
    if dist == "gelu_normal":
        from scipy.special import erf
        z = rng.standard_normal(shape, dtype=np.float32)
        # exact (erf) GeLU of the samples, evaluated in float64 block by block
        out = np.empty_like(z)
        flat_z, flat_o = z.reshape(-1), out.reshape(-1)
        step = 1 << 22
        for i in range(0, flat_z.size, step):
            zz = flat_z[i:i + step].astype(np.float64)
            flat_o[i:i + step] = (0.5 * zz * (1.0 + erf(zz / np.sqrt(2.0)))).astype(np.float32)
        return out
    raise ValueError(dist)


def make_inputs(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    """Returns (X_bits [M,K] uint16, W_bits [K,N] uint16); X drawn first."""
    rng = np.random.default_rng(w.resolved_seed())
    x = _draw(rng, w.x_dist, (w.M, w.K), w.K, 1.0)
    xb = f32_to_bf16_bits(x)
    del x
    ww = _draw(rng, w.w_dist, (w.K, w.N), w.K, w.w_std)
    wb = f32_to_bf16_bits(ww)
    return xb, wb


def make_small_int_inputs(M: int, N: int, K: int, seed: int, lo: int = -2, hi: int = 2):
    """Integer-valued bf16 inputs in [lo, hi]: every product and partial sum is
    exactly representable in fp32 (and fp64) as long as K*hi*hi < 2**24."""
    rng = np.random.default_rng(seed)
    x = rng.integers(lo, hi + 1, size=(M, K)).astype(np.float32)
    ww = rng.integers(lo, hi + 1, size=(K, N)).astype(np.float32)
    return f32_to_bf16_bits(x), f32_to_bf16_bits(ww)


def sample_rows(M: int, R: int, seed: int, stride: int = 16) -> np.ndarray:
    """Row sample for spot checks at full size: every `stride`-th row at phase
    seed % stride, plus the first and last row of every reduce-scatter chunk."""
    rows = set(range(seed % stride, M, stride))
    cr = M // R
    for c in range(R):
        rows.add(c * cr)
        rows.add((c + 1) * cr - 1)
    return np.array(sorted(rows), dtype=np.int64)
