"""Pins for the CPU oracle: everything here checks it against something other
than itself (exact rational arithmetic, dgemm, closed forms, invariants, the
paper's four-device ring example)."""
import os
import zlib
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2401_16677_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def _rand_bf16(rng, shape, scale=1.0):
    return _bits(rng.standard_normal(shape).astype(np.float32) * scale)


# --------------------------------------------------------------------------
# 1. exact rational brute force on tiny shapes
# --------------------------------------------------------------------------

def _brute_fraction(xb, wb):
    x = wl.bf16_bits_to_f64(xb)
    w = wl.bf16_bits_to_f64(wb)
    M, K = x.shape
    N = w.shape[1]
    out = np.empty((M, N), dtype=np.float64)
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                acc += Fraction(float(x[m, k])) * Fraction(float(w[k, n]))
            out[m, n] = float(acc)  # correctly rounded exact value
    return out


@pytest.mark.parametrize("M,N,K", [(4, 3, 8), (6, 5, 12), (8, 16, 16), (2, 7, 24)])
def test_brute_force_exact_rational(M, N, K):
    rng = np.random.default_rng(1234 + M * 100 + N * 10 + K)
    xb = _rand_bf16(rng, (M, K))
    wb = _rand_bf16(rng, (K, N))
    ref = _brute_fraction(xb, wb)
    scale = np.abs(wl.bf16_bits_to_f64(xb)) @ np.abs(wl.bf16_bits_to_f64(wb))
    for R in range(1, K + 1):
        if K % R or M % R:
            continue
        y = oracle.gemm_rs(xb, wb, R)
        # fp64 accumulation error bound: K * eps * sum|x||w|
        assert np.all(np.abs(y - ref) <= 4 * K * 2.0 ** -53 * scale + 1e-300), (R,)


# --------------------------------------------------------------------------
# 2. library special case: the K-split sum is a textbook GEMM (dgemm)
# --------------------------------------------------------------------------

def test_dgemm_config1_full():
    xb, wb = wl.make_inputs(wl.C1)
    y = oracle.gemm_rs(xb, wb, wl.C1.R)
    ref = wl.bf16_bits_to_f64(xb) @ wl.bf16_bits_to_f64(wb)
    assert y.shape == (256, 512)
    assert oracle.max_rel_err(y, ref) < 1e-12


@pytest.mark.parametrize("M,N,K,R", [
    (64, 1600, 6400, 8),    # config-2 widths (K_r = 800, not a multiple of 64)
    (64, 3072, 3072, 8),    # config-3 attention-out widths
    (32, 512, 2048, 16),
])
def test_dgemm_wide_shapes_row_sample(M, N, K, R):
    rng = np.random.default_rng(7)
    xb = _rand_bf16(rng, (M, K))
    wb = _rand_bf16(rng, (K, N), 0.02)
    rows = np.array([0, 1, M // R - 1, M // R, M - 1])
    y = oracle.gemm_rs(xb, wb, R, rows=rows)
    ref = wl.bf16_bits_to_f64(xb)[rows] @ wl.bf16_bits_to_f64(wb)
    assert oracle.max_rel_err(y, ref) < 1e-12


def test_operands_not_transposed():
    # asymmetric shapes and values: a transposed operand or swapped index fails
    rng = np.random.default_rng(3)
    M, K, N, R = 6, 16, 10, 2
    xb = _rand_bf16(rng, (M, K))
    wb = _rand_bf16(rng, (K, N))
    y = oracle.gemm_rs(xb, wb, R)
    ref = np.einsum("mk,kn->mn", wl.bf16_bits_to_f64(xb), wl.bf16_bits_to_f64(wb))
    assert np.allclose(y, ref, rtol=0, atol=1e-12)
    assert y.shape == (M, N)


# --------------------------------------------------------------------------
# 3. identity and one-hot weights
# --------------------------------------------------------------------------

def test_identity_weight_returns_input():
    rng = np.random.default_rng(11)
    M, K, R = 8, 32, 4
    xb = _rand_bf16(rng, (M, K))
    wb = _bits(np.eye(K))
    y = oracle.gemm_rs(xb, wb, R)
    assert np.array_equal(y, wl.bf16_bits_to_f64(xb))


def test_one_hot_columns_select_across_slices():
    rng = np.random.default_rng(12)
    M, K, N, R = 8, 48, 20, 4
    xb = _rand_bf16(rng, (M, K))
    pi = rng.permutation(K)[:N]          # crosses slice boundaries
    w = np.zeros((K, N), dtype=np.float32)
    w[pi, np.arange(N)] = 1.0
    y = oracle.gemm_rs(xb, _bits(w), R)
    assert np.array_equal(y, wl.bf16_bits_to_f64(xb)[:, pi])


# --------------------------------------------------------------------------
# 4. closed forms
# --------------------------------------------------------------------------

def test_all_ones_gives_K():
    M, K, N, R = 4, 64, 6, 4
    y = oracle.gemm_rs(_bits(np.ones((M, K))), _bits(np.ones((K, N))), R)
    assert np.array_equal(y, np.full((M, N), float(K)))


def test_rank_one():
    M, K, N, R = 8, 32, 5, 8
    u = np.array([1, 2, -3, 0.5, 4, -0.25, 8, 1.5], dtype=np.float32)
    v = np.array([1, -2, 0.5, 3, 0.125], dtype=np.float32)
    x = np.repeat(u[:, None], K, axis=1)
    w = np.repeat(v[None, :], K, axis=0)
    y = oracle.gemm_rs(_bits(x), _bits(w), R)
    assert np.array_equal(y, K * np.outer(u, v).astype(np.float64))


def test_slice_indicator_counts_only_that_slice():
    M, K, N, R = 5, 40, 3, 5
    Kr = K // R
    for r0 in range(R):
        x = np.zeros((M, K), dtype=np.float32)
        x[:, r0 * Kr:(r0 + 1) * Kr] = 1.0
        y, P = oracle.gemm_rs(_bits(x), _bits(np.ones((K, N))), R, return_partials=True)
        assert np.array_equal(y, np.full((M, N), float(Kr)))
        for r in range(R):
            want = float(Kr) if r == r0 else 0.0
            assert np.array_equal(P[r], np.full((M, N), want)), (r0, r)


def test_partials_are_the_slice_products_and_sum_to_y():
    rng = np.random.default_rng(21)
    M, K, N, R = 8, 64, 12, 4
    Kr = K // R
    xb, wb = _rand_bf16(rng, (M, K)), _rand_bf16(rng, (K, N))
    y, P = oracle.gemm_rs(xb, wb, R, return_partials=True)
    x, w = wl.bf16_bits_to_f64(xb), wl.bf16_bits_to_f64(wb)
    for r in range(R):
        ref = x[:, r * Kr:(r + 1) * Kr] @ w[r * Kr:(r + 1) * Kr]
        assert np.allclose(P[r], ref, rtol=0, atol=1e-12)
    assert np.allclose(P.sum(axis=0), y, rtol=0, atol=1e-12)


# --------------------------------------------------------------------------
# 5. exact-integer inputs: bit-for-bit
# --------------------------------------------------------------------------

@pytest.mark.parametrize("M,N,K,R", [(16, 24, 256, 4), (12, 40, 4096, 2), (9, 8, 96, 3)])
def test_exact_integer_inputs(M, N, K, R):
    if M % R:
        pytest.skip("shape")
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=5)
    y = oracle.gemm_rs(xb, wb, R)
    xi = wl.bf16_bits_to_f64(xb).astype(np.int64)
    wi = wl.bf16_bits_to_f64(wb).astype(np.int64)
    assert np.array_equal(y, (xi @ wi).astype(np.float64))


# --------------------------------------------------------------------------
# 6. linearity (no-rounding fp64 entry point)
# --------------------------------------------------------------------------

def test_linearity_in_x():
    rng = np.random.default_rng(31)
    M, K, N, R = 8, 64, 10, 4
    x1 = wl.bf16_bits_to_f64(_rand_bf16(rng, (M, K)))
    x2 = wl.bf16_bits_to_f64(_rand_bf16(rng, (M, K)))
    w = wl.bf16_bits_to_f64(_rand_bf16(rng, (K, N)))
    a = 2.0 ** -3
    lhs = oracle.gemm_rs_f64(a * x1 + x2, w, R)
    rhs = a * oracle.gemm_rs_f64(x1, w, R) + oracle.gemm_rs_f64(x2, w, R)
    assert oracle.max_rel_err(lhs, rhs) < 1e-13


def test_bf16_and_f64_entry_points_agree():
    rng = np.random.default_rng(32)
    M, K, N, R = 8, 64, 10, 2
    xb, wb = _rand_bf16(rng, (M, K)), _rand_bf16(rng, (K, N))
    a = oracle.gemm_rs(xb, wb, R)
    b = oracle.gemm_rs_f64(wl.bf16_bits_to_f64(xb), wl.bf16_bits_to_f64(wb), R)
    assert np.array_equal(a, b)


# --------------------------------------------------------------------------
# 7. invariance in R; 8. chunking and row independence
# --------------------------------------------------------------------------

def test_r_invariance():
    rng = np.random.default_rng(41)
    M, K, N = 16, 128, 9
    xb, wb = _rand_bf16(rng, (M, K)), _rand_bf16(rng, (K, N))
    base = oracle.gemm_rs(xb, wb, 1)
    for R in (2, 4, 8, 16):
        assert oracle.max_rel_err(oracle.gemm_rs(xb, wb, R), base) < 1e-13


def test_chunks_concatenate_and_rows_are_independent():
    rng = np.random.default_rng(42)
    M, K, N, R = 16, 32, 6, 4
    xb, wb = _rand_bf16(rng, (M, K)), _rand_bf16(rng, (K, N))
    y = oracle.gemm_rs(xb, wb, R)
    ch = oracle.chunks(y, R)
    assert len(ch) == R and all(c.shape == (M // R, N) for c in ch)
    assert np.array_equal(np.concatenate(ch, axis=0), y)
    # a row subset gives exactly those rows of the full result
    rows = [0, 3, 4, 15]
    assert np.array_equal(oracle.gemm_rs(xb, wb, R, rows=rows), y[rows])
    # chunk c equals the oracle run on those rows of X alone (R=1: one device)
    cr = M // R
    for c in range(R):
        alone = oracle.gemm_rs(xb[c * cr:(c + 1) * cr], wb, 1)
        assert oracle.max_rel_err(alone, ch[c]) < 1e-13


def test_bad_shapes_rejected():
    xb = np.zeros((6, 8), dtype=np.uint16)
    wb = np.zeros((8, 4), dtype=np.uint16)
    with pytest.raises(ValueError):
        oracle.gemm_rs(xb, wb, 4)      # M % R != 0
    with pytest.raises(ValueError):
        oracle.gemm_rs(xb, wb, 3)      # K % R != 0


# --------------------------------------------------------------------------
# 9. ring order (paper's four-device example) and the fp32 ring sum
# --------------------------------------------------------------------------

def test_ring_order_matches_four_gpu_example():
    want = {}
    with open(os.path.join(GOLDEN, "ring_order_R4.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            c, order = line.split(":")
            want[int(c)] = [int(t) for t in order.split()]
    assert sorted(want) == [0, 1, 2, 3]
    for c, o in want.items():
        assert oracle.ring_order(c, 4) == o


@pytest.mark.parametrize("R", [1, 2, 3, 8, 16])
def test_ring_order_is_a_permutation_ending_at_owner(R):
    for c in range(R):
        o = oracle.ring_order(c, R)
        assert sorted(o) == list(range(R))
        assert o[-1] == c
        if R > 1:
            assert o[0] == (c - 1) % R
        # R-1 ring steps (Section 2.3): each step moves to the lower neighbour
        for a, b in zip(o[:-1], o[1:]):
            assert b == (a - 1) % R


def test_ring_sum_f32_order_is_observable():
    # (1e8 + 1) - 1e8 = 0 in fp32, while (1e8 - 1e8) + 1 = 1: order matters.
    R, M, N = 3, 3, 1
    P = np.zeros((R, M, N), dtype=np.float32)
    P[0], P[1], P[2] = 1e8, 1.0, -1e8
    y = oracle.ring_sum_f32(P)
    # chunk 0: order [2,1,0] -> (-1e8 + 1) + 1e8 = 0
    # chunk 1: order [0,2,1] -> (1e8 - 1e8) + 1 = 1
    # chunk 2: order [1,0,2] -> (1 + 1e8) - 1e8 = 0
    assert y[:, 0].tolist() == [0.0, 1.0, 0.0]


def test_ring_sum_f32_matches_numpy_sequential_adds():
    rng = np.random.default_rng(51)
    R, M, N = 4, 8, 5
    P = rng.standard_normal((R, M, N)).astype(np.float32)
    y = oracle.ring_sum_f32(P)
    cr = M // R
    for m in range(M):
        o = oracle.ring_order(m // cr, R)
        acc = P[o[0], m].copy()
        for r in o[1:]:
            acc = (acc + P[r, m]).astype(np.float32)
        assert np.array_equal(acc, y[m])


# --------------------------------------------------------------------------
# 10. the comparison metric and the input generators
# --------------------------------------------------------------------------

def test_max_rel_err_metric():
    ref = np.array([[1.0, -2.0], [0.0, 4.0]])
    rms = np.sqrt(np.mean(ref ** 2))
    y = ref.copy()
    y[1, 0] = 0.5          # error at an exact zero is measured against rms
    assert oracle.max_rel_err(y, ref) == pytest.approx(0.5 / rms)
    y = ref.copy()
    y[1, 1] = 4.4
    assert oracle.max_rel_err(y, ref) == pytest.approx(0.1)
    y[0, 0] = np.nan
    assert oracle.max_rel_err(y, ref) == float("inf")


def test_bf16_rounding_is_rne():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(61)
    a = np.concatenate([
        rng.standard_normal(4096).astype(np.float32),
        np.array([1.0, 1.00390625, 1.005859375, 1.01171875, -1.00390625, 0.0, 3.0e38], dtype=np.float32),
    ])
    mine = wl.f32_to_bf16_bits(a)
    ref = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, ref)
    assert np.array_equal(wl.bf16_bits_to_f32(mine), torch.from_numpy(a).to(torch.bfloat16).float().numpy())


def test_workload_table_and_seeds():
    assert wl.C1.resolved_seed() == 0
    assert wl.C2.resolved_seed() == zlib.crc32(b"8192,1600,6400,8")
    assert (wl.C2.K_r, wl.C3A.K_r, wl.C3B.K_r, wl.C4.K_r) == (800, 384, 1536, 2048)
    assert [w.chunk_rows for w in (wl.C1, wl.C2, wl.C3A, wl.C4)] == [128, 1024, 512, 256]
    pts = wl.sweep_points()
    assert len(pts) == 36 and len({p.resolved_seed() for p in pts}) == 36
    assert all(p.K == 4 * p.N and p.K % p.R == 0 for p in pts)


def test_config1_inputs_distribution():
    xb, wb = wl.make_inputs(wl.C1)
    assert xb.shape == (256, 2048) and wb.shape == (2048, 512)
    x = wl.bf16_bits_to_f64(xb)
    lim = 1.0 / np.sqrt(2048.0)
    assert np.abs(x).max() <= lim * (1 + 2 ** -8)
    assert abs(x.mean()) < 1e-3 * lim * 10
    assert x.std() == pytest.approx(lim / np.sqrt(3.0), rel=2e-2)
    # same seed, same bits
    xb2, _ = wl.make_inputs(wl.C1)
    assert np.array_equal(xb, xb2)


def test_gelu_inputs_are_erf_gelu():
    from math import erf, sqrt
    w = wl.Workload("t", M=8, N=8, K=16, R=2, x_dist="gelu_normal", w_dist="normal", seed=3)
    xb, _ = wl.make_inputs(w)
    z = np.random.default_rng(3).standard_normal((8, 16), dtype=np.float32)
    want = np.array([[0.5 * float(v) * (1 + erf(float(v) / sqrt(2))) for v in row] for row in z])
    assert np.array_equal(xb, wl.f32_to_bf16_bits(want.astype(np.float32)))


def test_sample_rows_cover_chunks():
    rows = wl.sample_rows(4096, 16, seed=5)
    cr = 256
    for c in range(16):
        assert c * cr in rows and (c + 1) * cr - 1 in rows
    assert len(rows) <= 4096 // 16 + 32


# ---------------------------------------------------------------------------
# the element-wise tail on the reduced chunk (Section 7.6): bias, dropout mask, residual
# ---------------------------------------------------------------------------

def test_epilogue_closed_forms():
    """All-ones inputs with a constant bias give K + b everywhere; a dropped element is exactly the
    residual; a kept one is (K + b) * scale + residual.  A wrong order of the three steps (bias after the
    mask, residual before it) or a mask applied to the residual changes these values."""
    M, N, K, R = 8, 16, 32, 4
    ones = wl.f32_to_bf16_bits(np.ones((M, K), dtype=np.float32))
    wones = wl.f32_to_bf16_bits(np.ones((K, N), dtype=np.float32))
    Y = oracle.gemm_rs(ones, wones, R)
    assert np.all(Y == K)
    b = np.full(N, 0.5)
    assert np.all(oracle.epilogue(Y, bias=b) == K + 0.5)
    keep = np.zeros((M, N), dtype=np.uint8)
    keep[::2] = 1
    res = np.full((M, N), 3.0)
    out = oracle.epilogue(Y, bias=b, keep=keep, keep_scale=2.0, residual=res)
    assert np.all(out[::2] == (K + 0.5) * 2.0 + 3.0)
    assert np.all(out[1::2] == 3.0)
    # bias is per column, the mask and the residual per element
    b2 = np.arange(N, dtype=np.float64)
    out2 = oracle.epilogue(Y, bias=b2)
    assert np.array_equal(out2, K + np.tile(b2, (M, 1)))
    # no operand: identity
    assert np.array_equal(oracle.epilogue(Y), Y)


def test_epilogue_residual_cancels_the_product_exactly():
    """residual = -(X.W) on exact-integer inputs leaves exactly zero (the reduced sum and the residual
    meet with opposite signs: a sign slip or a dropped slice leaves a non-zero)."""
    M, N, K, R = 12, 24, 64, 4
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=9)
    x = wl.bf16_bits_to_f64(xb).astype(np.int64)
    w = wl.bf16_bits_to_f64(wb).astype(np.int64)
    out = oracle.epilogue(oracle.gemm_rs(xb, wb, R), residual=-(x @ w).astype(np.float64))
    assert np.all(out == 0.0)
    # the fp32 restatement agrees on exactly representable values
    s32 = oracle.gemm_rs(xb, wb, R).astype(np.float32)
    keep = (np.arange(M * N).reshape(M, N) % 3 != 0).astype(np.uint8)
    b = np.arange(N, dtype=np.float32) - 7
    r32 = np.arange(M * N, dtype=np.float32).reshape(M, N) % 11
    got = oracle.epilogue_f32(s32, bias=b, keep=keep, keep_scale=2.0, residual=r32)
    assert got.dtype == np.float32
    assert np.array_equal(got.astype(np.float64), oracle.epilogue(s32.astype(np.float64), bias=b, keep=keep, keep_scale=2.0, residual=r32))


def test_epilogue_f32_rounds_every_step():
    """(1e8 + 1) * 1 - 1e8 is 0 when the add is rounded to fp32 before the next step, 1 in fp64."""
    S = np.array([[1e8]], dtype=np.float32)
    out32 = oracle.epilogue_f32(S, bias=np.array([1.0]), keep=np.array([[1]], dtype=np.uint8), keep_scale=1.0,
                                residual=np.array([[-1e8]]))
    out64 = oracle.epilogue(S.astype(np.float64), bias=np.array([1.0]), keep=np.array([[1]], dtype=np.uint8), keep_scale=1.0,
                            residual=np.array([[-1e8]]))
    assert out32[0, 0] == 0.0 and out64[0, 0] == 1.0
