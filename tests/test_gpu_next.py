"""GPU parity of the options beyond the base path, through the C ABI, against the CPU oracle:
the element-wise tail fused on the reduced chunk (Section 7.6), the update-in-place reduction
(Sections 4.3 / 7.4), split-K producers in the tracker (Section 7.7), small-M shapes (Section 7.3), the
measured configuration choice (Section 4.5's analog), the per-call timeline, the per-device ordering of
launches, and guard bands around every caller-visible buffer."""
import numpy as np
import pytest

import oracle
from paper_2401_16677_b200 import build as t3build
from paper_2401_16677_b200 import t3
from paper_2401_16677_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = {t3.BF16_OUT_BF16: 2e-2, t3.BF16_OUT_F32: 1e-4}


@pytest.fixture(scope="module", autouse=True)
def _built():
    t3build.build()


def _gu():
    import gpu_util
    return gpu_util


def _to_f64(Y):
    return Y.float().cpu().numpy().astype(np.float64)


# ---------------------------------------------------------------------------
# element-wise tail on the reduced chunk (Section 7.6)
# ---------------------------------------------------------------------------

def _epi_operands(M, N, seed, integer, bias_f32, res_f32):
    import torch
    rng = np.random.default_rng(seed)
    if integer:
        bias = rng.integers(-4, 5, size=N).astype(np.float32)
        res = rng.integers(-8, 9, size=(M, N)).astype(np.float32)
    else:
        bias = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(rng.standard_normal(N).astype(np.float32)))
        res = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(rng.standard_normal((M, N)).astype(np.float32)))
    keep = (rng.random((M, N)) >= 0.25).astype(np.uint8)
    tb = torch.from_numpy(bias).cuda()
    tr = torch.from_numpy(res).cuda()
    tb = tb if bias_f32 else tb.to(torch.bfloat16)
    tr = tr if res_f32 else tr.to(torch.bfloat16)
    return bias, res, keep, tb, tr, torch.from_numpy(keep).cuda()


@pytest.mark.parametrize("M,N,K,R,kw", [
    (256, 512, 2048, 2, {}),
    (1000, 520, 1024, 8, {}),                     # ragged M and N
    (768, 1600, 1600, 8, dict(ring_slots=4, group_tiles=2)),   # K_r = 200 and a small ring
    (130, 264, 512, 2, {}),
])
@pytest.mark.parametrize("dtype", [t3.BF16_OUT_F32, t3.BF16_OUT_BF16])
@pytest.mark.parametrize("mode", [t3.MODE_FUSED, t3.MODE_SEQUENTIAL])
def test_epilogue_exact_integer_bitwise(M, N, K, R, kw, dtype, mode):
    """Integer inputs, integer bias and residual, scale 2: every step is exact, so the fused tail must
    equal the oracle's fp64 result bit for bit."""
    import torch
    gu = _gu()
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=M + N)
    bias, res, keep, tb, tr, tk = _epi_operands(M, N, seed=K, integer=True, bias_f32=(M % 3 == 0), res_f32=(N % 16 == 0))
    want = oracle.epilogue(oracle.gemm_rs(xb, wb, R), bias=bias, keep=keep, keep_scale=2.0, residual=res)
    X, W = gu.upload(xb, wb)
    Y = gu.out_tensor(M, N, dtype)
    epi = t3.epilogue(bias=tb.data_ptr(), residual=tr.data_ptr(), keep=tk.data_ptr(), keep_scale=2.0,
                      bias_dtype=t3.EPI_F32 if tb.dtype == torch.float32 else t3.EPI_BF16,
                      residual_dtype=t3.EPI_F32 if tr.dtype == torch.float32 else t3.EPI_BF16)
    with t3.Plan(M, N, K, R, dtype, t3.chunking(mode=mode, **kw)) as plan:
        gu.poison_partials(plan)
        plan.gemm_rs_ex(X.data_ptr(), W.data_ptr(), Y.data_ptr(), epi, gu.stream())
        assert plan.status().code == 0
    got = _to_f64(Y)
    if dtype == t3.BF16_OUT_BF16:      # the one rounding of the output
        want = wl.bf16_bits_to_f64(wl.f32_to_bf16_bits(want.astype(np.float32)))
    assert np.array_equal(got, want)


def test_epilogue_each_operand_alone_and_none():
    """Each step on its own (the others NULL), and epi = NULL equal to the plain call."""
    import torch
    gu = _gu()
    M, N, K, R = 512, 384, 1024, 4
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=5)
    bias, res, keep, tb, tr, tk = _epi_operands(M, N, seed=6, integer=True, bias_f32=False, res_f32=False)
    base = oracle.gemm_rs(xb, wb, R)
    X, W = gu.upload(xb, wb)
    with t3.Plan(M, N, K, R, t3.BF16_OUT_F32, None) as plan:
        cases = [
            (t3.epilogue(bias=tb.data_ptr()), oracle.epilogue(base, bias=bias)),
            (t3.epilogue(residual=tr.data_ptr()), oracle.epilogue(base, residual=res)),
            (t3.epilogue(keep=tk.data_ptr(), keep_scale=4.0), oracle.epilogue(base, keep=keep, keep_scale=4.0)),
            (None, base),
        ]
        for epi, want in cases:
            Y = gu.out_tensor(M, N, t3.BF16_OUT_F32)
            plan.gemm_rs_ex(X.data_ptr(), W.data_ptr(), Y.data_ptr(), epi, gu.stream())
            assert plan.status().code == 0
            assert np.array_equal(_to_f64(Y), want)
        # argument checks: misaligned operand, residual aliasing Y
        Y = gu.out_tensor(M, N, t3.BF16_OUT_F32)
        with pytest.raises(t3.T3Error) as e:
            plan.gemm_rs_ex(X.data_ptr(), W.data_ptr(), Y.data_ptr(), t3.epilogue(bias=tb.data_ptr() + 2), gu.stream())
        assert e.value.code == t3.ERR_INVALID_ARG
        with pytest.raises(t3.T3Error) as e:
            plan.gemm_rs_ex(X.data_ptr(), W.data_ptr(), Y.data_ptr(), t3.epilogue(residual=Y.data_ptr()), gu.stream())
        assert e.value.code == t3.ERR_INVALID_ARG


def test_epilogue_c3b_at_tolerance_and_stage_bitwise():
    """Mega-GPT-like FC-2 at full size with bias + dropout + residual: row sample against the fp64 oracle at
    the output tolerance; the tail stage bit for bit against the fp32 restatement applied to the device's
    own reduced sum; fused == sequential bit for bit."""
    import torch
    gu = _gu()
    w = wl.C3B
    xb, wb = wl.make_inputs(w)
    rows = wl.sample_rows(w.M, w.R, seed=w.resolved_seed(), stride=32)
    bias, res, keep, tb, tr, tk = _epi_operands(w.M, w.N, seed=77, integer=False, bias_f32=True, res_f32=False)
    scale = 1.0 / 0.75
    want = oracle.epilogue(oracle.gemm_rs(xb, wb, w.R, rows=rows), bias=bias, keep=keep[rows], keep_scale=np.float32(scale),
                           residual=res[rows])
    X, W = gu.upload(xb, wb)
    epi = t3.epilogue(bias=tb.data_ptr(), residual=tr.data_ptr(), keep=tk.data_ptr(), keep_scale=scale,
                      bias_dtype=t3.EPI_F32, residual_dtype=t3.EPI_BF16)
    ridx = torch.from_numpy(rows).cuda()
    for dtype in (t3.BF16_OUT_BF16, t3.BF16_OUT_F32):
        with t3.Plan(w.M, w.N, w.K, w.R, dtype, None) as plan:
            gu.poison_partials(plan)
            Y = gu.out_tensor(w.M, w.N, dtype)
            plan.gemm_rs_ex(X.data_ptr(), W.data_ptr(), Y.data_ptr(), epi, gu.stream())
            assert plan.status().code == 0
            assert oracle.max_rel_err(_to_f64(Y[ridx]), want) <= TOL[dtype]
            if dtype == t3.BF16_OUT_F32:
                S = gu.out_tensor(w.M, w.N, dtype)
                gu.run_once(plan, t3.MODE_FUSED, X, W, S)
                stage = oracle.epilogue_f32(S[ridx].cpu().numpy(), bias=bias, keep=keep[rows], keep_scale=np.float32(scale), residual=res[rows])
                assert np.array_equal(Y[ridx].cpu().numpy().view(np.uint32), stage.view(np.uint32))
        with t3.Plan(w.M, w.N, w.K, w.R, dtype, t3.chunking(mode=t3.MODE_SEQUENTIAL)) as plan2:
            Y2 = gu.out_tensor(w.M, w.N, dtype)
            plan2.gemm_rs_ex(X.data_ptr(), W.data_ptr(), Y2.data_ptr(), epi, gu.stream())
            assert plan2.status().code == 0
            assert np.array_equal(gu.y_bits(Y), gu.y_bits(Y2))


# ---------------------------------------------------------------------------
# update-in-place reduction (Sections 4.3, 7.4) and split-K producers (Section 7.7)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("M,N,K,R,kw", [
    (256, 512, 2048, 2, {}),
    (1000, 520, 1024, 8, {}),
    (768, 1600, 1600, 8, dict(ring_slots=4, group_tiles=2)),
    (2048, 1024, 4096, 16, dict(ring_slots=-1)),
    (130, 264, 512, 2, dict(split_k=2)),
    (64, 2048, 8192, 8, dict(split_k=4)),          # small M: few tiles, many producers per tile
    (16, 512, 4096, 4, dict(split_k=16)),
    (512, 256, 1600, 8, dict(split_k=3)),           # K_r = 200: 4 k-blocks split three ways (1, 1, 2)
])
@pytest.mark.parametrize("mode", [t3.MODE_FUSED, t3.MODE_SEQUENTIAL])
def test_inplace_exact_integer_bitwise_and_repeatable(M, N, K, R, kw, mode):
    """Integer sums are exact in any order: the update-in-place result must equal the oracle bit for
    bit, and again on later calls (every call leaves the accumulators cleared)."""
    gu = _gu()
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=M * 7 + R)
    want = oracle.gemm_rs(xb, wb, R)
    X, W = gu.upload(xb, wb)
    with t3.Plan(M, N, K, R, t3.BF16_OUT_F32, t3.chunking(mode=mode, reduce=t3.REDUCE_INPLACE, **kw)) as plan:
        info = plan.info()
        assert info.reduce == t3.REDUCE_INPLACE and info.expected == 2 * R * kw.get("split_k", 1)
        for call in range(3):
            Y = gu.out_tensor(M, N, t3.BF16_OUT_F32)
            gu.run_once(plan, mode, X, W, Y)
            assert np.array_equal(_to_f64(Y), want), f"call {call}"


@pytest.mark.parametrize("name,stride", [("C1_tiny", 1), ("C2_gpt2xl_fc2", 32), ("C3a_megagpt_attn_out", 32),
                                         ("C3b_megagpt_fc2", 32), ("C4_large_fc2", 64)])
def test_inplace_configs_against_oracle(name, stride):
    """The benchmark configurations with the update-in-place reduction: row samples at both tolerances."""
    import torch
    gu = _gu()
    w = wl.by_name(name)
    xb, wb = wl.make_inputs(w)
    rows = wl.sample_rows(w.M, w.R, seed=w.resolved_seed(), stride=stride)
    yref = oracle.gemm_rs(xb, wb, w.R, rows=rows)
    rms = float(np.sqrt(np.mean(yref ** 2)))
    X, W = gu.upload(xb, wb)
    del xb, wb
    ridx = torch.from_numpy(rows).cuda()
    for dtype in (t3.BF16_OUT_BF16, t3.BF16_OUT_F32):
        with t3.Plan(w.M, w.N, w.K, w.R, dtype, t3.chunking(reduce=t3.REDUCE_INPLACE)) as plan:
            info = plan.info()
            assert info.workspace_bytes < 0.3 * 4 * w.R * w.M * w.N or w.R <= 2      # one accumulator, not R copies
            for call in range(2):
                Y = gu.out_tensor(w.M, w.N, dtype)
                gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
                assert oracle.max_rel_err(_to_f64(Y[ridx]), yref, rms=rms) <= TOL[dtype], (name, dtype, call)
            chunk_rms = Y.float().reshape(w.R, w.chunk_rows, w.N).pow(2).mean(dim=(1, 2)).sqrt().cpu().numpy()
            assert np.all(np.abs(chunk_rms / rms - 1.0) < 0.05)
        del Y
    torch.cuda.empty_cache()


def test_inplace_option_checks():
    with pytest.raises(t3.T3Error) as e:      # split-K producers need the update-in-place reduction
        t3.geometry(256, 256, 1024, 2, chunk=t3.chunking(split_k=2))
    assert e.value.code == t3.ERR_UNSUPPORTED
    with pytest.raises(t3.T3Error) as e:      # more producers than k-blocks
        t3.geometry(256, 256, 256, 2, chunk=t3.chunking(split_k=4, reduce=t3.REDUCE_INPLACE))
    assert e.value.code == t3.ERR_INVALID_ARG
    with pytest.raises(t3.T3Error) as e:
        t3.geometry(256, 256, 1024, 2, chunk=t3.chunking(reduce=t3.REDUCE_INPLACE, partial_dtype=t3.PARTIAL_BF16))
    assert e.value.code == t3.ERR_UNSUPPORTED
    g = t3.geometry(4096, 3072, 12288, 8, chunk=t3.chunking(reduce=t3.REDUCE_INPLACE, ring_slots=-1))
    assert g.workspace_bytes < 1.2 * 4 * 4096 * 3072


def test_inplace_recovers_after_timeout():
    """A timed-out call leaves half-accumulated tiles behind; t3_plan_status clears them."""
    gu = _gu()
    M, N, K, R = 512, 512, 1024, 4
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=8)
    want = oracle.gemm_rs(xb, wb, R)
    X, W = gu.upload(xb, wb)
    ch = t3.chunking(reduce=t3.REDUCE_INPLACE, timeout_ms=50, debug_flags=t3.DEBUG_INFLATE_EXPECTED)
    with t3.Plan(M, N, K, R, t3.BF16_OUT_F32, ch) as bad:
        Y = gu.out_tensor(M, N, t3.BF16_OUT_F32)
        bad.gemm_rs(X.data_ptr(), W.data_ptr(), Y.data_ptr(), gu.stream())
        s = bad.status()
        assert s.code == t3.ERR_TIMEOUT and s.where == 4
        # the accumulators were cleared with the status: GEMM + separate reduce on the same plan is exact
        Y2 = gu.out_tensor(M, N, t3.BF16_OUT_F32)
        gu.run_once(bad, t3.MODE_SEQUENTIAL, X, W, Y2)
        assert np.array_equal(_to_f64(Y2), want)


@pytest.mark.parametrize("M", [16, 64, 128])
@pytest.mark.parametrize("N,K,R", [(2048, 8192, 8), (8192, 32768, 16)])
def test_generation_phase_shapes(M, N, K, R):
    """Token-generation shapes (Section 7.3): M <= 128 rows in a 256-row tile.  Ring mode against the
    oracle at both tolerances and bit-identical to the sequential baseline; update-in-place with split-K
    producers against the oracle."""
    gu = _gu()
    w = wl.Workload(f"gen_M{M}", M=M, N=N, K=K, R=R, x_dist="normal", w_dist="normal", w_std=0.02)
    xb, wb = wl.make_inputs(w)
    yref = oracle.gemm_rs(xb, wb, R)
    X, W = gu.upload(xb, wb)
    for dtype in (t3.BF16_OUT_BF16, t3.BF16_OUT_F32):
        with t3.Plan(M, N, K, R, dtype, None) as plan:
            gu.poison_partials(plan)
            Y = gu.out_tensor(M, N, dtype)
            gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
            Y2 = gu.out_tensor(M, N, dtype)
            gu.run_once(plan, t3.MODE_SEQUENTIAL, X, W, Y2)
        assert oracle.max_rel_err(_to_f64(Y), yref) <= TOL[dtype]
        assert np.array_equal(gu.y_bits(Y), gu.y_bits(Y2))
        with t3.Plan(M, N, K, R, dtype, t3.chunking(reduce=t3.REDUCE_INPLACE, split_k=2)) as plan:
            Y = gu.out_tensor(M, N, dtype)
            gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
        assert oracle.max_rel_err(_to_f64(Y), yref) <= TOL[dtype]


# ---------------------------------------------------------------------------
# measured configuration choice, timeline, ordering of launches
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("M,N,K,R,kw", [(256, 512, 2048, 2, {}), (4096, 2048, 8192, 16, {}),
                                        (4096, 3072, 3072, 8, dict(reduce=1))])
def test_tune_keeps_the_bits_and_records_the_choice(M, N, K, R, kw):
    import torch
    gu = _gu()
    w = wl.Workload("t", M=M, N=N, K=K, R=R, x_dist="normal", w_dist="normal", w_std=0.02)
    xb, wb = wl.make_inputs(w)
    rows = wl.sample_rows(M, R, seed=1, stride=32)
    yref = oracle.gemm_rs(xb, wb, R, rows=rows)
    X, W = gu.upload(xb, wb)
    ridx = torch.from_numpy(rows).cuda()
    with t3.Plan(M, N, K, R, t3.BF16_OUT_BF16, t3.chunking(**kw) if kw else None) as plan:
        Y0 = gu.out_tensor(M, N, t3.BF16_OUT_BF16)
        gu.run_once(plan, t3.MODE_FUSED, X, W, Y0)
        Y = gu.out_tensor(M, N, t3.BF16_OUT_BF16)
        res = plan.tune(X.data_ptr(), W.data_ptr(), Y.data_ptr(), gu.stream())
        assert plan.status().code == 0
        info = plan.info()
        cands = res.candidates()
        assert info.tuned == 1 and res.n_tried >= 3 and 0 <= res.chosen < res.n_tried
        assert all(c["us"] > 0 for c in cands)
        best = min(c["us"] for c in cands)
        assert cands[res.chosen]["us"] <= 1.0001 * best or res.chosen == 0
        assert info.mode == cands[res.chosen]["mode"] and info.reduce_rows == cands[res.chosen]["reduce_rows"]
        assert oracle.max_rel_err(_to_f64(Y[ridx]), yref) <= 2e-2
        if not kw:       # ring order: every candidate gives the same bits
            assert np.array_equal(gu.y_bits(Y), gu.y_bits(Y0))
        Y3 = gu.out_tensor(M, N, t3.BF16_OUT_BF16)
        plan.gemm_rs(X.data_ptr(), W.data_ptr(), Y3.data_ptr(), gu.stream())     # t3_gemm_rs follows the choice
        assert plan.status().code == 0
        if not kw:
            assert np.array_equal(gu.y_bits(Y3), gu.y_bits(Y0))


def test_timeline_of_a_fused_call():
    import torch
    gu = _gu()
    w = wl.C3A
    X = torch.randn(w.M, w.K, device="cuda").to(torch.bfloat16)
    W = (torch.randn(w.N, w.K, device="cuda") * 0.02).to(torch.bfloat16)
    Y = gu.out_tensor(w.M, w.N, t3.BF16_OUT_BF16)
    with t3.Plan(w.M, w.N, w.K, w.R, t3.BF16_OUT_BF16, None) as plan:
        with pytest.raises(t3.T3Error):
            plan.timeline()                                  # no fused call yet
        for _ in range(3):
            gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        plan.gemm_rs(X.data_ptr(), W.data_ptr(), Y.data_ptr(), gu.stream())
        e1.record()
        tl = plan.timeline()
        ev_us = 1e3 * e0.elapsed_time(e1)
        assert tl.ctas == plan.info().grid
        assert tl.total_us > 0 and tl.produce_us > 0 and tl.tail_us >= 0 and tl.drain_us >= 0
        assert abs(tl.produce_us + tl.tail_us + tl.drain_us - tl.total_us) < 1e-6
        assert 0.5 * ev_us < tl.total_us < 1.05 * ev_us + 5.0
        assert tl.produce_us > 0.3 * tl.total_us


def test_two_plans_on_two_streams_are_ordered_by_the_library():
    """Two persistent kernels must not share the GPU: calls made from two streams without any
    synchronisation by the caller are serialised by the library and both finish, well inside a short
    bound on the waits."""
    import torch
    gu = _gu()
    M, N, K, R = 2048, 2048, 4096, 8
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=21)
    want = oracle.gemm_rs(xb, wb, R, rows=np.arange(0, M, 37))
    X, W = gu.upload(xb, wb)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    ch = t3.chunking(timeout_ms=200)
    with t3.Plan(M, N, K, R, t3.BF16_OUT_F32, ch) as p1, t3.Plan(M, N, K, R, t3.BF16_OUT_F32, ch) as p2:
        Y1 = gu.out_tensor(M, N, t3.BF16_OUT_F32)
        Y2 = gu.out_tensor(M, N, t3.BF16_OUT_F32)
        torch.cuda.synchronize()
        for _ in range(20):
            p1.gemm_rs(X.data_ptr(), W.data_ptr(), Y1.data_ptr(), s1.cuda_stream)
            p2.gemm_rs(X.data_ptr(), W.data_ptr(), Y2.data_ptr(), s2.cuda_stream)
        assert p1.status().code == 0 and p2.status().code == 0
        torch.cuda.synchronize()
        idx = torch.arange(0, M, 37, device="cuda")
        assert np.array_equal(_to_f64(Y1[idx]), want) and np.array_equal(_to_f64(Y2[idx]), want)


def test_uncollected_timeout_does_not_disturb_later_calls():
    """An uncollected timeout of one call must not make later calls on the plan give up early."""
    gu = _gu()
    M, N, K, R = 512, 512, 1024, 4
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=4)
    want = oracle.gemm_rs(xb, wb, R)
    X, W = gu.upload(xb, wb)
    ch = t3.chunking(timeout_ms=50, debug_flags=t3.DEBUG_INFLATE_EXPECTED)
    with t3.Plan(M, N, K, R, t3.BF16_OUT_F32, ch) as bad:
        Y = gu.out_tensor(M, N, t3.BF16_OUT_F32)
        bad.gemm_rs(X.data_ptr(), W.data_ptr(), Y.data_ptr(), gu.stream())          # times out; not collected
        Y2 = gu.out_tensor(M, N, t3.BF16_OUT_F32)
        bad.gemm_rs_mode(t3.MODE_SEQUENTIAL, X.data_ptr(), W.data_ptr(), Y2.data_ptr(), gu.stream())   # no trigger involved
        s = bad.status()
        assert s.code == t3.ERR_TIMEOUT                      # the first call's report is still there ...
        assert np.array_equal(_to_f64(Y2), want)             # ... and the later call ran to completion


# ---------------------------------------------------------------------------
# guard bands: nothing is written outside Y or the export buffer
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("M,N,K,R", [(1000, 520, 1024, 8), (200, 264, 512, 2), (130, 264, 512, 2), (2, 8, 16, 2)])
@pytest.mark.parametrize("dtype", [t3.BF16_OUT_BF16, t3.BF16_OUT_F32])
def test_guard_bands_around_y_and_export_buffer(M, N, K, R, dtype):
    import torch
    gu = _gu()
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=M + 1)
    want = oracle.gemm_rs(xb, wb, R)
    X, W = gu.upload(xb, wb)
    esz = 4 if dtype == t3.BF16_OUT_F32 else 2
    tdt = torch.float32 if dtype == t3.BF16_OUT_F32 else torch.bfloat16
    for kw in ({}, dict(reduce=t3.REDUCE_INPLACE)):
        for mode in (t3.MODE_FUSED, t3.MODE_SEQUENTIAL):
            whole, off = gu.banded(M * N * esz)
            Y = whole[off:off + M * N * esz].view(tdt).view(M, N)
            with t3.Plan(M, N, K, R, dtype, t3.chunking(mode=mode, **kw)) as plan:
                gu.run_once(plan, mode, X, W, Y)
                if not kw and mode == t3.MODE_SEQUENTIAL:
                    pw, poff = gu.banded(4 * R * M * N)
                    plan.export_partials(pw.data_ptr() + poff, gu.stream())
                    torch.cuda.synchronize()
                    assert gu.bands_intact(pw), "export wrote outside its buffer"
                    P = pw[poff:poff + 4 * R * M * N].view(torch.float32).view(R, M, N).cpu().numpy()
                    assert np.array_equal(P.astype(np.float64).sum(axis=0), want)
            torch.cuda.synchronize()
            assert gu.bands_intact(whole), f"wrote outside Y: {kw} mode {mode}"
            got = _to_f64(Y)
            ref = want if dtype == t3.BF16_OUT_F32 else wl.bf16_bits_to_f64(wl.f32_to_bf16_bits(want.astype(np.float32)))
            assert np.array_equal(got, ref)

