"""The benchmark configurations at full size, in the launch configuration the
bench times (default chunking), checked on a row sample the oracle can
compute exactly: every 16th (32nd) row plus the first and last row of every
reduce-scatter chunk, all N columns, full K."""
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


@pytest.mark.parametrize("name,stride", [
    ("C2_gpt2xl_fc2", 16), ("C3a_megagpt_attn_out", 16), ("C3b_megagpt_fc2", 16), ("C4_large_fc2", 32),
    ("X_megagpt_bwd_ip", 32),        # backward input projection: K = 3H
])
def test_full_config_row_sample(name, stride):
    import torch
    import gpu_util as gu
    w = wl.by_name(name)
    xb, wb = wl.make_inputs(w)
    rows = wl.sample_rows(w.M, w.R, seed=w.resolved_seed(), stride=stride)
    yref = oracle.gemm_rs(xb, wb, w.R, rows=rows)
    rms = float(np.sqrt(np.mean(yref ** 2)))
    X, W = gu.upload(xb, wb)
    del xb, wb
    for out in w.out:
        dtype = t3.BF16_OUT_F32 if out == "f32" else t3.BF16_OUT_BF16
        Y = gu.out_tensor(w.M, w.N, dtype)
        with t3.Plan(w.M, w.N, w.K, w.R, dtype, None) as plan:
            gu.poison_partials(plan)
            assert plan.info().ring_slots > 0          # the benchmark configuration recycles a ring of region slots
            gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
            Yf = Y.float()
            assert bool(torch.isfinite(Yf).all())
            # fused and sequential agree bit for bit over the whole output
            Y2 = gu.out_tensor(w.M, w.N, dtype)
            gu.run_once(plan, t3.MODE_SEQUENTIAL, X, W, Y2)
            assert torch.equal(Y.view(torch.int16 if dtype == t3.BF16_OUT_BF16 else torch.int32),
                               Y2.view(torch.int16 if dtype == t3.BF16_OUT_BF16 else torch.int32))
        got = Yf[torch.from_numpy(rows).cuda()].cpu().numpy()
        err = oracle.max_rel_err(got, yref, rms=rms)
        assert err <= TOL[dtype], (name, out, err)
        # property that holds at any size: every chunk has the full sum's scale (no missed slice)
        cr = w.chunk_rows
        chunk_rms = Yf.reshape(w.R, cr, w.N).pow(2).mean(dim=(1, 2)).sqrt().cpu().numpy()
        assert np.all(np.abs(chunk_rms / rms - 1.0) < 0.05), chunk_rms / rms
        del Y, Y2, Yf
    torch.cuda.empty_cache()


def test_sweep_corner_small_chunks():
    """Sweep corner R=16, M=1024 (64-row chunks inside 128-row tiles), H=2048."""
    import torch
    import gpu_util as gu
    w = wl.by_name("C5_R16_M1024_H2048")
    xb, wb = wl.make_inputs(w)
    rows = wl.sample_rows(w.M, w.R, seed=w.resolved_seed(), stride=8)
    yref = oracle.gemm_rs(xb, wb, w.R, rows=rows)
    X, W = gu.upload(xb, wb)
    Y = gu.out_tensor(w.M, w.N, t3.BF16_OUT_BF16)
    with t3.Plan(w.M, w.N, w.K, w.R, t3.BF16_OUT_BF16, None) as plan:
        gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
    got = Y.float()[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert oracle.max_rel_err(got, yref) <= 2e-2


def test_backward_fc1_with_w_stored_k_by_n_and_16_bit_partials():
    """The FC-1 input-gradient sublayer (K = 4H) with the weight taken as stored [K][N] and the
    partial tiles on a 16-bit wire: row sample against the oracle at the bf16 tolerance."""
    import torch
    import gpu_util as gu
    w = wl.by_name("X_megagpt_bwd_fc1")
    xb, wb = wl.make_inputs(w)
    rows = wl.sample_rows(w.M, w.R, seed=w.resolved_seed(), stride=32)
    yref = oracle.gemm_rs(xb, wb, w.R, rows=rows)
    X = gu.to_device_bf16(xb)
    W = gu.to_device_bf16(wb)                       # [K][N]
    Y = gu.out_tensor(w.M, w.N, t3.BF16_OUT_BF16)
    ch = t3.chunking(w_layout=t3.W_KN, partial_dtype=t3.PARTIAL_BF16)
    with t3.Plan(w.M, w.N, w.K, w.R, t3.BF16_OUT_BF16, ch) as plan:
        gu.poison_partials(plan)
        gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
        Y2 = gu.out_tensor(w.M, w.N, t3.BF16_OUT_BF16)
        gu.run_once(plan, t3.MODE_SEQUENTIAL, X, W, Y2)
    assert torch.equal(Y.view(torch.int16), Y2.view(torch.int16))
    got = Y.float()[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert oracle.max_rel_err(got, yref) <= 2e-2


SWEEP = [w.name for w in wl.sweep_points()]
# the four points with the largest partial workspace (4*R*M*N): also checked with fp32 output at 1e-4
SWEEP_F32 = {w.name for w in sorted(wl.sweep_points(), key=lambda w: (w.R * w.M * w.N, w.K))[-4:]}


@pytest.mark.parametrize("name", SWEEP)
def test_sweep_point_row_sample(name):
    """Every point of the shape sweep (R x M x H grid, K = 4H) at full size, default chunking, fused
    mode - the launch configuration the bench's sweep times - on a row sample the oracle computes
    exactly: every 64th row plus the first and last row of every chunk, all N columns, full K.  These
    are the sizes at which element offsets pass 2^31 and the partial workspace reaches 8.6 GB."""
    import torch
    import gpu_util as gu
    w = wl.by_name(name)
    xb, wb = wl.make_inputs(w)
    rows = wl.sample_rows(w.M, w.R, seed=w.resolved_seed(), stride=64)
    yref = oracle.gemm_rs(xb, wb, w.R, rows=rows)
    rms = float(np.sqrt(np.mean(yref ** 2)))
    X, W = gu.upload(xb, wb)
    del xb, wb
    ridx = torch.from_numpy(rows).cuda()
    dtypes = [t3.BF16_OUT_BF16] + ([t3.BF16_OUT_F32] if name in SWEEP_F32 else [])
    for dtype in dtypes:
        Y = gu.out_tensor(w.M, w.N, dtype)
        with t3.Plan(w.M, w.N, w.K, w.R, dtype, None) as plan:
            gu.poison_partials(plan)
            gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
        assert bool(torch.isfinite(Y.float()).all())
        err = oracle.max_rel_err(Y[ridx].float().cpu().numpy(), yref, rms=rms)
        assert err <= TOL[dtype], (name, dtype, err)
        # no missed slice anywhere: every chunk has the full sum's scale
        chunk_rms = Y.float().reshape(w.R, w.chunk_rows, w.N).pow(2).mean(dim=(1, 2)).sqrt().cpu().numpy()
        assert np.all(np.abs(chunk_rms / rms - 1.0) < 0.08), chunk_rms / rms
        del Y
    del X, W
    torch.cuda.empty_cache()
