"""t3_gemm_rs_static: the entry point for callers that may not allocate device memory (a latency-bound
service thread that cannot take cudaMalloc's device-wide synchronisation, a process whose device memory
is all held by its own pool).  Its scratch is a static device array inside the library, so the test
checks what such a caller relies on: same bits as the plan-based entry point, call after call, with the
array reused (and its tracker words cleared) between calls; and, independently of the plan entry, the
CPU oracle's values (bit for bit on exact-integer inputs, within the output tolerance on config 1).

Collected last on purpose: a failure here cannot hide the other tests under `-x`."""
import numpy as np
import pytest

import oracle
from paper_2401_16677_b200 import build as t3build
from paper_2401_16677_b200 import t3
from paper_2401_16677_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    t3build.build()


def _reference_bits(M, N, K, R, dtype, X, W):
    import gpu_util as gu
    Y = gu.out_tensor(M, N, dtype)
    with t3.Plan(M, N, K, R, dtype, None) as plan:
        gu.run_once(plan, t3.MODE_FUSED, X, W, Y)
    return gu.y_bits(Y)


def test_static_scratch_entry_matches_plan_entry_twice_in_a_row():
    import torch
    import gpu_util as gu
    cases = [
        # first call: config 1 (1 MiB of partial tiles); second call: a different, larger shape with
        # ragged edges (15.6 MiB), so the second call starts on whatever the first one left behind
        (wl.C1.M, wl.C1.N, wl.C1.K, wl.C1.R, t3.BF16_OUT_BF16, "c1"),
        (1000, 520, 1024, 8, t3.BF16_OUT_F32, "ragged"),
        (wl.C1.M, wl.C1.N, wl.C1.K, wl.C1.R, t3.BF16_OUT_BF16, "c1"),
    ]
    st = gu.stream()
    for M, N, K, R, dtype, kind in cases:
        if kind == "c1":
            xb, wb = wl.make_inputs(wl.C1)
        else:
            xb, wb = wl.make_small_int_inputs(M, N, K, seed=11)
        X, W = gu.upload(xb, wb)
        want = _reference_bits(M, N, K, R, dtype, X, W)
        for call in range(2):                               # two calls in a row on the shared array
            Y = gu.out_tensor(M, N, dtype)
            t3.gemm_rs_static(M, N, K, R, dtype, X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)
            torch.cuda.synchronize()
            got = gu.y_bits(Y)
            assert np.array_equal(got, want), f"{kind}: call {call} differs from t3_gemm_rs"
            # and against the oracle itself, not only against the other entry point
            yref = oracle.gemm_rs(xb, wb, R)
            yf = Y.float().cpu().numpy().astype(np.float64)
            if kind == "c1":
                assert oracle.max_rel_err(yf, yref) <= 2e-2
            else:
                assert np.array_equal(yf, yref), f"{kind}: call {call} differs from the oracle"


def test_static_scratch_entry_rejects_what_does_not_fit():
    import gpu_util as gu
    M, N, K, R = 4096, 1024, 512, 4          # 64 MiB of partial tiles > 32 MiB of static scratch
    assert 4 * R * M * N > t3.STATIC_SCRATCH_BYTES
    xb, wb = wl.make_small_int_inputs(M, N, K, seed=3)
    X, W = gu.upload(xb, wb)
    Y = gu.out_tensor(M, N, t3.BF16_OUT_BF16)
    with pytest.raises(t3.T3Error) as e:
        t3.gemm_rs_static(M, N, K, R, t3.BF16_OUT_BF16, X.data_ptr(), W.data_ptr(), Y.data_ptr(), gu.stream())
    assert e.value.code == t3.ERR_TOO_LARGE
    with pytest.raises(t3.T3Error) as e:     # shape rules are those of t3_plan
        t3.gemm_rs_static(255, 256, 256, 2, t3.BF16_OUT_BF16, X.data_ptr(), W.data_ptr(), Y.data_ptr(), gu.stream())
    assert e.value.code == t3.ERR_SHAPE
