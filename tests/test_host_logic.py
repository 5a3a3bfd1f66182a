"""CPU-only checks of the C-ABI library's host logic: exported symbols, argument
validation, plan geometry, producer schedule, tracker thresholds, ring order."""
import ctypes
import os
import re
import sys
from collections import Counter

import pytest

import oracle
from paper_2401_16677_b200 import build as t3build
from paper_2401_16677_b200 import t3
from paper_2401_16677_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    t3build.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "t3.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(t3_[a-z_0-9]+)\s*\(", hdr))
    assert {"t3_plan", "t3_gemm_rs", "t3_destroy"} <= declared
    here = os.path.dirname(os.path.abspath(t3.__file__))
    libs = {t3.LIB_PATH, os.path.join(here, "libt3.so")}          # the variant in use and the portable build
    for path in sorted(libs):
        L = ctypes.CDLL(path)
        for name in sorted(declared):
            assert hasattr(L, name), f"{name} declared in t3.h but not exported by {os.path.basename(path)}"
    assert declared == set(t3.EXPORTS)
    assert t3.version() == 110


def test_shape_validation_codes():
    ok = dict(M=256, N=512, K=2048, R=2)
    t3.geometry(**ok)
    bad = [
        (dict(ok, M=255), t3.ERR_SHAPE),          # M % R
        (dict(ok, K=2050), t3.ERR_SHAPE),         # (K/R) % 8
        (dict(ok, K=2049), t3.ERR_SHAPE),         # K % R
        (dict(ok, N=500), t3.ERR_SHAPE),          # N % 8
        (dict(ok, M=0), t3.ERR_INVALID_ARG),
        (dict(ok, R=0), t3.ERR_INVALID_ARG),
        (dict(ok, N=-8), t3.ERR_INVALID_ARG),
    ]
    for kw, code in bad:
        with pytest.raises(t3.T3Error) as e:
            t3.geometry(**kw)
        assert e.value.code == code, kw
        assert t3.last_error() == code
    with pytest.raises(t3.T3Error):
        t3.geometry(**ok, dtype=7)
    with pytest.raises(t3.T3Error):
        t3.geometry(**ok, chunk=t3.chunking(tile_n=100))
    with pytest.raises(t3.T3Error):
        t3.geometry(**ok, chunk=t3.chunking(mode=9))
    assert "shape" in t3.strerror(t3.ERR_SHAPE)


def test_geometry_of_the_benchmark_configs():
    g = t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R)
    assert (g.tile_m, g.tile_n, g.n_m_tiles, g.n_n_tiles) == (256, 160, 32, 10)
    assert g.K_r == 800 and g.k_blocks == 13 and g.chunk_rows == 1024
    assert g.n_jobs == 32 * 10 * 8 and g.n_regions == 320
    assert g.flops == 2.0 * 8192 * 1600 * 6400
    assert g.bytes_gemm == 2 * 8192 * 6400 + 2 * 6400 * 1600 + 4 * 8 * 8192 * 1600
    assert g.bytes_reduce == 4 * 8 * 8192 * 1600 + 2 * 8192 * 1600
    assert g.bytes_fused == g.bytes_gemm + g.bytes_reduce
    assert g.smem_bytes <= 227 * 1024
    g4 = t3.geometry(wl.C4.M, wl.C4.N, wl.C4.K, wl.C4.R, t3.BF16_OUT_F32)
    assert (g4.tile_n, g4.n_n_tiles, g4.k_blocks) == (256, 32, 32)
    assert g4.bytes_reduce == 4 * 16 * 4096 * 8192 + 4 * 4096 * 8192
    g1 = t3.geometry(wl.C1.M, wl.C1.N, wl.C1.K, wl.C1.R)
    assert g1.n_jobs == 1 * 2 * 2 and g1.gemm_ctas == 8      # 4 jobs, one CTA pair each


@pytest.mark.parametrize("M,N,K,R,kw", [
    (256, 512, 2048, 2, {}),
    (8192, 1600, 6400, 8, {}),
    (1024, 2048, 8192, 16, {}),              # 64-row chunks: a 256-row tile spans four chunks
    (1152, 264, 512, 4, dict(group_tiles=4, tile_n=64)),   # ragged last group and last column tile
    (4096, 3072, 3072, 8, dict(group_tiles=1)),
    (200, 96, 64, 2, dict(reduce_rows=16)),  # M not a multiple of the tile height, half-chunk items
    (640, 512, 512, 4, dict(group_tiles=2)),  # odd number of 128-row halves: last pair half empty
])
def test_schedule_and_tracker_arithmetic(M, N, K, R, kw):
    ch = t3.chunking(**kw) if kw else None
    g = t3.geometry(M, N, K, R, chunk=ch)
    jobs = t3.schedule(M, N, K, R, chunk=ch)
    assert len(jobs) == g.n_jobs == g.n_m_tiles * g.n_n_tiles * R
    # every (row tile, column tile, slice) exactly once
    cnt = Counter(jobs)
    assert len(cnt) == len(jobs)
    assert set(cnt) == {(mt, nt, r) for mt in range(g.n_m_tiles) for nt in range(g.n_n_tiles) for r in range(R)}
    # tracker threshold = landed units per producer tile (one per CTA of the pair) x updates per element (R)
    assert g.expected == 2 * R
    per_region = Counter((mt, nt) for mt, nt, _ in jobs)
    assert all(v * 2 == g.expected for v in per_region.values())
    assert sum(per_region.values()) * 2 == g.n_regions * g.expected
    # a region's R partials are produced within group_tiles * R consecutive jobs
    first, last = {}, {}
    for j, (mt, nt, _) in enumerate(jobs):
        first.setdefault((mt, nt), j)
        last[(mt, nt)] = j
    assert max(last[k] - first[k] for k in first) < g.group_tiles * R
    # reducer tickets: every output row/column block exactly once, in completion order
    items = t3.reduce_schedule(M, N, K, R, chunk=ch)
    assert len(items) == g.n_reduce_items
    covered = Counter()
    for mt, nt, row0, nrows, col0, ncols in items:
        if nrows == 0 or ncols == 0:          # item wholly in the padding of a ragged tile
            assert nrows == 0 and ncols == 0
            assert row0 >= M or col0 >= min(N, (nt + 1) * g.tile_n)
            continue
        assert nrows <= g.reduce_rows and ncols <= 32 and ncols % 8 == 0
        assert mt * g.tile_m <= row0 and row0 + nrows <= min(M, (mt + 1) * g.tile_m)
        assert nt * g.tile_n <= col0 and col0 + ncols <= min(N, (nt + 1) * g.tile_n)
        for row in range(row0, row0 + nrows):
            covered[(row, col0 // 8)] += ncols // 8      # count 8-column groups
    assert set(covered) == {(m, c) for m in range(M) for c in range(N // 8) if c * 8 % g.tile_n % 32 == 0}
    total = sum(covered.values())
    assert total == M * (N // 8), "every output element belongs to exactly one reducer item"
    done_at = [last[(mt, nt)] for mt, nt, *_ in items]
    assert done_at == sorted(done_at), "tickets must follow region completion order"


def test_ring_order_agrees_with_oracle_and_paper_example():
    assert t3.ring_order(0, 4) == [3, 2, 1, 0]
    assert t3.ring_order(3, 4) == [2, 1, 0, 3]
    for R in (1, 2, 3, 8, 16):
        for c in range(R):
            assert t3.ring_order(c, R) == oracle.ring_order(c, R)
    with pytest.raises(t3.T3Error):
        t3.ring_order(4, 4)


def test_ring_slot_rules():
    g = t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R)
    assert g.ring_slots >= g.group_tiles and g.ring_slots < g.n_regions
    assert g.ring_slots * 8 * 256 * 160 * 4 <= 64 << 20      # the ring is sized to stay inside L2
    assert t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(ring_slots=-1)).ring_slots == 0
    assert t3.geometry(wl.C1.M, wl.C1.N, wl.C1.K, wl.C1.R).ring_slots == 0     # everything fits: no recycling
    with pytest.raises(t3.T3Error):      # fewer slots than the schedule group height could deadlock
        t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(ring_slots=2, group_tiles=4))


def test_sm_split_options():
    g = t3.geometry(4096, 3072, 3072, 8, chunk=t3.chunking(reducer_ctas=16, reducer_warps=-1))
    assert (g.grid, g.gemm_ctas, g.reducer_ctas, g.reducer_warps) == (148, 132, 16, 0)
    with pytest.raises(t3.T3Error):   # fused mode with nobody to reduce
        t3.geometry(4096, 3072, 3072, 8, chunk=t3.chunking(reducer_warps=-1))
    g = t3.geometry(4096, 3072, 3072, 8, chunk=t3.chunking(mode=t3.MODE_SEQUENTIAL, reducer_warps=-1))
    assert g.reducer_warps == 0


def test_cluster_size_rules():
    # one CTA pair per cluster always works; two pairs per cluster need the library variant that holds
    # that kernel and an even number of 256-row tiles in every schedule group
    g2 = t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(cluster_ctas=2))
    assert g2.cluster_ctas == 2 and g2.grid % 2 == 0
    with pytest.raises(t3.T3Error):
        t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(cluster_ctas=3))
    assert t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R).cluster_ctas == 2      # short problem: all SMs, pairs
    auto = t3.geometry(wl.C4.M, wl.C4.N, wl.C4.K, wl.C4.R)                        # long, power-limited problem
    if t3.shared_fetch_available():
        assert auto.cluster_ctas == 4
        auto = t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(cluster_ctas=4))
        assert auto.cluster_ctas == 4 and auto.grid % 4 == 0 and auto.gemm_ctas % 4 == 0
        # same tiles, same schedule, same tracker arithmetic: only the fetch of W is shared
        for f in ("tile_n", "n_jobs", "n_regions", "expected", "group_tiles", "n_reduce_items", "ring_slots"):
            assert getattr(auto, f) == getattr(g2, f), f
        assert t3.schedule(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(cluster_ctas=4)) == \
            t3.schedule(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(cluster_ctas=2))
        # jobs j, j + 1 (j even) of a 4-CTA cluster: vertically adjacent tiles of one W tile and slice
        jobs = t3.schedule(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(cluster_ctas=4))
        for j in range(0, len(jobs), 2):
            (m0, n0, r0), (m1, n1, r1) = jobs[j], jobs[j + 1]
            assert (m1, n1, r1) == (m0 + 1, n0, r0)
        with pytest.raises(t3.T3Error):      # 3 row tiles: a pair of pairs would straddle W tiles
            t3.geometry(768, 512, 512, 4, chunk=t3.chunking(cluster_ctas=4))
        assert t3.geometry(768, 512, 512, 4).cluster_ctas == 2
        with pytest.raises(t3.T3Error):      # odd group height
            t3.geometry(1024, 512, 512, 4, chunk=t3.chunking(cluster_ctas=4, group_tiles=1))
        with pytest.raises(t3.T3Error):      # reducer-only CTAs come in whole clusters
            t3.geometry(1024, 512, 512, 4, chunk=t3.chunking(cluster_ctas=4, reducer_ctas=6))
    else:
        assert auto.cluster_ctas == 2
        with pytest.raises(t3.T3Error):
            t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(cluster_ctas=4))


def test_partial_dtype_option():
    g32 = t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R)
    g16 = t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(partial_dtype=t3.PARTIAL_BF16))
    assert (g32.partial_dtype, g16.partial_dtype) == (t3.PARTIAL_F32, t3.PARTIAL_BF16)
    RMN = wl.C2.R * wl.C2.M * wl.C2.N
    # the reduction traffic of the cost model halves; operands and Y do not change
    assert g32.bytes_fused - g16.bytes_fused == pytest.approx(2 * 2.0 * RMN)
    assert g32.bytes_gemm - g16.bytes_gemm == pytest.approx(2.0 * RMN)
    # same bytes of ring, twice the region slots
    assert g16.ring_slots in (2 * g32.ring_slots, 2 * g32.ring_slots + 1)
    with pytest.raises(t3.T3Error):
        t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(partial_dtype=2))


def test_w_layout_option():
    g = t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(w_layout=t3.W_KN))
    assert g.w_layout == t3.W_KN and g.tile_n in (128, 256)     # each CTA's half tile is whole 64-column boxes
    assert t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R).w_layout == t3.W_NK
    with pytest.raises(t3.T3Error):
        t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(w_layout=t3.W_KN, tile_n=160))
    with pytest.raises(t3.T3Error):
        t3.geometry(wl.C2.M, wl.C2.N, wl.C2.K, wl.C2.R, chunk=t3.chunking(w_layout=2))


def test_staggered_order_follows_the_ring_steps():
    # Section 4.4: in step s device r produces chunk (r + s + 1) mod R; its own chunk comes last
    M, N, K, R = 4096, 1024, 2048, 4
    ch = t3.chunking(order=t3.ORDER_STAGGERED)
    g = t3.geometry(M, N, K, R, chunk=ch)
    assert g.order == t3.ORDER_STAGGERED and g.ring_slots == 0 and g.cluster_ctas == 2
    jobs = t3.schedule(M, N, K, R, chunk=ch)
    assert sorted(jobs) == sorted(t3.schedule(M, N, K, R))          # the same jobs, another order
    tiles_per_chunk = (M // R) // g.tile_m
    per_step = len(jobs) // R
    for j, (mt, nt, r) in enumerate(jobs):
        step = j // per_step
        assert mt // tiles_per_chunk == (r + step + 1) % R
    for mt, nt, r in jobs[-per_step:]:
        assert mt // tiles_per_chunk == r                             # last step: every device on its own chunk
    # a region only completes in the last step
    last = {}
    for j, (mt, nt, _) in enumerate(jobs):
        last[(mt, nt)] = j
    assert min(last.values()) >= (R - 1) * per_step
    items = t3.reduce_schedule(M, N, K, R, chunk=ch)
    done_at = [last[(mt, nt)] for mt, nt, *_ in items]
    assert done_at == sorted(done_at), "tickets must follow region completion order"
    with pytest.raises(t3.T3Error):          # chunks of 64 rows are not whole tiles
        t3.geometry(1024, 2048, 8192, 16, chunk=ch)


def test_plan_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(t3.T3Error) as e:
        t3.Plan(256, 512, 2048, 2)
    assert e.value.code == t3.ERR_DEVICE
    assert t3.lib().t3_gemm_rs(None, None, None, None, None) == t3.ERR_INVALID_ARG
    assert t3.lib().t3_destroy(None) == 0


def test_multicast_variant_is_never_chosen_in_a_multi_process_launch():
    """The library variant with the multicast W fetch is for one process on one GPU: any launch with
    WORLD_SIZE or LOCAL_WORLD_SIZE above 1 gets the portable library, whatever files exist and whatever
    T3_LIB_PATH asks for."""
    here = os.path.dirname(os.path.abspath(t3.__file__))
    portable = os.path.join(here, "libt3.so")
    sf = os.path.join(here, "libt3_sf.so")
    for env in ({"WORLD_SIZE": "2"}, {"LOCAL_WORLD_SIZE": "8"}, {"WORLD_SIZE": "2", "T3_LIB_PATH": sf},
                {"WORLD_SIZE": "junk"}):
        assert t3.multi_process_launch(env)
        assert t3.choose_lib_path(env) == portable, env
    assert not t3.multi_process_launch({"WORLD_SIZE": "1"})
    assert not t3.multi_process_launch({})
    assert t3.choose_lib_path({"T3_LIB_PATH": "/x/y.so"}) == "/x/y.so"
    # a fresh interpreter started as rank 0 of 2 binds the portable library
    import subprocess
    env = dict(os.environ, WORLD_SIZE="2", RANK="0")
    env.pop("T3_LIB_PATH", None)
    out = subprocess.check_output([sys.executable, "-c",
                                   "from paper_2401_16677_b200 import t3; print(t3.LIB_PATH); "
                                   "print(t3.shared_fetch_available())"], cwd=ROOT, env=env, text=True).split()
    assert out[0] == portable and out[1] == "False"


def test_environment_overrides_fill_only_fields_left_at_zero():
    import subprocess
    code = ("from paper_2401_16677_b200 import t3; "
            "g = t3.geometry(4096, 3072, 12288, 8); "
            "h = t3.geometry(4096, 3072, 12288, 8, chunk=t3.chunking(group_tiles=2, ring_slots=20)); "
            "print(g.group_tiles, g.ring_slots, g.reduce_rows, h.group_tiles, h.ring_slots)")
    env = dict(os.environ, T3_GROUP_TILES="4", T3_RING_SLOTS="24", T3_REDUCE_ROWS="16", T3_TIMEOUT_MS="junk")
    out = subprocess.check_output([sys.executable, "-c", code], cwd=ROOT, env=env, text=True).split()
    assert out == ["4", "24", "16", "2", "20"]
    base = t3.geometry(4096, 3072, 12288, 8)
    assert (base.group_tiles, base.reduce_rows) == (8, 32)
