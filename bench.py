#!/usr/bin/env python
"""Benchmark of the fused GEMM + reduce-scatter reduction on B200.

A "step" is one pass of the whole hot path over one synthetic batch: the
fused kernel (producer GEMM per K-slice, partial stores, tracker, triggered
ring-order reduction) on the largest single-GPU configuration, the large-model
FC-2 sublayer (R=16, M=4096, K=32768, N=8192, bf16 output), unless --workload
says otherwise.  The same JSON line carries `per_config`: the other
configurations (tiny, GPT-2-XL-like FC-2, Mega-GPT-like attention-out and
FC-2, the large FC-2 with fp32 output) with the four modes timed interleaved.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
  python bench.py --impl reference ...      # the CPU oracle on the host cores

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run)
every rank runs an independent replica of the same sublayer on its own GPU;
no data-path collective exists on this path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused_gemm_rs_tflops"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "C4_large_fc2"
L2_FLUSH_BYTES = 512 << 20

# DRAM traffic of one fused-kernel launch (dram__bytes_read.sum + dram__bytes_write.sum) as captured by
# ncu in an EARLIER, separate run (never measured inside this script): bytes per launch and the summary
# under profiles/ that holds the capture's command and figures.  Absent: no capture for that workload.
NCU_TRAFFIC = {
    "C2_gpt2xl_fc2": (708.1e6, "profiles/t3_fused_kernel_C2.md"),
    "C3b_megagpt_fc2": (1272.4e6, "profiles/t3_fused_kernel_C3b.md"),
    # captured on the same shape scaled to M = 1 024 (1.555 GB per launch); traffic is proportional to M there
    "C4_large_fc2": (4 * 1.555e9, "profiles/t3_fused_kernel_C4_scaled.md, x4 from the M = 1 024 capture"),
}
CHUNK_ARGS = ("tile_n", "group_tiles", "reducer_ctas", "reducer_warps", "reduce_rows", "stages", "ring_slots", "cluster_ctas",
              "partial_dtype", "order", "reduce", "split_k", "l2_hints")
PER_CONFIG = ["C1_tiny", "C2_gpt2xl_fc2", "C3a_megagpt_attn_out", "C3b_megagpt_fc2", "C4_large_fc2:f32"]


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            h = None
            for i in range(pynvml.nvmlDeviceGetCount()):
                hi = pynvml.nvmlDeviceGetHandleByIndex(i)
                u = pynvml.nvmlDeviceGetUUID(hi)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u:
                    h = hi
                    break
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._h = h
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    _REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
        0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown",
    }

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                self.samples.append(mhz)
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self._REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self._h is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": int(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _cpu_oracle_sample(w, xb, wb, budget_s: float, block_rows: int = 256):
    """Times the oracle as it stands on blocks of rows until ~budget_s of CPU work."""
    import numpy as np
    import oracle
    done_rows, t_total = 0, 0.0
    start = 0
    while start < w.M and t_total < budget_s:
        rows = np.arange(start, min(w.M, start + block_rows), dtype=np.int64)
        t0 = time.perf_counter()
        oracle.gemm_rs(xb, wb, w.R, rows=rows)
        t_total += time.perf_counter() - t0
        done_rows += len(rows)
        start += block_rows
    flops = 2.0 * done_rows * w.N * w.K
    return dict(value=flops / t_total / 1e12, unit=UNIT, cores=oracle.threads(), kind="oracle",
                sample=f"rows 0..{done_rows - 1} of {w.M} (all N, full K, R={w.R}), {t_total:.1f} s of CPU work")


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import numpy as np
    import oracle
    from paper_2401_16677_b200 import workloads as wl
    w = wl.by_name(args.workload)
    xb, wb = wl.make_inputs(w)
    rows_per_step = max(8, min(w.M, int(2.0e10 / (2.0 * w.N * w.K))))   # ~20 GFLOP per step
    rows_per_step = min(rows_per_step, 256)
    times = []
    for it in range(args.warmup + args.steps):
        start = (it * rows_per_step) % max(1, w.M - rows_per_step + 1)
        rows = np.arange(start, start + rows_per_step, dtype=np.int64)
        t0 = time.perf_counter()
        oracle.gemm_rs(xb, wb, w.R, rows=rows)
        dt = time.perf_counter() - t0
        if it >= args.warmup:
            times.append(dt)
    total = sum(times)
    flops = 2.0 * rows_per_step * w.N * w.K * len(times)
    value = flops / total / 1e12
    sample = f"{rows_per_step} rows of {w.M} per step (all N, full K, R={w.R})"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "N": w.N, "K": w.K, "R": w.R, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def _time_mode(torch, plan, mode, X, W, Y, st, steps, warmup, flush_buf):
    """CUDA-event time of `steps` calls, L2 flushed (outside the events) before each."""
    for _ in range(warmup):
        if flush_buf is not None:
            flush_buf.zero_()
        plan.gemm_rs_mode(mode, X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    torch.cuda.synchronize()
    for a, b in evs:
        if flush_buf is not None:
            flush_buf.zero_()
        a.record()
        plan.gemm_rs_mode(mode, X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)
        b.record()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    s = plan.status()
    if s.code != 0:
        raise RuntimeError(f"device status {s.code} (where={s.where}, block={s.block}, detail={s.detail})")
    return ms


def _max_over_ranks(value: float, dist, device) -> float:
    """Max of a per-rank time over all ranks (identity without a process group)."""
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def _whole_job_value(world: int, flops_per_replica: float, ms_per_step: float) -> float:
    """TFLOP/s of all replicas together: every rank runs the same sublayer (weak scaling)."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


MODE_NAMES = ("fused", "sequential", "gemm_only", "reduce_only")


def _interleaved(torch, t3, plan, X, W, Y, st, flush, rounds, per_round):
    """The four modes timed round-robin on one plan (same tile shape, schedule and workspace), L2 flushed
    before every call: `rounds` rounds of `per_round` calls per mode.  Returns per mode the list of
    per-round medians in microseconds, and the fused kernel's timeline medians."""
    modes = (t3.MODE_FUSED, t3.MODE_SEQUENTIAL, t3.MODE_GEMM_ONLY, t3.MODE_REDUCE_ONLY)
    for m in (t3.MODE_GEMM_ONLY,) + modes:       # reduce-only needs valid partial tiles; then one warm call each
        flush.zero_()
        plan.gemm_rs_mode(m, X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)
    torch.cuda.synchronize()
    us = {n: [] for n in MODE_NAMES}
    tl = {"produce_us": [], "tail_us": [], "drain_us": [], "total_us": []}
    for _ in range(rounds):
        for name, m in zip(MODE_NAMES, modes):
            ms = _time_mode(torch, plan, m, X, W, Y, st, per_round, 0, flush)
            us[name].append(1e3 * statistics.median(ms))
            if m == t3.MODE_FUSED:
                t = plan.timeline()
                for k in tl:
                    tl[k].append(getattr(t, k))
    return us, {k: statistics.median(v) for k, v in tl.items()}


def _overlap_figures(us, timeline):
    """Exposed / hidden reduction from the per-round medians (Section 5.3's configurations: Sequential,
    and the ideal overlap max(GEMM, RS))."""
    med = statistics.median
    f, q, g, r = (med(us[n]) for n in MODE_NAMES)
    per_round_hidden = [1.0 - max(0.0, fi - gi) / ri for fi, gi, ri in zip(us["fused"], us["gemm_only"], us["reduce_only"])]
    after_last_tile = timeline["tail_us"] + timeline["drain_us"]
    return {
        "us": {"fused": round(f, 2), "sequential": round(q, 2), "gemm_only": round(g, 2), "reduce_only": round(r, 2)},
        "seq_over_fused": round(q / f, 4),
        # definition 1: against the GEMM-only MODE (which writes full partial buffers to DRAM)
        "exposed_reduce_us": round(max(0.0, f - g), 2),
        "hidden_reduce_frac": round(1.0 - max(0.0, f - g) / r, 4),
        "hidden_reduce_frac_range": [round(min(per_round_hidden), 4), round(max(per_round_hidden), 4)],
        # against the ideal overlap of Section 5.3: max(GEMM, reduction), no contention
        "ideal_overlap_us": round(max(g, r), 2),
        "exposed_vs_ideal_us": round(f - max(g, r), 2),
        # definition 2: inside the fused kernel itself - what is left after its last partial tile landed
        "fused_timeline_us": {k.replace("_us", ""): round(v, 2) for k, v in timeline.items()},
        "exposed_after_last_tile_us": round(after_last_tile, 2),
        "hidden_after_last_tile_frac": round(1.0 - after_last_tile / r, 4),
    }


def _roofline(info, avg_s, peaks, workload_name):
    t_flop = info.flops / (peaks["bf16_tflops"] * 1e12)
    t_byte = info.bytes_fused / (peaks["hbm_gbs"] * 1e9)
    bound = "hbm" if t_byte >= t_flop else "tensor"
    if bound == "hbm":
        achieved, peak, runit = info.bytes_fused / avg_s / 1e9, peaks["hbm_gbs"], "GB/s"
    else:
        achieved, peak, runit = info.flops / avg_s / 1e12, peaks["bf16_tflops"], "TFLOP/s"
    traffic, source = NCU_TRAFFIC.get(workload_name, (None, None))
    return {
        "bound": bound, "achieved": achieved, "peak": peak, "unit": runit, "frac": achieved / peak,
        "traffic": traffic,
        "traffic_source": (source + " (ncu capture of an earlier run of this kernel, not measured in this run)") if source else None,
        "peak_source": peaks["source"] + " (burst figure: each step is one kernel timed alone between L2 flushes)",
        "kernel": "t3_fused_kernel", "algorithmic_bytes": info.bytes_fused, "flops": info.flops,
        "t_roof_us": 1e6 * max(t_flop, t_byte),
        "tensor_frac_of_burst": info.flops / avg_s / 1e12 / peaks["bf16_tflops"],
        "tensor_frac_of_sustained": info.flops / avg_s / 1e12 / peaks["bf16_tflops_sustained"],
        "hbm_frac_by_algorithmic_bytes": info.bytes_fused / avg_s / 1e9 / peaks["hbm_gbs"],
    }


def _per_config(torch, np, t3, wl, spec, st, flush, peaks, rounds, per_round):
    """One entry of the per_config list: a whole configuration, default chunking, four modes interleaved."""
    name, _, out = spec.partition(":")
    w = wl.by_name(name)
    dtype = t3.BF16_OUT_F32 if out == "f32" else t3.BF16_OUT_BF16
    xb, wb = wl.make_inputs(w)
    X = torch.from_numpy(xb.view(np.int16)).cuda()
    W = torch.from_numpy(wl.w_nk(wb).view(np.int16)).cuda()
    del xb, wb
    Y = torch.zeros((w.M, w.N), dtype=torch.float32 if dtype == t3.BF16_OUT_F32 else torch.bfloat16, device="cuda")
    plan = t3.Plan(w.M, w.N, w.K, w.R, dtype, None)
    info = plan.info()
    us, tl = _interleaved(torch, t3, plan, X, W, Y, st, flush, rounds, per_round)
    plan.destroy()
    entry = {"workload": w.name, "out": out or "bf16", "M": w.M, "N": w.N, "K": w.K, "R": w.R,
             "tile": [info.tile_m, info.tile_n], "cluster_ctas": info.cluster_ctas, "ring_slots": info.ring_slots}
    entry.update(_overlap_figures(us, tl))
    fused_s = entry["us"]["fused"] * 1e-6
    roof = _roofline(info, fused_s, peaks, w.name)
    entry["fused_tflops"] = round(info.flops / fused_s / 1e12, 1)
    entry["roofline"] = {k: roof[k] for k in ("bound", "achieved", "peak", "unit", "frac", "t_roof_us", "traffic", "traffic_source")}
    del X, W, Y
    torch.cuda.empty_cache()
    return entry


def _workload(wl, args):
    """The named workload, or (profiling aid) --shape M,N,K,R with the large-FC-2 value distributions."""
    if args.shape:
        M, N, K, R = (int(v) for v in args.shape.split(","))
        return wl.Workload(f"shape_{M}x{N}x{K}_R{R}", M=M, N=N, K=K, R=R, x_dist="normal", w_dist="normal", w_std=0.01)
    return wl.by_name(args.workload)


def run_ours(args):
    import numpy as np
    import torch

    from paper_2401_16677_b200 import build as t3build
    from paper_2401_16677_b200 import t3
    from paper_2401_16677_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    if world > 1 and args.cluster_ctas == 4:
        raise SystemExit("--cluster-ctas 4 is for one process on one GPU (its W fetches are multicast TMA loads)")
    if world > 1:
        assert t3.LIB_PATH.endswith("libt3.so"), t3.LIB_PATH
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        t3build.build()
    if dist is not None:
        dist.barrier()
    t3.lib()

    w = _workload(wl, args)
    dtype = t3.BF16_OUT_F32 if args.out == "f32" else t3.BF16_OUT_BF16
    xb, wb = wl.make_inputs(w)
    wnk = wl.w_nk(wb)
    X = torch.from_numpy(xb.view(np.int16)).cuda()
    W = torch.from_numpy(wnk.view(np.int16)).cuda()
    Y = torch.zeros((w.M, w.N), dtype=torch.float32 if dtype == t3.BF16_OUT_F32 else torch.bfloat16, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    ch_kw = {}
    for k in CHUNK_ARGS:
        v = getattr(args, k)
        if v is not None:
            ch_kw[k] = v
    plan = t3.Plan(w.M, w.N, w.K, w.R, dtype, t3.chunking(**ch_kw) if ch_kw else None)
    tuned = None
    if args.tune:
        res = plan.tune(X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)
        tuned = {"tried": res.n_tried, "chosen": res.candidates()[res.chosen]}
    info = plan.info()
    peaks = _peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    if args.only is not None:
        mode = {"fused": t3.MODE_FUSED, "sequential": t3.MODE_SEQUENTIAL, "gemm_only": t3.MODE_GEMM_ONLY,
                "reduce_only": t3.MODE_REDUCE_ONLY}[args.only]
        if mode == t3.MODE_REDUCE_ONLY:   # needs valid partials
            plan.gemm_rs_mode(t3.MODE_GEMM_ONLY, X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)
        ms = _time_mode(torch, plan, mode, X, W, Y, st, args.steps, args.warmup, flush)
        print(json.dumps({"only": args.only, "workload": w.name, "us": [round(1e3 * m, 2) for m in ms]}), flush=True)
        plan.destroy()
        return 0

    sampler = ClockSampler(local_rank)
    # ---- headline: fused path, inputs resident in HBM, L2 flushed between steps
    barrier()
    sampler.start()
    ms_fused = _time_mode(torch, plan, plan.info().mode, X, W, Y, st, args.steps, args.warmup, flush)
    sampler.stop()
    barrier()
    clocks = sampler.summary()
    # companions on the same plan (same tile shape and schedule), interleaved round-robin
    us_modes, timeline = _interleaved(torch, t3, plan, X, W, Y, st, flush, args.rounds, args.per_round)
    ms_fused_warm = _time_mode(torch, plan, t3.MODE_FUSED, X, W, Y, st, max(3, min(args.steps, 20)), 3, None)

    total_ms = float(sum(ms_fused))
    total_ms_max = _max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms_max / args.steps
    value = _whole_job_value(world, info.flops, ms_per_step)

    # ---- end to end through the host-pointer C-ABI call: H2D of X and W, the op, D2H of Y
    Xh = torch.from_numpy(xb.view(np.int16)).pin_memory()
    Wh = torch.from_numpy(wnk.view(np.int16)).pin_memory()
    Yh = torch.empty((w.M, w.N), dtype=Y.dtype).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    plan.gemm_rs(X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)       # the device-resident result to compare with
    for _ in range(2):
        plan.gemm_rs_host(Xh.data_ptr(), Wh.data_ptr(), Yh.data_ptr(), st)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        plan.gemm_rs_host(Xh.data_ptr(), Wh.data_ptr(), Yh.data_ptr(), st)
    e1.record()
    barrier()
    assert plan.status().code == 0
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms_step = _max_over_ranks(e2e_ms, dist, "cuda") / e2e_steps
    e2e_value = _whole_job_value(world, info.flops, e2e_ms_step)
    # the device result must be the one the host got back
    ity = torch.int16 if Y.dtype == torch.bfloat16 else torch.int32
    assert torch.equal(Yh.view(ity).cuda(), Y.view(ity)), "e2e output differs"
    sy = 4 if dtype == t3.BF16_OUT_F32 else 2
    plan.destroy()
    del Xh, Wh, Yh, X, W, Y
    torch.cuda.empty_cache()

    per_config = None
    if world == 1 and not args.no_per_config:
        per_config = [_per_config(torch, np, t3, wl, spec, st, flush, peaks, args.rounds, args.per_round) for spec in PER_CONFIG]

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    med = statistics.median
    avg_s = (total_ms / args.steps) * 1e-3
    roofline = _roofline(info, avg_s, peaks, w.name)
    overlap = _overlap_figures(us_modes, timeline)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = _cpu_oracle_sample(w, xb, wb, budget_s=args.cpu_seconds)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": w.name, "M": w.M, "N": w.N, "K": w.K, "R": w.R, "out": args.out,
            "parallelism": "replicas only" if world > 1 else "single GPU, R K-slices",
            "l2": f"flushed before every timed step ({L2_FLUSH_BYTES >> 20} MiB write)",
            "tile": [info.tile_m, info.tile_n], "group_tiles": info.group_tiles, "grid": info.grid,
            "gemm_ctas": info.gemm_ctas, "reducer_ctas": info.reducer_ctas, "reducer_warps": info.reducer_warps,
            "stages": info.stages, "ring_slots": info.ring_slots, "cluster_ctas": info.cluster_ctas,
            "reduce_rows": info.reduce_rows, "partials": "bf16" if info.partial_dtype == t3.PARTIAL_BF16 else "f32",
            "reduce": "in place" if info.reduce == t3.REDUCE_INPLACE else "ring order", "mode": MODE_NAMES[info.mode],
            "companions": f"four modes interleaved, {args.rounds} rounds x {args.per_round} flushed calls each",
        },
        "us_per_sublayer": dict(overlap["us"], fused_headline=1e3 * med(ms_fused), fused_min=1e3 * min(ms_fused),
                                fused_l2_warm=1e3 * med(ms_fused_warm)),
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 2 * w.M * w.K + 2 * w.K * w.N,
                "d2h_bytes_per_step": sy * w.M * w.N, "ms_per_step": e2e_ms_step,
                "api": "t3_gemm_rs_host (pinned host buffers)"},
        "gpu_launches": args.steps,
        "clocks": clocks,
    }
    for k in ("seq_over_fused", "exposed_reduce_us", "hidden_reduce_frac", "hidden_reduce_frac_range", "ideal_overlap_us",
              "exposed_vs_ideal_us", "fused_timeline_us", "exposed_after_last_tile_us", "hidden_after_last_tile_frac"):
        line[k] = overlap[k]
    if tuned is not None:
        line["tuned"] = tuned
    if per_config is not None:
        line["per_config"] = per_config
    if cpu is not None:
        line["cpu_baseline"] = cpu
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()
    return 0


def run_sweep(args):
    """--sweep: configuration 5 (R x M x H grid, K = 4H) plus C1..C4: per point fused, sequential,
    GEMM-only and reduce-only microseconds, TFLOP/s, roofline fractions and the hidden-reduction
    fraction, one JSON line each (also checks fused == sequential bit for bit at every point).
    With --tune the "fused" column is t3_gemm_rs after t3_plan_tune, whatever mode that chose."""
    import numpy as np
    import torch

    from paper_2401_16677_b200 import build as t3build
    from paper_2401_16677_b200 import t3
    from paper_2401_16677_b200 import workloads as wl

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(0)
    t3build.build()
    peaks = _peaks()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    points = list(wl.CONFIGS.values()) + wl.sweep_points()
    if args.sweep_filter:
        points = [w for w in points if args.sweep_filter in w.name]
    med = statistics.median
    for w in points:
        xb, wb = wl.make_inputs(w)
        X = torch.from_numpy(xb.view(np.int16)).cuda()
        W = torch.from_numpy(wl.w_nk(wb).view(np.int16)).cuda()
        del xb, wb
        Y = torch.zeros((w.M, w.N), dtype=torch.bfloat16, device="cuda")
        Y2 = torch.zeros_like(Y)
        ch_kw = {k: getattr(args, k) for k in CHUNK_ARGS if getattr(args, k, None) is not None}
        try:
            plan = t3.Plan(w.M, w.N, w.K, w.R, t3.BF16_OUT_BF16, t3.chunking(**ch_kw) if ch_kw else None)
        except t3.T3Error as e:      # an override that this shape does not admit
            print(json.dumps({"workload": w.name, "skipped": str(e)}), flush=True)
            continue
        chosen = None
        if args.tune:
            res = plan.tune(X.data_ptr(), W.data_ptr(), Y.data_ptr(), st)
            chosen = res.candidates()[res.chosen]
        info = plan.info()
        n = max(3, args.sweep_steps)
        us = {}
        for name, mode, out in (("fused", info.mode, Y), ("sequential", t3.MODE_SEQUENTIAL, Y2),
                                ("gemm_only", t3.MODE_GEMM_ONLY, Y2), ("reduce_only", t3.MODE_REDUCE_ONLY, Y2)):
            us[name] = 1e3 * med(_time_mode(torch, plan, mode, X, W, out, st, n, 3, flush))
        same = bool(torch.equal(Y.view(torch.int16), Y2.view(torch.int16)))
        plan.destroy()
        t_flop = info.flops / (peaks["bf16_tflops"] * 1e12)
        t_byte = info.bytes_fused / (peaks["hbm_gbs"] * 1e9)
        t_flop_nom, t_byte_nom = info.flops / 2.25e15, info.bytes_fused / 8.0e12
        exposed = max(0.0, us["fused"] - us["gemm_only"])
        line = {
            "workload": w.name, "M": w.M, "N": w.N, "K": w.K, "R": w.R,
            "us": {k: round(v, 1) for k, v in us.items()},
            "fused_tflops": round(info.flops / us["fused"] / 1e6, 1),
            "bound": "hbm" if t_byte >= t_flop else "tensor",
            "t_roof_us_measured": round(1e6 * max(t_flop, t_byte), 1),
            "roofline_frac_measured": round(1e6 * max(t_flop, t_byte) / us["fused"], 3),
            "roofline_frac_nominal": round(1e6 * max(t_flop_nom, t_byte_nom) / us["fused"], 3),
            "fused_vs_sequential": round(us["sequential"] / us["fused"], 3),
            "hidden_reduce_frac": round(1.0 - exposed / us["reduce_only"], 3),
            "fused_equals_sequential_bitwise": same,
            "tile": [info.tile_m, info.tile_n], "ring_slots": info.ring_slots, "group_tiles": info.group_tiles,
            "cluster_ctas": info.cluster_ctas, "reduce_rows": info.reduce_rows,
            "partials": "bf16" if info.partial_dtype == t3.PARTIAL_BF16 else "f32",
            "reduce": "in place" if info.reduce == t3.REDUCE_INPLACE else "ring order",
            "workspace_MB": round(info.workspace_bytes / 1e6, 1),
        }
        if chosen is not None:
            line["tuned"] = chosen
        print(json.dumps(line), flush=True)
        del X, W, Y, Y2
        torch.cuda.empty_cache()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--shape", default="", help="profiling aid: M,N,K,R instead of a named workload (e.g. a configuration "
                    "scaled down in M for an ncu capture)")
    ap.add_argument("--out", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", default=None, choices=["fused", "sequential", "gemm_only", "reduce_only"],
                    help="profiling aid: launch just this mode (warmup + steps calls), print a short line, exit")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--sweep", action="store_true", help="configuration 5: one JSON line per shape, then exit")
    ap.add_argument("--sweep-steps", type=int, default=10)
    ap.add_argument("--sweep-filter", default="")
    ap.add_argument("--rounds", type=int, default=5, help="interleaved companion timing: rounds")
    ap.add_argument("--per-round", type=int, default=10, help="interleaved companion timing: flushed calls per mode and round")
    ap.add_argument("--no-per-config", action="store_true", help="skip the per_config block (the other configurations)")
    ap.add_argument("--tune", action="store_true", help="let t3_plan_tune choose the configuration before timing")
    for k in CHUNK_ARGS:
        ap.add_argument("--" + k.replace("_", "-"), dest=k, type=int, default=None)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    if args.sweep:
        return run_sweep(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
