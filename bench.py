#!/usr/bin/env python
"""Benchmark of the structure-adaptive SpMM path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--configs 1,2,3,4] [--impl reference]

One *step* is one pass of the whole hot path: one sd_spmm call on each benchmark workload
(stencil N=64 -> family (a), GCN R-MAT N=128 and skewed N=32 -> family (b), block16 N=256 in
fp32 and bf16 -> family (c)), inputs resident in HBM, L2 flushed before every call.  The JSON
line's `value` is sum(2*nnz*N) / sum(device time) over the step; `per_config` carries each
workload's own GFLOP/s, effective GB/s on the compulsory-traffic model and fraction of the
measured HBM peak.  `e2e` runs the same step through sd_spmm_host_async / sd_plan_sync with pinned host buffers
(B copied in, C copied out, every call).  `--impl reference` times the CPU oracle instead.

With N > 1 ranks (torchrun), every rank runs the step on its own dense operands (independent
problems, no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
METRIC = "SpMM GFLOP/s (2*nnz*N) and effective HBM GB/s as % of B200 peak, 1 GPU"

# (label, config index, dtype): the five benchmark configurations (the block config in both value types)
BENCH_SET = [("tiny_f32", 0, W.SD_F32), ("stencil_f32", 1, W.SD_F32), ("gcn_rmat_f32", 2, W.SD_F32),
             ("block16_f32", 3, W.SD_F32), ("block16_bf16", 3, W.SD_BF16), ("skewed_f32", 4, W.SD_F32)]
# The block configuration's text has a second reading ("about 8.4K blocks, about 2.1M nnz" instead of 0.2 % of the
# block positions): timed as labelled context rows of their own, outside the step.
CONTEXT_SET = [("block16_f32_reading_8389_blocks", 3, W.SD_F32, dict(nblocks=8389)),
               ("block16_bf16_reading_8389_blocks", 3, W.SD_BF16, dict(nblocks=8389))]
HBM_BAR = 0.60   # the target of the memory-bound configurations, as a fraction of the HBM peak on the compulsory model


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def ncu_traffic():
    """Per-launch DRAM bytes of the kernels, as captured with ncu (profiles/traffic.json)."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(p):
        try:
            return json.load(open(p))
        except Exception:
            pass
    return {}


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) during the timed region."""

    def __init__(self, index: int, period: float = 0.002):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _once(self):
        nv = self.nv
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
            try:
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
            except Exception:
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                     0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}
            for bit, name in names.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def start(self):
        if self.nv is None:
            return
        def loop():
            while not self._stop.is_set():
                self._once()
                time.sleep(self.period)
        self._thread = threading.Thread(target=loop, daemon=True)
        self._thread.start()

    def stop(self) -> dict:
        if self._thread:
            self._stop.set()
            self._thread.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- multi-rank plumbing
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(x: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(w: W.Workload, budget_flops: float, seed: int):
    """Rows of a seeded random order until their 2*nnz*N reaches the budget."""
    rng = np.random.Generator(np.random.PCG64(seed))
    order = rng.permutation(w.M)
    per_row = 2.0 * np.diff(w.rowptr)[order] * w.N
    n = int(np.searchsorted(np.cumsum(per_row), budget_flops)) + 1
    rows = np.sort(order[:min(n, w.M)]).astype(np.int64)
    flops = float(2.0 * np.diff(w.rowptr)[rows].sum() * w.N)
    return rows, flops


def time_oracle(sets, budget_flops: float):
    """One pass of the oracle (the plain double-precision loop, without the abs-sum companion that only
    the tolerance check needs) over the row samples.  Returns (seconds, flops)."""
    import oracle
    total_t, total_f = 0.0, 0.0
    for w, rows, flops in sets:
        t0 = time.perf_counter()
        oracle.spmm_rows(rows, w.rowptr, w.colind, w.vals, w.B, w.N, w.C0, w.alpha, w.beta, want_abs=False)
        total_t += time.perf_counter() - t0
        total_f += flops
    return total_t, total_f


def run_reference(args, rank, world):
    """--impl reference: the CPU oracle on a bounded row sample of the same workloads."""
    if rank != 0:
        return
    import oracle
    ws = [make_workload(args, ci, dt) for _, ci, dt in select_set(args)]
    budget = 2.0e8   # flops per workload per step: about a second of host work per step in total
    sets = []
    for i, w in enumerate(ws):
        rows, flops = oracle_sample(w, budget, 1234 + i)
        sets.append((w, rows, flops))
    for _ in range(args.warmup):
        time_oracle(sets, budget)
    ts, fl = [], 0.0
    for _ in range(args.steps):
        t, fl = time_oracle(sets, budget)
        ts.append(t)
    sec = float(np.mean(ts))
    value = fl / sec / 1e9
    sample = "seeded random rows, ~2e8 flops per workload per step: " + ", ".join(
        f"{lab}:{len(r)} rows" for (lab, _, _), (_, r, _) in zip(select_set(args), sets))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args)},
        "cpu_baseline": {"value": value, "unit": "GFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU leg
SMALL_KW = {0: dict(), 1: dict(n=768), 2: dict(scale=18), 3: dict(Mb=2048, Kb=2048),
            4: dict(M=1 << 20, scale_c=2.4e7 / 4, cap=50000)}


def make_workload(args, ci, dt, extra=None):
    kw = dict(SMALL_KW[ci]) if args.small else {}
    if args.width:
        kw["N"] = args.width
    if extra and not args.small:
        kw.update(extra)
    return W.config(ci, dtype=dt, **kw)


def select_set(args):
    if not args.configs:
        return BENCH_SET
    want = {int(x) for x in args.configs.split(",")}
    return [b for b in BENCH_SET if b[1] in want]


def workload_name(args):
    return "suite: " + " | ".join(lab for lab, _, _ in select_set(args)) + \
        " (tiny uniform 2048^2 Poisson(8) rows N=32; stencil 1024^2 grid N=64 beta=0.5; R-MAT scale 20 GCN N=128; " \
        "16x16 dense blocks 0.2% of 4096^2 positions N=256 in fp32 and bf16; rank-size Zipf(1.2) rows cap 200000 N=32)"


def run_gpu(args, rank, local_rank, world):
    import torch
    import paper_2608_05033_b200 as sd

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    sd.load()
    peak, peak_kind = measured_peak()

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).to(dev)

    cases = []
    t_gen0 = time.time()
    selected = [(lab, ci, dt, None, True) for lab, ci, dt in select_set(args)]
    if not args.configs or "3" in args.configs.split(","):
        selected += [(lab, ci, dt, kw, False) for lab, ci, dt, kw in CONTEXT_SET]
    for lab, ci, dt, extra, in_step in selected:
        w = make_workload(args, ci, dt, extra)
        if rank > 0:   # independent problems: every rank draws its own dense operands
            rng = np.random.Generator(np.random.PCG64(W.SEED_BASE + 100 * rank + ci))
            Bf = rng.standard_normal(size=(w.K, w.N), dtype=np.float32)
            w.B = Bf if dt == W.SD_F32 else W.f32_to_bf16_bits(Bf).reshape(w.K, w.N)
        rowptr, colind, vals = to_dev(w.rowptr), to_dev(w.colind), to_dev(w.vals)
        t0 = time.time()
        plan = sd.Plan(rowptr, colind, vals, w.M, w.K, w.N, dtype=w.dtype, windows=args.windows)
        torch.cuda.synchronize()
        plan_ms = (time.time() - t0) * 1e3
        Bd = to_dev(w.B)
        Cd = to_dev(w.C0) if w.C0 is not None else torch.zeros((w.M, w.N), dtype=torch.float32, device=dev)
        cases.append({"label": lab, "w": w, "plan": plan, "B": Bd, "C": Cd, "plan_ms": plan_ms,
                      "info": plan.info(), "times": [], "in_step": in_step})
    gen_s = time.time() - t_gen0
    context_cases = [c for c in cases if not c["in_step"]]
    cases = [c for c in cases if c["in_step"]]

    flush = torch.empty(512 * 1024 * 1024 // 4, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def one_step(record: bool):
        evs = []
        for c in cases:
            flush.fill_(1.0)                         # L2 flush, outside the timed interval
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            c["plan"].spmm(c["B"], c["C"], c["w"].alpha, c["w"].beta, stream)
            e1.record(stream)
            evs.append((c, e0, e1))
        torch.cuda.synchronize()
        tot = 0.0
        for c, e0, e1 in evs:
            ms = e0.elapsed_time(e1)
            tot += ms
            if record:
                c["times"].append(ms)
        return tot

    for _ in range(max(args.warmup, 3)):
        one_step(False)
    barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    wall0 = time.perf_counter()
    step_ms = [one_step(True) for _ in range(args.steps)]
    torch.cuda.synchronize()
    barrier()
    wall_ms = (time.perf_counter() - wall0) * 1e3 / args.steps
    clocks = sampler.stop()

    # ---- beside the cold numbers: warm L2 (back to back, no flush) and the paper's protocol (5 warm-up calls,
    # then 10 timed back to back, arithmetic mean; plan creation excluded) for every workload ---------------
    def back_to_back(c, warm, reps):
        for _ in range(warm):
            c["plan"].spmm(c["B"], c["C"], c["w"].alpha, c["w"].beta, stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            c["plan"].spmm(c["B"], c["C"], c["w"].alpha, c["w"].beta, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    for c in cases + context_cases:
        c["ms_paper_protocol"] = back_to_back(c, 5, 10)
        c["ms_warm"] = back_to_back(c, 3, 50)
    for c in context_cases:   # the labelled second reading of the block configuration: cold, outside the step
        for i in range(13):
            flush.fill_(1.0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            c["plan"].spmm(c["B"], c["C"], c["w"].alpha, c["w"].beta, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                c["times"].append(e0.elapsed_time(e1))
    # the tiny configuration is bound by launch latency: 100 calls replayed as one CUDA graph show the floor
    for c in cases:
        if c["label"] != "tiny_f32" or rank != 0:
            continue
        try:
            graph = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                c["plan"].spmm(c["B"], c["C"], c["w"].alpha, c["w"].beta, side)
                with torch.cuda.graph(graph, stream=side):
                    for _ in range(100):
                        c["plan"].spmm(c["B"], c["C"], c["w"].alpha, c["w"].beta, side)
            torch.cuda.synchronize()
            graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(5):
                graph.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            c["us_per_call_in_graph_of_100"] = e0.elapsed_time(e1) * 1e3 / 500
        except Exception as exc:   # an extra figure: never fails the bench
            c["graph_error"] = str(exc)[:160]

    local_ms = float(np.mean(step_ms))
    ms_per_step = max_over_ranks(local_ms, dev)
    flops_local = float(sum(c["w"].flops() for c in cases))
    bytes_local = float(sum(c["w"].compulsory_bytes() for c in cases))
    flops_all = sum_over_ranks(flops_local, dev)
    bytes_all = sum_over_ranks(bytes_local, dev)
    value = flops_all / (ms_per_step * 1e-3) / 1e9

    # ---- end to end: host buffers through sd_spmm_host, copies inside the timed region --------
    e2e_steps = 0 if args.no_e2e else max(10, min(args.steps, 20))
    h2d = d2h = 0
    hosts = []
    for c in ([] if args.no_e2e else cases):
        w = c["w"]
        Bh = torch.from_numpy(w.B.view(np.int16) if w.B.dtype == np.uint16 else w.B).pin_memory()
        Ch = (torch.from_numpy(w.C0.copy()) if w.C0 is not None else torch.zeros((w.M, w.N))).pin_memory()
        hosts.append((Bh, Ch))
        h2d += Bh.numel() * Bh.element_size() + (Ch.numel() * 4 if w.beta != 0.0 else 0)
        d2h += Ch.numel() * 4

    def e2e_step():
        # every call queues its copies and kernels on its plan's own stream: one workload's result
        # travels to the host while the next one's operand travels to the device
        # (largest result first, so that the copy-out left over at the end of the step is the smallest)
        for c, (Bh, Ch) in sorted(zip(cases, hosts), key=lambda t: -t[1][1].numel()):
            c["plan"].spmm_host_async(Bh, Ch, c["w"].alpha, c["w"].beta)
        for c in cases:
            c["plan"].sync()

    if e2e_steps:
        e2e_step()
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_local = (time.perf_counter() - t0) * 1e3 / max(e2e_steps, 1) if e2e_steps else float("inf")
    e2e_ms = max_over_ranks(e2e_local, dev)
    e2e_value = flops_all / (e2e_ms * 1e-3) / 1e9

    # ---- gather ceiling: the workload's own index stream as bare row gathers ------------------------
    if args.probe and rank == 0:
        import bench_probes
        bench_probes.build()
        sink = torch.zeros(bench_probes.sink_floats(), dtype=torch.float32, device=dev)
        for c in cases:
            w = c["w"]
            row_bytes = w.N * (4 if w.dtype == W.SD_F32 else 2)
            if row_bytes not in (16, 32, 64, 128, 256, 512):
                continue
            colind = to_dev(w.colind)
            ts = []
            for i in range(8):
                flush.fill_(1.0)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                bench_probes.gather(0, colind, w.nnz, c["B"], row_bytes, sink, stream=stream)
                e1.record(stream)
                torch.cuda.synchronize()
                if i >= 3:
                    ts.append(e0.elapsed_time(e1))
            c["probe_ms"] = float(np.mean(ts))
            del colind

    # ---- context only: cuSPARSE CSR SpMM (what the paper compares against), fp32 workloads ------
    if args.cusparse and rank == 0:
        for c in cases:
            w = c["w"]
            if w.dtype != W.SD_F32:
                continue
            try:
                A = torch.sparse_csr_tensor(to_dev(w.rowptr).long(), to_dev(w.colind).long(), to_dev(w.vals),
                                            size=(w.M, w.K))
                ts = []
                for i in range(8):
                    flush.fill_(1.0)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    out = torch.sparse.mm(A, c["B"])   # alpha = 1, beta = 0 product only
                    e1.record(stream)
                    torch.cuda.synchronize()
                    if i >= 3:
                        ts.append(e0.elapsed_time(e1))
                    del out
                c["cusparse_ms"] = float(np.mean(ts))
                del A
            except Exception as exc:   # context only: never fails the bench
                c["cusparse_ms"] = None
                c["cusparse_error"] = str(exc)[:120]

    if rank != 0:
        return

    # ---- per-config table, roofline of the dominant kernel ------------------------------------------
    traffic = ncu_traffic()
    per = []
    for c in cases + context_cases:
        w, info = c["w"], c["info"]
        ms = float(np.mean(c["times"]))
        gbs = w.compulsory_bytes() / (ms * 1e-3) / 1e9
        per.append({"workload": c["label"], "in_step": c["in_step"], "family": sd.FAMILY_NAMES[info.family], "M": w.M, "N": w.N,
                    "nnz": w.nnz, "ms": ms, "ms_cold": ms, "ms_min": float(np.min(c["times"])),
                    "ms_warm": c.get("ms_warm"), "ms_paper_protocol": c.get("ms_paper_protocol"),
                    "gflops": w.flops() / (ms * 1e-3) / 1e9, "compulsory_bytes": w.compulsory_bytes(),
                    "effective_gbs": gbs, "frac_of_measured_hbm": gbs / peak,
                    "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBS, "launches": int(info.launches), "windows": int(info.windows),
                    "plan_ms": c["plan_ms"], "plan_bytes": int(info.plan_bytes)})
        if c["label"] == "tiny_f32":
            per[-1]["bound"] = "launch latency (no roofline applies)"
            per[-1]["us_per_call_cold"] = ms * 1e3
            for k in ("us_per_call_in_graph_of_100", "graph_error"):
                if k in c:
                    per[-1][k] = c[k]
        elif info.family == sd.SD_BSR_TC:
            per[-1]["bound"] = "hbm behind the tensor pipe (tensor-pipe utilisation: profiles/bsr_block16_small.md)"
        else:
            per[-1]["bound"] = "hbm"
            per[-1]["meets_60pct_of_measured_hbm"] = bool(gbs / peak >= HBM_BAR)
        if "probe_ms" in c:
            per[-1]["gather_probe_ms"] = c["probe_ms"]
            per[-1]["gather_probe_tbs"] = w.nnz * w.N * (4 if w.dtype == W.SD_F32 else 2) / (c["probe_ms"] * 1e-3) / 1e12
            per[-1]["spmm_over_gather_probe"] = ms / c["probe_ms"]
        if "cusparse_ms" in c:
            per[-1]["context_cusparse_ms"] = c["cusparse_ms"]
            if c["cusparse_ms"]:
                per[-1]["context_speedup_over_cusparse"] = c["cusparse_ms"] / ms
    dom = max((p for p in per if p["in_step"]), key=lambda p: p["ms"])
    bar = {"target_frac_of_measured_hbm": HBM_BAR,
           "met": [p["workload"] for p in per if p.get("meets_60pct_of_measured_hbm") is True],
           "missed": [p["workload"] for p in per if p.get("meets_60pct_of_measured_hbm") is False],
           "note": "the merge-family workloads gather a row of B per nonzero and run at the rate L2 feeds the SMs "
                   "(profiles/gather_paths_gcn_rmat.md), not at the HBM rate: the bar is not met there"}
    roofline = {"bound": "hbm", "kernel": dom["family"] + " on " + dom["workload"],
                "achieved": dom["effective_gbs"], "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": dom["effective_gbs"] / peak,
                "traffic": traffic.get(dom["workload"], {}).get("dram_bytes_per_launch"),
                "note": "achieved = compulsory-model bytes of the call / its CUDA-event time"}

    # ---- CPU baseline: the oracle on a bounded sample, this machine's host cores --------------------------
    import oracle
    sets = []
    for i, c in enumerate([] if args.no_e2e else cases):
        rows, fl = oracle_sample(c["w"], 1.0e10, 1234 + i)
        sets.append((c["w"], rows, fl))
    tsec, fl = time_oracle(sets, 1.0e10)
    tsec2, _ = time_oracle(sets, 1.0e10)
    tsec = max(min(tsec, tsec2), 1e-9)
    cpu = {"value": fl / tsec / 1e9, "unit": "GFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
           "sample": "seeded random rows up to 1e10 flops per workload (here: every row): " + ", ".join(
               f"{c['label']}:{len(r)} rows" for c, (_, r, _) in zip(cases, sets)), "seconds": tsec}

    line = {
        "metric": METRIC, "value": value, "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(args),
                   "l2": "512 MB flush write before every call (outside the timed events); every workload "
                         "but tiny and block16 also exceeds the 126 MB L2; per_config adds ms_warm (back to back) and "
                         "ms_paper_protocol (5 warm-up + 10 timed calls back to back, arithmetic mean)",
                   "timing": "CUDA events on the launching stream around each sd_spmm call, summed per step"},
        "effective_gbs": bytes_all / (ms_per_step * 1e-3) / 1e9,
        "frac_of_measured_hbm": bytes_all / (ms_per_step * 1e-3) / 1e9 / (peak * world),
        "wall_ms_per_step_incl_flush": wall_ms,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "GFLOP/s", "ms_per_step": e2e_ms, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "steps": e2e_steps},
        "gpu_launches": int(sum(p["launches"] for p in per if p["in_step"]) * args.steps),
        "hbm_bar": bar,
        "roofline": roofline,
        "cpu_baseline": cpu,
        "per_config": per,
        "setup_seconds": gen_s,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- GCN epoch mode
def run_gcn_epoch(args, local_rank):
    """Sparse aggregations of a two-layer full-batch GCN (paper, Sec. 5 "End-to-End Application
    Evaluation"): four products with the normalised adjacency per epoch, two forward (features,
    hidden activations) and two backward (their gradients); the adjacency is symmetric, so the
    backward products reuse the forward plan.  One plan per dense width, made once; the dense
    layers and activations of the training loop are not this library's work and are not run.
    Prints one JSON line of its own (not the benchmark line)."""
    import torch
    import paper_2608_05033_b200 as sd

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    sd.load()
    stream = torch.cuda.current_stream()
    kw = dict(SMALL_KW[2]) if args.small else {}
    base = W.config(2, dtype=W.SD_F32, N=8, **kw)
    rowptr = torch.from_numpy(base.rowptr).to(dev)
    colind = torch.from_numpy(base.colind).to(dev)
    vals = torch.from_numpy(base.vals).to(dev)
    warm, epochs = max(args.warmup, 3), args.steps
    rows = []
    sampler = ClockSampler(local_rank)
    sampler.start()
    for width in (8, 32, 128, 256):
        t0 = time.time()
        plan = sd.Plan(rowptr, colind, vals, base.M, base.K, width, dtype=W.SD_F32)
        torch.cuda.synchronize()
        plan_ms = (time.time() - t0) * 1e3
        gen = torch.Generator(device=dev)
        gen.manual_seed(W.SEED_BASE + width)
        # features, hidden activations and the two gradients: four different operands per epoch
        ops = [torch.randn((base.K, width), dtype=torch.float32, device=dev, generator=gen) for _ in range(4)]
        outs = [torch.empty((base.M, width), dtype=torch.float32, device=dev) for _ in range(2)]

        def epoch():
            for i, X in enumerate(ops):
                plan.spmm(X, outs[i & 1], 1.0, 0.0, stream)

        for _ in range(warm):
            epoch()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(epochs):
            epoch()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / epochs
        info = plan.info()
        row = {"width": width, "aggregation_ms_per_epoch": ms, "ms_per_product": ms / 4,
               "gflops": 4 * 2.0 * base.nnz * width / (ms * 1e-3) / 1e9, "family": sd.FAMILY_NAMES[info.family],
               "launches_per_product": int(info.launches), "plan_ms": plan_ms,
               "operand_mb": base.K * width * 4 / 1e6}
        if args.cusparse:
            try:
                A = torch.sparse_csr_tensor(rowptr.long(), colind.long(), vals, size=(base.M, base.K))
                for _ in range(3):
                    for X in ops:
                        torch.sparse.mm(A, X)
                torch.cuda.synchronize()
                n_ctx = max(3, epochs // 10)
                e0.record(stream)
                for _ in range(n_ctx):
                    for X in ops:
                        torch.sparse.mm(A, X)
                e1.record(stream)
                torch.cuda.synchronize()
                row["context_cusparse_ms_per_epoch"] = e0.elapsed_time(e1) / n_ctx
                row["context_speedup_over_cusparse"] = row["context_cusparse_ms_per_epoch"] / ms
                del A
            except Exception as exc:   # context only
                row["context_cusparse_error"] = str(exc)[:120]
        rows.append(row)
        plan.close()
        del ops, outs
    clocks = sampler.stop()
    print(json.dumps({
        "mode": "gcn-epoch", "metric": "gcn_sparse_aggregation_ms_per_epoch", "unit": "ms", "higher_is_better": False,
        "n_gpus": 1, "epochs": epochs, "warmup_epochs": warm, "data": "synthetic", "dtype": "f32",
        "config": {"workload": f"{base.name}: symmetrised R-MAT + I, D^-1/2 (A+I) D^-1/2, M = {base.M}, nnz = {base.nnz}; "
                               "four products per epoch on four different dense operands, one plan per width reused "
                               "for the forward and the backward products (symmetric adjacency)",
                   "l2": "no flush inside an epoch; the four operands and two results of a width together exceed the "
                         "126 MB L2 from width 8 on (6 x 33.5 MB at width 8)"},
        "clocks": clocks, "per_width": rows}))


# --------------------------------------------------------------------------- the decision rules against the clock
def regret_rows(level: str, device_index: int = 0, log=None):
    """The plan's fixed rules (family by block fill, class split by dense width, column windows) against measured
    times (the paper ranks plans by measured runtime, Sec. 3.2-3.3; it prints no thresholds, so the clock on this
    GPU is what the constants can be held to).  For every point each alternative is forced and timed (cold L2,
    median), then the automatic plan; regret = automatic / fastest - 1.  `level`: "full" = the sweep behind the
    committed table, "test" = a subset that a GPU test can afford."""
    import torch
    import paper_2608_05033_b200 as sd

    dev = torch.device("cuda", device_index)
    torch.cuda.set_device(dev)
    sd.load()
    flush = torch.empty(512 * 1024 * 1024 // 4, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).to(dev)

    def median_ms(plan, Bd, Cd, w, reps):
        ts = []
        for i in range(reps + 3):
            flush.fill_(1.0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            plan.spmm(Bd, Cd, w.alpha, w.beta, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    def point(rule, w, label, alternatives, reps):
        """alternatives: {name: plan options}; the automatic plan is timed last."""
        rowptr, colind, vals, Bd = to_dev(w.rowptr), to_dev(w.colind), to_dev(w.vals), to_dev(w.B)
        Cd = torch.zeros((w.M, w.N), dtype=torch.float32, device=dev)
        times = {}
        for name, opts in alternatives.items():
            plan = sd.Plan(rowptr, colind, vals, w.M, w.K, w.N, dtype=w.dtype, **opts)
            times[name] = median_ms(plan, Bd, Cd, w, reps)
            plan.close()
        plan = sd.Plan(rowptr, colind, vals, w.M, w.K, w.N, dtype=w.dtype)
        info = plan.info()
        auto_ms = median_ms(plan, Bd, Cd, w, reps)
        plan.close()
        best = min(times.values())
        row = {"rule": rule, "point": label, "dtype": "bf16" if w.dtype == W.SD_BF16 else "f32", "N": w.N, "nnz": w.nnz,
               "ms": {k: round(v, 4) for k, v in times.items()}, "automatic_ms": round(auto_ms, 4),
               "automatic": {"family": sd.FAMILY_NAMES[info.family], "windows": int(info.windows),
                             "class_split": int(info.class_split)},
               "regret": auto_ms / best - 1.0}
        if log:
            log(row)
        return row

    full = level == "full"
    reps = 9 if full else 5
    rows = []
    # (A) 16x16 blocks on the tensor cores or CSR kernels: block fill x dense width x value type
    fills = (1.0, 0.8, 0.5, 0.35, 0.2, 0.13) if full else (1.0, 0.5, 0.2)
    widths = (64, 128, 256) if full else (64, 256)
    for dt in (W.SD_F32, W.SD_BF16):
        for N in widths:
            base = W.g4_block(N=N, dtype=W.SD_F32)
            for fill in fills:
                w = W.thin_blocks(base, fill)
                if dt == W.SD_BF16:
                    w = W.Workload(w.name, w.M, w.K, w.N, w.rowptr, w.colind, W.f32_to_bf16_bits(w.vals),
                                   W.f32_to_bf16_bits(w.B).reshape(w.B.shape), None, w.alpha, w.beta, W.SD_BF16, dict(w.meta))
                rows.append(point("family: blocks on tensor cores vs CSR kernels", w, f"block fill {fill:g}",
                                  {"bsr_tc": dict(family=sd.SD_BSR_TC), "rowsplit": dict(family=sd.SD_ROWSPLIT),
                                   "merge": dict(family=sd.SD_MERGE)}, reps))
    # (B) skewed rows without column windows: merge-path tiles, class split or hybrid family, by dense width
    for dt in (W.SD_F32, W.SD_BF16):
        for N in ((5, 8, 16, 32, 64, 96, 128, 256) if full else (8, 32, 128)):
            w = W.config(2, dtype=dt, N=N, **({} if full else dict(scale=18)))
            rows.append(point("skewed rows, no column windows: tiles, class split or hybrid", w, "R-MAT scale %d" % (20 if full else 18),
                              {"tiles": dict(family=sd.SD_MERGE, windows=1), "class_split": dict(family=sd.SD_MERGE, windows=-1),
                               "hybrid": dict(family=sd.SD_HYBRID, windows=1)}, reps))
    # (C) column windows of the skewed workload: none, the rule's count, twice that
    w = W.config(4, **({} if full else dict(M=1 << 20, scale_c=2.4e7 / 4, cap=50000)))
    rule_w = 8 if full else 2
    rows.append(point("merge family: column windows", w, f"rank-size rows, M = {w.M}",
                      {"tiles, no windows": dict(family=sd.SD_MERGE, windows=1),
                       "class split, one window": dict(family=sd.SD_MERGE, windows=-1),
                       f"{rule_w} windows": dict(family=sd.SD_MERGE, windows=rule_w),
                       f"{2 * rule_w} windows": dict(family=sd.SD_MERGE, windows=2 * rule_w),
                       f"hybrid, {rule_w} windows": dict(family=sd.SD_HYBRID, windows=rule_w)}, reps))
    # (D) hybrid family or windowed class split, by the bytes of one row of B
    for dt, widths in ((W.SD_F32, (16, 24, 32, 48, 64) if full else (16, 32, 64)),
                       (W.SD_BF16, (32, 48, 64, 128) if full else (64,))):
        for N in widths:
            w = W.config(4, dtype=dt, N=N, **({} if full else dict(M=1 << 20, scale_c=2.4e7 / 4, cap=50000)))
            rows.append(point("hybrid family vs windowed class split", w, f"rank-size rows, M = {w.M}",
                              {"class split, windows": dict(family=sd.SD_MERGE), "hybrid": dict(family=sd.SD_HYBRID)}, reps))
    return rows


def run_regret(args, local_rank):
    rows = regret_rows("test" if args.small else "full", local_rank, log=lambda r: print(json.dumps(r), file=sys.stderr, flush=True))
    print(json.dumps({"mode": "regret", "level": "test" if args.small else "full", "worst_regret": max(r["regret"] for r in rows),
                      "rows": rows}))


def run_row_split(args, rank, local_rank, world):
    """--split rows: ONE product (the GCN workload) over all ranks.  Rank k owns a contiguous range of rows of A and
    C (balanced by rows + nonzeros) and an equal piece of the rows of B; every step gathers B into the rank's own
    memory with one NCCL all-gather and then runs the rank's plan on it (no kernel reads a peer's memory).  Total
    work is fixed: strong scaling.  At one rank the gather is a local copy."""
    import torch
    import torch.distributed as dist
    import paper_2608_05033_b200 as sd
    from paper_2608_05033_b200.shard import RowSplitSpmm, b_row_shard

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    sd.load()
    kw = dict(SMALL_KW[2]) if args.small else {}
    if args.width:
        kw["N"] = args.width
    w = W.config(2, dtype=W.SD_F32, **kw)            # every rank draws the same seeded matrix, keeps its share
    rs = RowSplitSpmm(w.rowptr, w.colind, w.vals, w.M, w.K, w.N, w.dtype, dev)
    k0, k1, per = b_row_shard(w.K, world, rank)
    piece = np.zeros((per, w.N), dtype=np.float32)
    piece[:k1 - k0] = w.B[k0:k1]
    b_local = torch.from_numpy(piece).to(dev)
    c_local = torch.zeros((rs.r1 - rs.r0, w.N), dtype=torch.float32, device=dev)
    flush = torch.empty(512 * 1024 * 1024 // 4, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        flush.fill_(1.0)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        bf = None
        from paper_2608_05033_b200.shard import gather_b
        bf = gather_b(b_local, w.K, out=rs.b_full)
        e1.record(stream)
        if rs.r1 > rs.r0:
            rs.plan.spmm(bf, c_local, w.alpha, w.beta, stream)
        e2.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e2), e0.elapsed_time(e1)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    ts = [step() for _ in range(args.steps)]
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    local_ms = float(np.mean([t[0] for t in ts]))
    gather_ms = float(np.mean([t[1] for t in ts]))
    ms = max_over_ranks(local_ms, dev)
    gms = max_over_ranks(gather_ms, dev)
    my_nnz = float(rs.plan.info().nnz)
    if rank == 0:
        print(json.dumps({
            "mode": "split-rows", "metric": METRIC, "value": w.flops() / (ms * 1e-3) / 1e9, "unit": "GFLOP/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
            "all_gather_ms": gms, "higher_is_better": True, "scaling": "strong", "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{w.name}: one product split by rows over {world} rank(s), B row-sharded and "
                                   "gathered into local memory every step (one all-gather), cold L2"},
            "rank0_rows": [rs.r0, rs.r1], "rank0_nnz": my_nnz, "b_bytes_gathered_per_rank": int(world * per * w.N * 4),
            "clocks": clocks}))
    rs.close()
    if world > 1:
        dist.destroy_process_group()


def run_probe_paths(args, local_rank):
    """Fetch paths for the gathers of the dense operand, timed on the GCN workload's own column stream
    (512-byte rows, storage order): plain loads with 4 / 8 / 16 gathers in flight per lane, L2 evict-last and
    L1 no-allocate hints, tile order with staged indices, half a warp per row, bulk copies into a shared-memory
    ring, and the hottest rows kept in the distributed shared memory of a thread-block cluster.  Every round
    times every path once (cold L2), so drifts hit all paths alike; prints one JSON line of its own."""
    import torch
    import bench_probes as bp

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    bp.build()
    kw = dict(SMALL_KW[2]) if args.small else {}
    w = W.config(2, dtype=W.SD_F32, **kw)
    assert w.N * 4 == 512
    colind = torch.from_numpy(w.colind).to(dev)
    table = torch.from_numpy(w.B).to(dev)
    sink = torch.zeros(bp.sink_floats(), dtype=torch.float32, device=dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(512 * 1024 * 1024 // 4, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    # hub rows = the most referenced columns; their indices in the stream carry bit 31 and the hub slot
    deg = np.bincount(w.colind, minlength=w.K)
    order = np.argsort(-deg, kind="stable").astype(np.int32)
    hub_streams = {}
    for path, cl in bp.HUB_CLUSTER.items():
        nh = cl * bp.HUB_ROWS_PER_CTA
        slot = np.full(w.K, -1, dtype=np.int64)
        slot[order[:nh]] = np.arange(nh)
        s = slot[w.colind]
        enc = np.where(s >= 0, s | 0x80000000, w.colind).astype(np.uint32).view(np.int32)
        hub_streams[path] = (torch.from_numpy(enc).to(dev), torch.from_numpy(order[:nh].copy()).to(dev), float((s >= 0).mean()))
    paths = sorted(bp.PATHS)
    times = {p: [] for p in paths}
    info = {}
    sampler = ClockSampler(local_rank)
    sampler.start()
    rounds = max(args.steps, 5) + 2
    for rep in range(rounds):
        for p in paths:
            idx, hub = (hub_streams[p][0], hub_streams[p][1]) if p in hub_streams else (colind, None)
            flush.fill_(1.0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            info[p] = bp.gather(p, idx, w.nnz, table, 512, sink, err=err, hubrows=hub, stream=stream)
            e1.record(stream)
            torch.cuda.synchronize()
            if rep >= 2:
                times[p].append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    rows = []
    for p in paths:
        ms = float(np.median(times[p]))
        row = {"path": p, "name": bp.PATHS[p], "ms_median": ms, "ms_min": float(np.min(times[p])),
               "gathered_tbs": w.nnz * 512 / (ms * 1e-3) / 1e12, "resident": info[p]}
        if p in hub_streams:
            row["hub_fraction_of_gathers"] = hub_streams[p][2]
        rows.append(row)
    print(json.dumps({"mode": "probe-paths", "workload": w.name, "nnz": w.nnz, "row_bytes": 512, "rounds": rounds - 2,
                      "bulk_ring_error_word": int(err.item()), "clocks": clocks, "paths": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="sd", choices=["sd", "reference"])
    ap.add_argument("--configs", default="", help="comma list of config indices (0..4) to restrict the step")
    ap.add_argument("--windows", type=int, default=0, help="column windows of the merge family (0 = plan's rule)")
    ap.add_argument("--probe", action="store_true",
                    help="also replay every workload's colind stream as bare row gathers (bench_probes, path 0) and "
                         "report its time beside the SpMM time: the gather ceiling of the memory system for that stream")
    ap.add_argument("--regret", action="store_true",
                    help="time every alternative of the plan's fixed rules (family by block fill, class split by width, "
                         "column windows) against the automatic choice; prints its own JSON line (--small: the subset "
                         "the GPU test runs)")
    ap.add_argument("--split", default="", choices=["", "rows"],
                    help="rows: one product (the GCN workload) split by rows over all ranks, B row-sharded and gathered "
                         "into local memory with one all-gather per step (strong scaling; prints its own JSON line)")
    ap.add_argument("--probe-paths", action="store_true",
                    help="time the fetch paths of bench_probes on the GCN workload's column stream (prints its own JSON line)")
    ap.add_argument("--width", type=int, default=0,
                    help="override the dense width N of every selected workload (width sweep: 1 = SpMV, 8, 32, "
                         "128, 256); not the benchmark configuration")
    ap.add_argument("--cusparse", action="store_true",
                    help="also time cuSPARSE CSR SpMM through torch.sparse.mm on the fp32 workloads, as context "
                         "only (the paper's comparison baseline; the library never calls it)")
    ap.add_argument("--small", action="store_true",
                    help="reduced sizes of the same workloads (dense operands still above the L2 size where "
                         "the full-size ones are); for profiler captures, not a bench number")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer and CPU-baseline legs")
    ap.add_argument("--gcn-epoch", action="store_true",
                    help="time the four sparse aggregations of a two-layer GCN epoch on the R-MAT adjacency at dense "
                         "widths 8, 32, 128, 256 (--steps epochs after --warmup epochs; the paper averages 100 after "
                         "10); one GPU, prints its own JSON line")
    args = ap.parse_args()
    rank, local_rank, world = dist_env()
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.gcn_epoch:
        if rank == 0:
            run_gcn_epoch(args, local_rank)
        return
    if args.probe_paths:
        if rank == 0:
            run_probe_paths(args, local_rank)
        return
    if args.regret:
        if rank == 0:
            run_regret(args, local_rank)
        return
    if args.split == "rows":
        run_row_split(args, rank, local_rank, world)
        return
    run_gpu(args, rank, local_rank, world)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
