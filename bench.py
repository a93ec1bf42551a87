#!/usr/bin/env python
"""Benchmark of the SPMM / SDDMM / FusedMM hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl b200|reference]

One *step* = one pass of the whole hot path over one synthetic problem: SPMM, SDDMM and FusedMM
once each on the same CSR pattern (row extents, work assignment, index staging, sampled dot
products, their store, the gather-AXPY sweep, the output store and the fused pass).
Metric: GFLOP/s with 2*nnz*width flop per stage (FusedMM = its two stages), whole job.

Default workload `sweep_d30_n128`: S 8192 x 8192, power-law row lengths at 30% mean density,
Kd = N = 128 -- the size, width and density of the paper's headline case (8k/8k/128/70%).

Prints ONE JSON line (rank 0).  `value` has all inputs resident in HBM; `e2e` goes through the
host-buffer C-ABI entry points with the copies inside the timed region.
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

from paper_2311_00368_b200 import replicas  # noqa: E402
from paper_2311_00368_b200 import workloads as W  # noqa: E402

OPS = ("spmm", "sddmm", "fusedmm")
SM_COUNT, FP32_LANES_PER_SM = 148, 128
L2_FLUSH_BYTES = 256 << 20

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel,
# from the ncu captures summarised under profiles/; None where no capture exists yet.
MEASURED_TRAFFIC_BYTES = {
    # (workload, kernel family of the FusedMM op) -> bytes; see profiles/fusedmm_row_sweep_d30_n128.md
    ("sweep_d30_n128", "row"): 182_986_752,
    # profiles/fusedmm_tile_sweep_d30_n128.md (the kernel reads the window table, not col_idx)
    ("sweep_d30_n128", "tile"): 127_987_200,
}


def make_workload(name: str, rank: int = 0) -> W.Problem:
    if name.startswith("sweep_d"):
        d, n = name[len("sweep_d"):].split("_n")
        return W.sweep_case(int(d) / 100.0, int(n), seed=replicas.instance_seed(4, rank))
    if name == "tiny":
        return W.tiny(replicas.instance_seed(0, rank))
    if name == "spmm":
        p = W.spmm_case(replicas.instance_seed(1, rank))
        rng = np.random.default_rng(99)
        p.Kd, p.A, p.B = 128, W.dense_normal(rng, p.M, 128), W.dense_normal(rng, p.K, 128)
        return p
    if name == "sddmm":
        p = W.sddmm_case(replicas.instance_seed(2, rank))
        rng = np.random.default_rng(99)
        p.N, p.D = 128, W.dense_normal(rng, p.K, 128)
        return p
    if name.startswith("attn"):
        return W.attention_case(int(name[4:] or 0) + 8 * rank)
    if name.startswith("grid_"):
        return W.paper_grid_case(name, seed=replicas.instance_seed(5, rank))
    raise SystemExit(f"unknown workload {name}")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        m = json.load(open(path))
        return float(m["hbm_gbs"]), float(m.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


class ClockSampler:
    """Samples SM clock, power and throttle reasons (read-only NVML queries) from a thread while the
    timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.004):
        self.idx, self.period, self.rows = device_index, period_s, []
        self._stop = threading.Event()
        self.t = None
        self.err = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            import torch
            uuid = "GPU-" + str(torch.cuda.get_device_properties(self.idx).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(self.idx)
            self.nv = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # noqa: BLE001
            self.err = f"NVML unavailable: {e}"
            return
        self.t = threading.Thread(target=self._loop, daemon=True)
        self.t.start()

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                try:
                    power = nv.nvmlDeviceGetPowerUsage(self.h) / 1e3
                except Exception:
                    power = float("nan")
                self.rows.append((mhz, reasons, power))
            except Exception as e:  # noqa: BLE001
                self.err = str(e)
                return
            time.sleep(self.period)

    def stop(self):
        if self.t is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [self.err or "not sampled"]}
        self._stop.set()
        self.t.join(timeout=2)
        nv = self.nv
        bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                "sw_power_cap": 0x4, "hw_power_brake_slowdown": 0x80}
        seen = set()
        for _, r, _ in self.rows:
            for name, bit in bits.items():
                if r & bit:
                    seen.add(name)
        sm = [r[0] for r in self.rows]
        pw = [r[2] for r in self.rows if r[2] == r[2]]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": self.max_mhz, "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(seen)}


def oracle_sample(p: W.Problem, budget_s: float):
    """Times the CPU oracle (as it stands) on a bounded sample of the workload: the first R rows of
    S for all three ops, R sized from a short calibration so the sample costs about budget_s."""
    import oracle
    M = p.M

    def run(r1):
        t0 = time.perf_counter()
        oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D, rows=(0, r1))
        oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, rows=(0, r1))
        oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D, rows=(0, r1))
        return time.perf_counter() - t0

    r_cal = min(M, max(oracle.num_threads() * 16, 64))
    run(min(M, 8))  # load the library, touch the pages
    t_cal = run(r_cal)
    nnz_cal = int(p.row_ptr[r_cal])
    if r_cal >= M or t_cal >= budget_s:
        rows, t, nnz_s = r_cal, t_cal, nnz_cal
    else:
        want_nnz = nnz_cal * budget_s / max(t_cal, 1e-6)
        rows = int(np.searchsorted(p.row_ptr, min(want_nnz, p.nnz), side="left"))
        rows = max(r_cal, min(M, rows))
        t = run(rows)
        nnz_s = int(p.row_ptr[rows])
    fl = sum(W.flops(op, nnz_s, p.Kd, p.N) for op in OPS)
    return {"value": fl / t / 1e9, "unit": "GFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"rows 0..{rows} of {M} ({nnz_s} of {p.nnz} nonzeros), spmm+sddmm+fusedmm once, "
                      f"{t:.1f} s", "rows": rows}, t


def parity_on_sample(p, rows, gpu_spmm, gpu_sddmm, gpu_fused):
    """Element-wise check of the timed run's own outputs against the oracle on rows [0, rows):
    |gpu - ref| <= 1e-5 * sum|terms| + 1e-6.  Part of the cpu_baseline leg (the oracle runs here anyway)."""
    import oracle
    nnz_s = int(p.row_ptr[rows])
    out = {"rows": int(rows), "tolerance": "|gpu-ref| <= 1e-5*sum|terms| + 1e-6", "ops": {}}
    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D, rows=(0, rows))
    ok, ratio = oracle.within_tolerance(gpu_spmm[:rows].cpu().numpy(), ref, T)
    out["ops"]["spmm"] = {"ok": bool(ok), "worst_error_over_allowed": float(ratio)}
    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, rows=(0, rows))
    ok, ratio = oracle.within_tolerance(gpu_sddmm[:nnz_s].cpu().numpy(), ref, T)
    out["ops"]["sddmm"] = {"ok": bool(ok), "worst_error_over_allowed": float(ratio)}
    ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D, rows=(0, rows))
    ok, ratio = oracle.within_tolerance(gpu_fused[:rows].cpu().numpy(), ref, T)
    out["ops"]["fusedmm"] = {"ok": bool(ok), "worst_error_over_allowed": float(ratio)}
    out["ok"] = all(v["ok"] for v in out["ops"].values())
    return out


def time_calls(torch, stream, flush, fn, reps):
    """Mean and minimum device time (ms) of `fn` over `reps` calls, L2 flushed (untimed) before each."""
    ev = []
    for _ in range(reps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        ev.append((e0, e1))
    torch.cuda.synchronize()
    ms = [a.elapsed_time(z) for a, z in ev]
    return float(np.mean(ms)), float(np.min(ms))


def measure_problems(torch, b, device, flush, problems, ops, fp32_peak_gflops, hbm_gbs, reps, check=True):
    """One entry of the bench line's `configs` object: the given ops on a list of independent problems of one
    configuration (eight for the attention-shaped one, else one), per op summed over the problems.  Same
    protocol as the headline: L2 flushed before every call, CUDA events on the launching stream.  Three
    timings per op: the window table of S prepared once and reused (`ms`), a stateless call that rebuilds it
    (`stateless_ms`), and the CUDA-core row family (`row_ms`).  Every output of the prepared calls is
    checked against the oracle, every element."""
    import oracle
    stream = torch.cuda.current_stream()
    dev = lambda x: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).to(device)
    out = {"problems": len(problems), "ops": {}}
    acc = {op: {"ms": 0.0, "ms_min": 0.0, "stateless_ms": 0.0, "row_ms": 0.0, "flops": 0, "bytes": 0, "worst": 0.0,
                "ok": True, "algo": None, "launches": 0} for op in ops}
    for p in problems:
        rp, ci, v, A, B, D = map(dev, (p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D))
        O = torch.empty((p.M, max(p.N, 1)), dtype=torch.float32, device=device)
        C = torch.empty(p.nnz, dtype=torch.float32, device=device)
        ws = torch.empty(max(b.workspace_bytes(i, p.M, p.K, p.Kd, p.N, p.nnz) for i in range(3)),
                         dtype=torch.uint8, device=device)
        calls = {"spmm": lambda a: b.spmm(rp, ci, v, D, K=p.K, out=O, workspace=ws, algo=a),
                 "sddmm": lambda a: b.sddmm(rp, ci, v, A, B, out=C, workspace=ws, algo=a),
                 "fusedmm": lambda a: b.fusedmm(rp, ci, v, A, B, D, out=O, workspace=ws, algo=a)}
        for op in ops:
            i = OPS.index(op)
            calls[op](b.ALGO_AUTO)
            torch.cuda.synchronize()
            auto = b.last_algo(i)
            a = acc[op]
            a["algo"] = b.ALGO_NAMES[auto]
            if auto == b.ALGO_TILE:
                b.prepare_pattern(rp, ci, p.K, ws)
                fn = lambda: calls[op](b.ALGO_TILE_PREPARED)
            else:
                fn = lambda: calls[op](b.ALGO_AUTO)
            for _ in range(3):
                fn()
            mean, mn = time_calls(torch, stream, flush, fn, reps)
            a["launches"] += b.last_launches(i)
            a["ms"] += mean
            a["ms_min"] += mn
            if check:
                got = (C if op == "sddmm" else O).cpu().numpy()
                if op == "spmm":
                    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, p.D)
                elif op == "sddmm":
                    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, p.A, p.B)
                else:
                    ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
                ok, ratio = oracle.within_tolerance(got, ref, T)
                a["ok"] = a["ok"] and bool(ok) and b.device_status(ws) == 0
                a["worst"] = max(a["worst"], float(ratio))
            fn = lambda: calls[op](b.ALGO_AUTO)
            for _ in range(3):
                fn()
            a["stateless_ms"] += time_calls(torch, stream, flush, fn, reps)[0]
            fn = lambda: calls[op](b.ALGO_ROW)
            fn()
            a["row_ms"] += time_calls(torch, stream, flush, fn, max(3, reps // 4))[0]
            a["flops"] += W.flops(op, p.nnz, p.Kd, p.N)
            a["bytes"] += W.compulsory_bytes(op, p.M, p.K, p.nnz, p.Kd, p.N)
        del rp, ci, v, A, B, D, O, C, ws
    for op, a in acc.items():
        t_alu = a["flops"] / (fp32_peak_gflops * 1e9)
        t_hbm = a["bytes"] / (hbm_gbs * 1e9)
        t_roof = max(t_alu, t_hbm)
        out["ops"][op] = {"ms": round(a["ms"], 4), "ms_min": round(a["ms_min"], 4),
                          "roofline_frac": round(t_roof / (a["ms"] * 1e-3), 4),
                          "roofline_bound": "alu" if t_alu >= t_hbm else "hbm",
                          "gflops": round(a["flops"] / a["ms"] / 1e6, 1),
                          "algo": a["algo"] + (" (window table prepared once)" if a["algo"] == "tile" else ""),
                          "launches": a["launches"],
                          "stateless_ms": round(a["stateless_ms"], 4),
                          "stateless_roofline_frac": round(t_roof / (a["stateless_ms"] * 1e-3), 4),
                          "row_family_ms": round(a["row_ms"], 4),
                          "parity_ok": a["ok"] if check else None,
                          "parity_worst_error_over_allowed": round(a["worst"], 4) if check else None}
    return out


def measure_batched(torch, b, device, flush, problems, fp32_peak_gflops, hbm_gbs, reps, check=True):
    """The attention-shaped configuration through b2sp_fusedmm_batched: all problems in ONE call (one pattern
    pre-pass, one operand pre-pass, one tile launch).  Same protocol and fields as measure_problems."""
    import oracle
    stream = torch.cuda.current_stream()
    nb, p0 = len(problems), problems[0]
    stride = (max(p.nnz for p in problems) + 3) // 4 * 4
    ci = np.zeros((nb, stride), dtype=np.int32)
    sv = np.zeros((nb, stride), dtype=np.float32)
    for i, p in enumerate(problems):
        ci[i, :p.nnz], sv[i, :p.nnz] = p.col_idx, p.values
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(device)
    rp, ci, sv = dev(np.stack([p.row_ptr for p in problems])), dev(ci), dev(sv)
    A, B, D = (dev(np.stack([getattr(p, k) for p in problems])) for k in "ABD")
    O = torch.empty((nb, p0.M, p0.N), dtype=torch.float32, device=device)
    ws = torch.empty(b.workspace_bytes_batched(nb, p0.M, p0.K, p0.Kd, p0.N, stride), dtype=torch.uint8, device=device)
    call = lambda a: b.fusedmm_batched(rp, ci, sv, A, B, D, out=O, workspace=ws, algo=a)
    call(b.ALGO_AUTO)
    torch.cuda.synchronize()
    auto = b.last_algo(2)
    if auto == b.ALGO_TILE:
        b.prepare_pattern_batched(rp, ci, p0.K, ws)
        fn = lambda: call(b.ALGO_TILE_PREPARED)
    else:
        fn = lambda: call(b.ALGO_AUTO)
    for _ in range(3):
        fn()
    mean, mn = time_calls(torch, stream, flush, fn, reps)
    launches = b.last_launches(2)
    ok, worst = True, 0.0
    if check:
        got = O.cpu().numpy()
        for i, p in enumerate(problems):
            ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D)
            k, ratio = oracle.within_tolerance(got[i], ref, T)
            ok, worst = ok and bool(k), max(worst, float(ratio))
        ok = ok and b.device_status(ws) == 0
    fn = lambda: call(b.ALGO_AUTO)
    for _ in range(3):
        fn()
    stateless = time_calls(torch, stream, flush, fn, reps)[0]
    # the same batch with bfloat16 Q, K, V (fp32 accumulation), prepared tables
    bf16_ms = None
    if auto == b.ALGO_TILE:
        A16, B16, D16 = (t.to(torch.bfloat16) for t in (A, B, D))
        b.prepare_pattern_batched(rp, ci, p0.K, ws)
        fn = lambda: b.fusedmm_batched(rp, ci, sv, A16, B16, D16, out=O, workspace=ws, algo=b.ALGO_TILE_PREPARED,
                                       dtype=torch.bfloat16)
        for _ in range(3):
            fn()
        bf16_ms = time_calls(torch, stream, flush, fn, reps)[0]
        del A16, B16, D16
    flops = sum(W.flops("fusedmm", p.nnz, p.Kd, p.N) for p in problems)
    nbytes = sum(W.compulsory_bytes("fusedmm", p.M, p.K, p.nnz, p.Kd, p.N) for p in problems)
    t_alu, t_hbm = flops / (fp32_peak_gflops * 1e9), nbytes / (hbm_gbs * 1e9)
    t_roof = max(t_alu, t_hbm)
    return {"ms": round(mean, 4), "ms_min": round(mn, 4), "roofline_frac": round(t_roof / (mean * 1e-3), 4),
            "roofline_bound": "alu" if t_alu >= t_hbm else "hbm", "gflops": round(flops / mean / 1e6, 1),
            "algo": b.ALGO_NAMES[auto] + (" (window tables prepared once)" if auto == b.ALGO_TILE else ""),
            "launches": launches, "stateless_ms": round(stateless, 4),
            "stateless_roofline_frac": round(t_roof / (stateless * 1e-3), 4),
            "call": f"b2sp_fusedmm_batched, {nb} problems in one call",
            "bf16_operands_ms": None if bf16_ms is None else round(bf16_ms, 4),
            "parity_ok": ok if check else None, "parity_worst_error_over_allowed": round(worst, 4) if check else None}


# The "largest configurations" besides the headline workload: SPMM config, SDDMM config, the eight
# attention-shaped problems, and the 30% sweep points at the wider outputs.
EXTRA_CONFIGS = (
    ("spmm_2048_d20_n256", lambda: [W.spmm_case()], ("spmm",)),
    ("sddmm_4096_d10_kd128", lambda: [W.sddmm_case()], ("sddmm",)),
    ("attention_8x4096_d20_hd64", lambda: [W.attention_case(i) for i in range(8)], ("fusedmm", "sddmm", "spmm")),
    ("sweep_d30_n256", lambda: [W.sweep_case(0.3, 256)], OPS),
    ("sweep_d30_n512", lambda: [W.sweep_case(0.3, 512)], OPS),
)


def run_reference(args):
    rank, _, world = replicas.env_world()
    if rank != 0:
        return 0
    p = make_workload(args.workload)
    total = args.steps + args.warmup
    budget = min(20.0, 150.0 / max(total, 1))
    vals, secs = [], []
    for s in range(total):
        cb, t = oracle_sample(p, budget)
        if s >= args.warmup:
            vals.append(cb["value"]); secs.append(t)
    v = float(np.mean(vals))
    cb["value"] = v
    cb.pop("rows", None)
    line = {"impl": "reference", "metric": "SPMM+SDDMM+FusedMM GFLOP/s (2*nnz*width per stage)",
            "value": v, "unit": "GFLOP/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": float(np.mean(secs)) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(p, args.workload),
            "cpu_baseline": cb,
            "e2e": {"value": v, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def workload_config(p, name):
    lens = np.diff(p.row_ptr)
    return {"workload": name, "M": p.M, "K": p.K, "Kd": p.Kd, "N": p.N, "nnz": int(p.nnz),
            "density": round(p.nnz / (p.M * p.K), 4),
            "row_len_min_med_max": [int(lens.min()), int(np.median(lens)), int(lens.max())],
            "step": "spmm + sddmm + fusedmm, once each",
            "l2": "flushed between steps (256 MiB write, untimed)"}


def run_grid(args):
    """The paper's evaluation grid on one GPU: per case and op, the minimum of 20 warm calls (the paper's
    protocol: minimum of 20 runs, operands cache-warm) through the stateless C-ABI entry points with
    algo = AUTO, timed call by call with CUDA events and as 20 calls inside one CUDA graph, the fraction of the roofline, and the parity of the timed outputs against the oracle on a
    bounded sample of rows (with the oracle's own rate on that sample: the cpu_baseline of the case)."""
    import torch
    from paper_2311_00368_b200 import binding as b
    import oracle

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    hbm_gbs, sm_max_mhz, _ = peaks()
    fp32_peak = SM_COUNT * FP32_LANES_PER_SM * 2 * sm_max_mhz / 1e3   # GFLOP/s
    stream = torch.cuda.current_stream()
    for name in W.paper_grid_names():
        if args.grid_filter and args.grid_filter not in name:
            continue
        p = make_workload(name)
        dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(device)
        rp, ci, v, A, B, D = map(dev, (p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D))
        O = torch.empty((p.M, p.N), dtype=torch.float32, device=device)
        O2 = torch.empty_like(O)
        C = torch.empty(p.nnz, dtype=torch.float32, device=device)
        ws = torch.empty(max(b.workspace_bytes(op, p.M, p.K, p.Kd, p.N, p.nnz, 0) for op in range(3)),
                         dtype=torch.uint8, device=device)
        calls = {"sddmm": lambda: b.sddmm(rp, ci, v, A, B, out=C, workspace=ws, algo=0),
                 "spmm": lambda: b.spmm(rp, ci, v, D, K=p.K, out=O2, workspace=ws, algo=0),
                 "fusedmm": lambda: b.fusedmm(rp, ci, v, A, B, D, out=O, workspace=ws, algo=0)}
        line = {"workload": name, "M": p.M, "K": p.K, "N": p.N, "nnz": p.nnz, "ops": {}}
        for i, op in enumerate(("sddmm", "spmm", "fusedmm")):
            for _ in range(3):
                calls[op]()
            ev = []
            for _ in range(20):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                calls[op]()
                e1.record(stream)
                ev.append((e0, e1))
            torch.cuda.synchronize()
            ms = [x.elapsed_time(y) for x, y in ev]
            # the same call 20 times inside one CUDA graph: device time per call without the host's launch
            # latency, which is all a 5-us kernel shows when it is timed call by call from Python
            ms_graph = None
            try:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for _ in range(20):
                        calls[op]()
                reps = []
                for _ in range(5):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    g.replay()
                    e1.record(stream)
                    torch.cuda.synchronize()
                    reps.append(e0.elapsed_time(e1) / 20)
                ms_graph = float(np.min(reps))
                del g
            except Exception:   # a capture that fails leaves the call-by-call number
                torch.cuda.synchronize()
            fl = W.flops(op, p.nnz, p.Kd, p.N)
            by = W.compulsory_bytes(op, p.M, p.K, p.nnz, p.Kd, p.N)
            t_roof = max(fl / (fp32_peak * 1e9), by / (hbm_gbs * 1e9))
            best = min(float(np.min(ms)), ms_graph) if ms_graph else float(np.min(ms))
            line["ops"][op] = {"ms_min": round(float(np.min(ms)), 4), "ms_median": round(float(np.median(ms)), 4),
                               "ms_in_graph": round(ms_graph, 4) if ms_graph else None,
                               "gflops": round(fl / best / 1e6, 1),
                               "roofline_frac": round(t_roof / (best * 1e-3), 4),
                               "algo": b.ALGO_NAMES[b.last_algo({"spmm": 0, "sddmm": 1, "fusedmm": 2}[op])]}
        rows = min(p.M, 64)
        t0 = time.perf_counter()
        par = parity_on_sample(p, rows, O2, C, O)
        t = time.perf_counter() - t0
        nnz_s = int(p.row_ptr[rows])
        line["parity_ok"] = par["ok"]
        line["parity_worst"] = max(x["worst_error_over_allowed"] for x in par["ops"].values())
        line["cpu_baseline"] = {"value": round(sum(W.flops(op, nnz_s, p.Kd, p.N) for op in OPS) / t / 1e9, 2),
                                "unit": "GFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                                "sample": f"rows 0..{rows}, spmm+sddmm+fusedmm once"}
        print(json.dumps(line), flush=True)
        del rp, ci, v, A, B, D, O, O2, C, ws
        torch.cuda.empty_cache()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="sweep_d30_n128")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--algo", type=int, default=0, help="B2SP_ALGO_* (0 = auto)")
    ap.add_argument("--no-prepare", action="store_true",
                    help="every op rebuilds S's window table itself instead of sharing one per step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the `configs` object (the other large configurations, timed beside the headline workload)")
    ap.add_argument("--config-reps", type=int, default=50, help="timed calls per op of the `configs` object")
    ap.add_argument("--min-warmup", type=int, default=3,
                    help="lower bound on warm-up steps (only profiler captures go below 3)")
    ap.add_argument("--grid", action="store_true",
                    help="run the paper's 72-case grid (uniform-random stand-ins), one JSON line per case")
    ap.add_argument("--grid-filter", default="", help="only grid cases whose name contains this text")
    ap.add_argument("--shard-rows", action="store_true",
                    help="N > 1: one problem cut into contiguous row ranges of about equal stored entries, one per rank "
                         "(strong scaling; B and D replicated, no data-path collective) instead of one instance per rank")
    ap.add_argument("--only-config", default="",
                    help="time just this entry of the `configs` object (for profiler captures) and print it")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.grid:
        return run_grid(args)

    import torch
    from paper_2311_00368_b200 import binding as b  # raises if libb2sp.so is missing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    rank, local_rank, world = replicas.env_world()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    replicas.init("nccl", device)
    hbm_gbs, sm_max_mhz, peak_src = peaks()
    fp32_peak_gflops = SM_COUNT * FP32_LANES_PER_SM * 2 * sm_max_mhz / 1e3

    if args.only_config:
        flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
        for cname, make, cops in EXTRA_CONFIGS:
            if cname != args.only_config:
                continue
            probs = make()
            if cname.startswith("attention"):
                res = measure_batched(torch, b, device, flush, probs, fp32_peak_gflops, hbm_gbs, args.config_reps, check=False)
            else:
                res = measure_problems(torch, b, device, flush, probs, cops, fp32_peak_gflops, hbm_gbs, args.config_reps, check=False)
            print(json.dumps({"config": cname, "result": res}))
        return 0

    p = make_workload(args.workload, 0 if args.shard_rows else rank)
    if args.shard_rows and world > 1:
        r0, r1, rp_loc, ci_loc, v_loc, A_loc = replicas.row_shard(p.row_ptr, p.col_idx, p.values, rank, world, A=p.A)
        p = W.Problem(p.name, r1 - r0, p.K, rp_loc, np.ascontiguousarray(ci_loc), np.ascontiguousarray(v_loc), p.Kd, p.N,
                      np.ascontiguousarray(A_loc), p.B, p.D)
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(device)
    rp, ci, v, A, B, D = map(dev, (p.row_ptr, p.col_idx, p.values, p.A, p.B, p.D))
    O = torch.empty((p.M, p.N), dtype=torch.float32, device=device)
    O2 = torch.empty_like(O)
    C = torch.empty(p.nnz, dtype=torch.float32, device=device)
    ws_bytes = max(b.workspace_bytes(op, p.M, p.K, p.Kd, p.N, p.nnz) for op in range(3))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream()

    # Which kernel family does the library pick for each op?  If all three resolve to the dense-tile
    # family, a step builds S's window table once (b2sp_prepare_pattern) and the ops share it.
    probe = {"spmm": lambda a: b.spmm(rp, ci, v, D, K=p.K, out=O2, workspace=ws, algo=a),
             "sddmm": lambda a: b.sddmm(rp, ci, v, A, B, out=C, workspace=ws, algo=a),
             "fusedmm": lambda a: b.fusedmm(rp, ci, v, A, B, D, out=O, workspace=ws, algo=a)}
    op_algo = {op: args.algo for op in OPS}
    shared_table = False
    if args.algo == b.ALGO_AUTO and not args.no_prepare:
        for op in OPS:
            probe[op](b.ALGO_AUTO)
        torch.cuda.synchronize()
        if all(b.last_algo(i) == b.ALGO_TILE for i in range(3)):
            shared_table = True
            op_algo = {op: b.ALGO_TILE_PREPARED for op in OPS}
    calls = {op: (lambda op=op: probe[op](op_algo[op])) for op in OPS}
    fl = {op: W.flops(op, p.nnz, p.Kd, p.N) for op in OPS}
    by = {op: W.compulsory_bytes(op, p.M, p.K, p.nnz, p.Kd, p.N) for op in OPS}

    def step(events=None):
        if shared_table:
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            b.prepare_pattern(rp, ci, p.K, ws)
            if events is not None:
                e1.record(stream)
                events.append(("prepare", e0, e1))
        for op in OPS:
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            calls[op]()
            if events is not None:
                e1.record(stream)
                events.append((op, e0, e1))

    for _ in range(max(args.warmup, args.min_warmup)):
        flush.fill_(1)
        step()
    torch.cuda.synchronize()
    launches = {op: b.last_launches(i) for i, op in enumerate(OPS)}
    algos = {op: b.ALGO_NAMES[b.last_algo(i)] for i, op in enumerate(OPS)}

    sampler = ClockSampler(local_rank)
    replicas.barrier()
    torch.cuda.synchronize()
    if rank == 0:
        sampler.start()
    events, step_events = [], []
    for _ in range(args.steps):
        flush.fill_(1)  # evict the operands from L2 (untimed)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        step(events)
        s1.record(stream)
        step_events.append((s0, s1))
    torch.cuda.synchronize()
    replicas.barrier()
    clocks = sampler.stop() if rank == 0 else None
    step_ms = [a.elapsed_time(z) for a, z in step_events]
    total_ms_local = float(np.sum(step_ms))
    total_ms = replicas.max_over_ranks(total_ms_local, device)
    flops_all = replicas.sum_over_ranks(float(sum(fl.values())), device)
    ms_per_step = total_ms / args.steps
    value = flops_all / (ms_per_step * 1e-3) / 1e9

    per_op = {}
    for op in OPS:
        ms = [a.elapsed_time(z) for (o, a, z) in events if o == op]
        mean_ms, min_ms = float(np.mean(ms)), float(np.min(ms))
        t_alu = fl[op] / (fp32_peak_gflops * 1e9)
        t_hbm = by[op] / (hbm_gbs * 1e9)
        per_op[op] = {"ms": round(mean_ms, 4), "ms_min": round(min_ms, 4),
                      "gflops": round(fl[op] / mean_ms / 1e6, 1),
                      "gflops_at_min": round(fl[op] / min_ms / 1e6, 1),
                      "compulsory_gbs": round(by[op] / mean_ms / 1e6, 1),
                      "roofline_bound": "alu" if t_alu >= t_hbm else "hbm",
                      "roofline_frac": round(max(t_alu, t_hbm) / (mean_ms * 1e-3), 4),
                      "launches": launches[op], "algo": algos[op]}
    prep_ms = [a.elapsed_time(z) for (o, a, z) in events if o == "prepare"]
    if prep_ms:
        per_op["prepare_pattern"] = {"ms": round(float(np.mean(prep_ms)), 4), "ms_min": round(float(np.min(prep_ms)), 4),
                                     "launches": 1, "note": "S's window table, built once per step, shared by the three ops"}
    # warm protocol (no L2 flush; the paper's statistic is the minimum of 20 runs): per op, 20 calls
    for op in OPS:
        calls[op]()
        ev = []
        for _ in range(20):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            calls[op]()
            e1.record(stream)
            ev.append((e0, e1))
        torch.cuda.synchronize()
        warm = [a.elapsed_time(z) for a, z in ev]
        per_op[op]["warm_ms_min"] = round(float(np.min(warm)), 4)
        per_op[op]["warm_ms_median"] = round(float(np.median(warm)), 4)
    # the same ops as stateless calls (each builds S's window table itself), L2 flushed before every call
    if shared_table:
        for i, op in enumerate(OPS):
            fn = lambda op=op: probe[op](b.ALGO_AUTO)
            for _ in range(3):
                fn()
            mean, mn = time_calls(torch, stream, flush, fn, 20)
            t_roof = max(fl[op] / (fp32_peak_gflops * 1e9), by[op] / (hbm_gbs * 1e9))
            per_op[op]["stateless_ms"] = round(mean, 4)
            per_op[op]["stateless_roofline_frac"] = round(t_roof / (mean * 1e-3), 4)
            per_op[op]["stateless_launches"] = b.last_launches(i)
        step()   # the outputs the parity check reads come from the timed configuration (prepared table)
        torch.cuda.synchronize()
    # the same workload with bfloat16 dense operands and fp32 accumulation (b2sp_*_bf16), beside the fp32 ops
    bf16 = None
    if shared_table:
        A16, B16, D16 = (t.to(torch.bfloat16) for t in (A, B, D))
        O16 = torch.empty_like(O)
        C16 = torch.empty_like(C)
        b.prepare_pattern(rp, ci, p.K, ws)
        bcalls = {"spmm": lambda: b.spmm(rp, ci, v, D16, K=p.K, out=O16, workspace=ws, algo=b.ALGO_TILE_PREPARED, dtype=torch.bfloat16),
                  "sddmm": lambda: b.sddmm(rp, ci, v, A16, B16, out=C16, workspace=ws, algo=b.ALGO_TILE_PREPARED, dtype=torch.bfloat16),
                  "fusedmm": lambda: b.fusedmm(rp, ci, v, A16, B16, D16, out=O16, workspace=ws, algo=b.ALGO_TILE_PREPARED, dtype=torch.bfloat16)}
        bf16 = {"dtype": "bf16 A/B/D, fp32 S values, one tf32 MMA per exact product, fp32 accumulate", "ops": {}}
        rows16 = min(p.M, 256)
        nnz16 = int(p.row_ptr[rows16])
        for op in OPS:
            for _ in range(3):
                bcalls[op]()
            mean, mn = time_calls(torch, stream, flush, bcalls[op], 20)
            t_roof = max(fl[op] / (fp32_peak_gflops * 1e9), by[op] / (hbm_gbs * 1e9))
            bf16["ops"][op] = {"ms": round(mean, 4), "ms_min": round(mn, 4),
                               "fp32_roofline_frac": round(t_roof / (mean * 1e-3), 4),
                               "speedup_over_fp32": round(per_op[op]["ms"] / mean, 3)}
            if not args.no_cpu_baseline and rank == 0:
                import oracle
                r16 = lambda t: t.to(torch.float32).cpu().numpy()
                if op == "spmm":
                    ref, T = oracle.spmm(p.row_ptr, p.col_idx, p.values, r16(D16), rows=(0, rows16))
                    got = O16[:rows16]
                elif op == "sddmm":
                    ref, T = oracle.sddmm(p.row_ptr, p.col_idx, p.values, r16(A16), r16(B16), rows=(0, rows16))
                    got = C16[:nnz16]
                else:
                    ref, T = oracle.fusedmm(p.row_ptr, p.col_idx, p.values, r16(A16), r16(B16), r16(D16), rows=(0, rows16))
                    got = O16[:rows16]
                ok, ratio = oracle.within_tolerance(got.cpu().numpy(), ref, T)
                bf16["ops"][op]["parity_ok"] = bool(ok)
                bf16["ops"][op]["parity_worst_error_over_allowed"] = round(float(ratio), 4)
                bf16["ops"][op]["parity_rows"] = rows16
        bf16["fused_speedup_over_separate_launches"] = round(
            (bf16["ops"]["sddmm"]["ms"] + bf16["ops"]["spmm"]["ms"]) / bf16["ops"]["fusedmm"]["ms"], 3)
        del A16, B16, D16, O16, C16
    sep_ms = per_op["sddmm"]["ms"] + per_op["spmm"]["ms"]
    fused_vs_separate = sep_ms / per_op["fusedmm"]["ms"]

    # roofline object for the dominant kernel (FusedMM): FP32-FMA bound on this workload
    dom = "fusedmm"
    dom_ms = per_op[dom]["ms"]
    t_alu = fl[dom] / (fp32_peak_gflops * 1e9)
    t_hbm = by[dom] / (hbm_gbs * 1e9)
    if t_alu >= t_hbm:
        roof = {"bound": "alu", "achieved": fl[dom] / dom_ms / 1e9, "peak": fp32_peak_gflops / 1e3,
                "unit": "TFLOP/s"}
        roof["peak_source"] = (f"{SM_COUNT} SMs x {FP32_LANES_PER_SM} FP32 lanes x 2 flop x "
                               f"{sm_max_mhz:.0f} MHz (clocks.max.sm, {peak_src})")
    else:
        roof = {"bound": "hbm", "achieved": by[dom] / dom_ms / 1e6, "peak": hbm_gbs, "unit": "GB/s",
                "peak_source": f"hbm_gbs of {peak_src}"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["kernel"] = dom
    # the same achieved rate against the FP32 FMA rate this GPU sustains right now (register-only FMA
    # chains on every SM, best of 10): the nominal peak assumes clocks.max.sm under load
    probe_gflops = b.probe_fp32_peak(4096, device)
    roof["fp32_fma_probe"] = {"tflops": probe_gflops / 1e3, "achieved_over_probe": fl[dom] / dom_ms / 1e6 / probe_gflops,
                              "how": "b2sp_probe_fp32_peak: 8 FMA chains x 2048 threads x every SM, CUDA events, best of 10"}
    # second resource of the dense-tile kernels: the B / D operand tiles every CTA streams from L2 into shared memory
    # (tf32 hi + lo, 8 bytes per element, once per 128-row tile and 128-column block of S), against the rate at which
    # the SMs can pull 32 KB chunks out of L2 right now
    if algos[dom] == "tile":
        per_sm, total = b.probe_l2_pull(device)
        row_tiles, blocks = -(-p.M // 128), -(-p.K // 128)
        widths = {"spmm": p.N, "sddmm": p.Kd, "fusedmm": p.Kd + p.N}[dom]
        stream_bytes = row_tiles * blocks * 128 * (-(-widths // 32) * 32) * 8
        roof["l2_operand_stream"] = {"bytes_per_launch": stream_bytes, "gbs": stream_bytes / dom_ms / 1e6,
                                     "probe_gbs": total, "probe_gbs_per_sm": per_sm, "frac_of_probe": stream_bytes / dom_ms / 1e6 / total,
                                     "how": "b2sp_probe_l2_pull: cp.async.bulk of 32 KB chunks, three in flight per SM, every SM, best of 5"}
    roof["traffic"] = MEASURED_TRAFFIC_BYTES.get((args.workload, algos[dom]))
    roof["traffic_source"] = ("one ncu capture of this kernel on this workload (dram__bytes_read.sum + dram__bytes_write.sum, "
                              "summary under profiles/), not measured in this run" if roof["traffic"] else None)
    roof["variant"] = ("window table of S prepared once per step and shared by the three ops (its pass is timed inside the "
                       "step and listed under ops.prepare_pattern); ops.*.stateless_* = the same op building the table itself"
                       if shared_table else "stateless calls")
    roof["algorithmic_bytes"] = by[dom]
    roof["algorithmic_flops"] = fl[dom]

    # end to end: host buffers through the C ABI, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        pin = lambda x: torch.from_numpy(np.ascontiguousarray(x)).pin_memory()
        h = {k: pin(x) for k, x in (("rp", p.row_ptr), ("ci", p.col_idx), ("v", p.values), ("A", p.A),
                                    ("B", p.B), ("D", p.D))}
        hO = torch.empty((p.M, p.N), dtype=torch.float32).pin_memory()
        hC = torch.empty(p.nnz, dtype=torch.float32).pin_memory()
        nb = lambda *ts: int(sum(t.numel() * t.element_size() for t in ts))
        h2d = (nb(h["rp"], h["ci"], h["v"], h["D"]) + nb(h["rp"], h["ci"], h["v"], h["A"], h["B"]) +
               nb(h["rp"], h["ci"], h["v"], h["A"], h["B"], h["D"]))
        d2h = nb(hO) + nb(hC) + nb(hO)

        def host_step():
            b.spmm_host(h["rp"], h["ci"], h["v"], h["D"], hO)
            b.sddmm_host(h["rp"], h["ci"], h["v"], h["A"], h["B"], hC)
            b.fusedmm_host(h["rp"], h["ci"], h["v"], h["A"], h["B"], h["D"], hO)

        e2e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            host_step()
        replicas.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            host_step()  # each call synchronises its stream before returning
        torch.cuda.synchronize()
        t_local = (time.perf_counter() - t0) / e2e_steps
        t_e2e = replicas.max_over_ranks(t_local, device)
        e2e = {"value": flops_all / t_e2e / 1e9, "unit": "GFLOP/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": t_e2e * 1e3, "steps": e2e_steps,
               "timer": "host wall clock around synchronous C-ABI calls"}

    # the other large configurations, same protocol
    configs, configs_clocks = None, None
    if rank == 0 and world == 1 and not args.no_configs:
        sampler2 = ClockSampler(local_rank)
        sampler2.start()
        configs = {}
        for cname, make, cops in EXTRA_CONFIGS:
            configs[cname] = measure_problems(torch, b, device, flush, make(), cops, fp32_peak_gflops, hbm_gbs,
                                              args.config_reps, check=not args.no_cpu_baseline)
            if cname.startswith("attention"):
                probs = make()
                o = configs[cname]["ops"]
                o["fusedmm_one_call_each"] = o["fusedmm"]
                o["fusedmm"] = measure_batched(torch, b, device, flush, probs, fp32_peak_gflops, hbm_gbs,
                                               args.config_reps, check=not args.no_cpu_baseline)
                del probs
            if set(("sddmm", "spmm", "fusedmm")) <= set(cops):
                o = configs[cname]["ops"]
                configs[cname]["fused_speedup_over_separate_launches"] = round(
                    (o["sddmm"]["ms"] + o["spmm"]["ms"]) / o["fusedmm"]["ms"], 3)
            torch.cuda.empty_cache()
        configs_clocks = sampler2.stop()

    cpu_baseline, parity = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline, _ = oracle_sample(p, 15.0)
        # the outputs of the last timed step, checked against the oracle on the same sample of rows
        parity = parity_on_sample(p, cpu_baseline.pop("rows"), O2, C, O)

    if rank == 0:
        line = {"metric": "SPMM+SDDMM+FusedMM GFLOP/s (2*nnz*width per stage)", "value": value,
                "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, args.min_warmup),
                "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong" if (args.shard_rows and world > 1) else "weak",
                "vs_baseline": None, "dtype": ("f32 in/out, 3xTF32 products, fp32 accumulate"
                                              if any(a == "tile" for a in algos.values()) else "f32"),
                "data": "synthetic",
                "config": workload_config(p, args.workload),
                "pattern_table": ("built once per step, shared by the ops" if shared_table
                                  else "built inside each op that needs it"),
                "roofline": roof, "cpu_baseline": cpu_baseline, "parity": parity,
                "e2e": e2e, "gpu_launches": int((sum(launches.values()) + (1 if shared_table else 0)) * args.steps),
                "clocks": clocks, "ops": per_op, "bf16": bf16, "configs": configs, "configs_clocks": configs_clocks,
                "fused_speedup_over_separate_launches": round(fused_vs_separate, 3),
                "paper_context": "Intel Max 1550 (1 stack), 8k/8k/128/70%: SDDMM 9732, SPMM 11482, "
                                 "FusedMM 12647 GFLOP/s (other hardware; context only)"}
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
