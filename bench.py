#!/usr/bin/env python
"""Benchmark of the fused DSA indexer top-k on B200.

One "step" is one pass of the whole hot path (sample scoring, sample statistics, fused
score + filter scan, final select, exact fallback rounds) over one synthetic chunk.  Default
workload: `fp8_1m`, the last 4096-query chunk of a 1,048,576-token prefill (H = 64, D = 128,
top-k = 2048, e4m3 codes with per-token fp32 scales), the configuration the headline metric is
quoted on.  The metric is scored (query, key) pairs per second over the causally valid pairs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

N > 1 (launched under torchrun) runs N independent replicas, one per GPU: the path has no exchange
step, so there is no data-path collective; only the timing barrier and the max-over-ranks
reduction go through NCCL.  `--impl reference` times the CPU oracle on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "scored_query_key_pairs_per_second"
UNIT = "pairs/s"
NOMINAL_FP8_TFLOPS = 4500.0
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes of one launch of the fused scan kernel (dram__bytes_read.sum + dram__bytes_write.sum) from an
# ncu capture of a 592-row case of the same workload: 164.3 MB, of which the key stream (N * D bytes, read
# once whatever the number of rows) is 134.2 MB and the rest (candidate write-back, queries, weights) grows
# with the rows: (164.3 - 134.2) MB / 592 rows.
SCAN_TRAFFIC = {"fp8_1m": {"fixed_bytes": 134.2e6, "bytes_per_row": (164.3e6 - 134.2e6) / 592}}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def time_graph_replay(torch, lt, step, flush, reps: int):
    """The same step captured once into a CUDA graph and replayed (L2 flushed between replays, untimed): what is
    left of a step when the host launches nothing.  Phase profiling is off while capturing (event records
    inside a graph cannot be read back)."""
    try:
        lt.lt_set_profiling(False)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        graph.replay()
        torch.cuda.synchronize()
        ms = []
        for _ in range(reps):
            if flush is not None:
                flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            e1.synchronize()
            ms.append(e0.elapsed_time(e1))
        return {"ms_per_step": statistics.mean(ms), "ms_per_step_min": min(ms), "replays": reps}
    except Exception as exc:  # noqa: BLE001 - an extra figure, never the headline
        return {"unavailable": f"{type(exc).__name__}: {exc}"[:160]}
    finally:
        lt.lt_set_profiling(True)


def measure_fp8_gemm(torch, n: int = 8192, sustained_s: float = 2.0):
    """Dense e4m3 x e4m3 -> bf16 GEMM through the library (cuBLASLt via torch._scaled_mm), measured like the
    bf16 peaks of MEASURED_PEAKS.json: best of 10 single launches (burst) and a back-to-back loop (sustained).
    Context for the tensor roofline only; `roofline.peak` stays the measured bf16 figure x the nominal ratio.
    Returns None when this torch build does not offer the call."""
    try:
        a = (torch.randn(n, n, device="cuda") * 0.25).to(torch.float8_e4m3fn)
        b = (torch.randn(n, n, device="cuda") * 0.25).to(torch.float8_e4m3fn)
        one = torch.ones((), device="cuda", dtype=torch.float32)

        def gemm():
            return torch._scaled_mm(a, b.t(), scale_a=one, scale_b=one, out_dtype=torch.bfloat16)

        for _ in range(3):
            gemm()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            gemm()
            e1.record()
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        reps = max(10, int(sustained_s * 1e3 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            gemm()
        e1.record()
        e1.synchronize()
        flops = 2.0 * n * n * n
        return {"burst_tflops": flops / (best * 1e-3) / 1e12,
                "sustained_tflops": flops * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12,
                "how": f"torch._scaled_mm e4m3 {n}^3 -> bf16: best of 10, and {reps} back to back"}
    except Exception as exc:  # noqa: BLE001 - context figure only
        return {"unavailable": f"{type(exc).__name__}: {exc}"[:160]}


def measure_umma_stream(torch, lt, gpu_index: int, seconds: float = 3.0):
    """The library's bare FP8 UMMA stream (lt_debug_umma_stream: tcgen05.mma kind::f8f6f4 tiles of the scan's shape on
    operands resident in shared memory, no TMA, no epilogue), one CTA per SM and as CTA pairs, each launched back to back
    for `seconds` with the SM clock and the board power sampled: the tensor ceiling of this board at the power it is
    granted.  Context for the tensor roofline; `roofline.peak` stays the measured bf16 figure x the nominal ratio."""
    out = {}
    try:
        n_sm = torch.cuda.get_device_properties(0).multi_processor_count
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        iters, per_block = 4000, 20
        for name, pair in (("single", False), ("pair", True)):
            grid = n_sm & ~1 if pair else n_sm
            flops = grid * iters * 16777216.0
            for _ in range(3):
                lt.lt_debug_umma_stream(pair, iters, status)
            torch.cuda.synchronize()
            sampler = ClockSampler(gpu_index)
            sampler.start()
            t0 = time.time()
            ms_blocks = []
            while time.time() - t0 < seconds:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(per_block):
                    lt.lt_debug_umma_stream(pair, iters, status)
                e1.record()
                e1.synchronize()
                ms_blocks.append(e0.elapsed_time(e1) / per_block)
            clocks = sampler.stop()
            tail = ms_blocks[len(ms_blocks) // 2:]  # the steady state: second half of the run
            out[name] = {"tflops": flops / (statistics.median(tail) * 1e-3) / 1e12,
                         "tflops_first_block": flops / (ms_blocks[0] * 1e-3) / 1e12,
                         "sm_mhz": clocks.get("sm_mhz"), "power_w": clocks.get("power_w"), "reasons": clocks.get("reasons")}
        out["status_bits"] = int(status.item())
        out["how"] = (f"{iters} iterations x 8 UMMAs (M128 N256 K32, e4m3) per CTA and launch, launches back to back for "
                      f"{seconds:.0f} s per form; tflops = median of the second half")
    except Exception as exc:  # noqa: BLE001 - context figure only
        return {"unavailable": f"{type(exc).__name__}: {exc}"[:160]}
    return out


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,power.limit,power.draw.instant")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        fields = self.FIELDS
        try:
            probe = subprocess.run(["nvidia-smi", f"--id={self.gpu_index}", "--query-gpu=power.draw.instant", "--format=csv,noheader,nounits"],
                                   capture_output=True, text=True, timeout=20)
            float(probe.stdout.strip().splitlines()[0])
        except (OSError, ValueError, IndexError, subprocess.TimeoutExpired):
            fields = fields.replace(",power.draw.instant", "")  # older drivers: the averaged reading only
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={fields}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, limit, reasons = [], [], [], [], set()
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            try:
                limit.append(float(parts[7]))
                power[-1] = float(parts[8])  # the instantaneous reading where the driver has one (power.draw averages over ~1 s)
            except (ValueError, IndexError):
                pass
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # the busiest samples are the ones under load
        loaded = [c for c, p in zip(sm, power) if power and p >= 0.6 * max(power)] or sm
        loaded_w = [p for p in power if p >= 0.6 * max(power)] or power
        return {"sm_mhz": statistics.median(loaded) if loaded else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w": statistics.median(loaded_w) if loaded_w else None, "power_w_max": max(power) if power else None,
                "power_limit_w": max(limit) if limit else None, "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(value: float, world: int, device) -> float:
    """MAX of a per-rank scalar over all ranks (the timing rule for multi-GPU numbers)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist

    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(pairs_per_rank: int, steps: int, total_ms_max: float, world: int) -> float:
    """Whole-job pairs/s of `world` independent replicas, each doing pairs_per_rank pairs per step,
    when the slowest rank took total_ms_max for its steps."""
    return world * pairs_per_rank * steps / (total_ms_max * 1e-3)


def algorithmic_bytes(inp) -> int:
    """Minimum HBM traffic of one call: read q, w, k (+ k_scale) once, write indices and scores."""
    esz = {"f32": 4, "bf16": 2, "e4m3": 1}[inp.dtype]
    reads = inp.T * inp.H * inp.D * esz + inp.T * inp.H * 4 + inp.N * inp.D * esz + (inp.N * 4 if inp.k_scale is not None else 0)
    return reads + inp.T * inp.topk * 8


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info

        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(inp, budget_s: float, max_rows: int = 64):
    """Times the CPU oracle, as it stands, on a bounded sample of rows of the same workload:
    evenly spaced rows (each against every key it may see), stopping once the budget is spent."""
    from oracle import decode, oracle_topk

    np.matmul(np.ones((64, 64)), np.ones((64, 64)))  # start the BLAS threads
    rows = np.unique(np.linspace(0, inp.T - 1, max_rows).astype(np.int64))
    t0 = time.perf_counter()
    # the oracle decodes K on every call; do the sample in row batches so the budget can stop it
    done_rows, pairs = 0, 0
    batch = 4
    for i in range(0, len(rows), batch):
        chunk = rows[i:i + batch]
        oracle_topk(inp, rows=chunk)
        done_rows += len(chunk)
        pairs += sum(inp.visible(int(t)) for t in chunk)
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return pairs / dt, done_rows, pairs, dt


def run_reference_knn(args):
    """`--impl reference` for the k-NN workloads: the fp64 oracle on a few query rows per step."""
    from oracle import knn_topk
    from workloads import make_knn

    inp = make_knn(args.workload, N=args.knn_corpus or None)
    np.matmul(np.ones((64, 64)), np.ones((64, 64)))
    rows_per_step = 2
    for _ in range(min(args.warmup, 1)):
        knn_topk(inp.q, inp.x, inp.topk, rows=[0])
    vals = []
    budget = args.cpu_budget / max(1, args.steps)
    for s_i in range(args.steps):
        t0 = time.perf_counter()
        done = 0
        while done < inp.T and (done == 0 or time.perf_counter() - t0 < budget):
            r0 = (s_i * 16 + done) % inp.T
            knn_topk(inp.q, inp.x, inp.topk, rows=list(range(r0, min(inp.T, r0 + rows_per_step))))
            done += rows_per_step
        dt = time.perf_counter() - t0
        vals.append((done * inp.N / dt, dt, done))
    value = statistics.mean(v for v, _, _ in vals)
    sample = f"{vals[-1][2]} query rows x the whole corpus per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": statistics.mean(dt for _, dt, _ in vals) * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "T": inp.T, "N": inp.N, "D": inp.D, "topk": inp.topk,
                   "note": "CPU oracle (numpy fp64 matmul + full sort) on a bounded row sample of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_reference(args, rank: int):
    """`--impl reference`: the CPU oracle on the host cores, rank 0 only."""
    if rank != 0:
        return
    if args.workload.startswith("knn"):
        run_reference_knn(args)
        return
    from workloads import make_config

    inp = make_config(args.workload)
    steps_val = []
    for _ in range(args.warmup):
        time_oracle(inp, budget_s=1.0, max_rows=4)
    sample = ""
    for _ in range(args.steps):
        v, rows, pairs, dt = time_oracle(inp, budget_s=args.cpu_budget / max(1, args.steps), max_rows=16)
        steps_val.append((v, dt))
        sample = f"{rows} evenly spaced rows x all visible keys ({pairs} pairs) per step"
    value = statistics.mean(v for v, _ in steps_val)
    ms = statistics.mean(dt for _, dt in steps_val) * 1e3
    cores = cpu_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "T": inp.T, "N": inp.N, "H": inp.H, "D": inp.D, "topk": inp.topk,
                   "causal_offset": inp.causal_offset, "valid_pairs": inp.valid_pairs(), "parallelism": "replicas x1",
                   "note": "CPU oracle (numpy fp64 + full sort) on a bounded row sample of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def time_aux_ops(torch, lt, out_idx, inp, hbm_gbs, peak_kind, reps=5):
    """HBM-bound integer ops that consume a chunk's top-k matrix; algorithmic bytes = the index matrix once + outputs."""
    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(torch.cuda.current_stream())
        for _ in range(reps):
            fn()
        e1.record(torch.cuda.current_stream())
        e1.synchronize()
        return e0.elapsed_time(e1) / reps

    T, k, N = inp.T, inp.topk, inp.N
    out = {}
    n_out = min(3 * k, lt.LT_MAX_TOPK, N)
    pos = torch.empty(n_out, dtype=torch.int32, device="cuda")
    ws = torch.empty(lt.lt_topk_frequent_workspace_bytes(N), dtype=torch.uint8, device="cuda")
    ms = timed(lambda: lt.lt_topk_frequent(out_idx, N, pos, None, ws))
    nbytes = T * k * 4 + N * 4 + n_out * 4  # index matrix once, counts written once, result
    out["lt_topk_frequent"] = {"ms": ms, "algorithmic_bytes": nbytes, "gbs": nbytes / ms / 1e6,
                               "frac_of_hbm_peak": nbytes / ms / 1e6 / hbm_gbs, "peak_kind": peak_kind, "n_out": n_out}
    group = 64
    n_groups = -(-T // group)
    cap = group * k
    upos = torch.empty((n_groups, cap), dtype=torch.int32, device="cuda")
    ulen = torch.empty(n_groups, dtype=torch.int32, device="cuda")
    mask = torch.empty((T, (cap + 31) // 32), dtype=torch.int32, device="cuda")
    ms = timed(lambda: lt.lt_dsa_union_mask(out_idx, N, group, upos, ulen, mask))
    n_union = int(ulen.sum().item())
    # index matrix once + the union entries + one mask bit per (row, union slot of its group), without the
    # clearing of the full-capacity outputs (which the call does with two memsets and which is what dominates)
    nbytes = T * k * 4 + n_union * 4 + sum(int(n) for n in ulen.tolist()) * group // 8
    cleared = upos.numel() * 4 + mask.numel() * 4
    out["lt_dsa_union_mask"] = {"ms": ms, "group": group, "mean_union_len": n_union / n_groups, "algorithmic_bytes": nbytes,
                                "cleared_bytes": cleared, "gbs": nbytes / ms / 1e6, "gbs_with_clears": (nbytes + cleared) / ms / 1e6,
                                "frac_of_hbm_peak": nbytes / ms / 1e6 / hbm_gbs, "peak_kind": peak_kind}
    return out


# ---------------------------------------------------------------------------------------------------------
# the other configurations and the "next" operations, measured briefly in the same run (default line only)
# ---------------------------------------------------------------------------------------------------------
def _timed_ms(torch, fn, steps, flush=None):
    """Mean device time of `steps` calls, each bracketed by CUDA events; L2 flushed (untimed) before each."""
    stream = torch.cuda.current_stream()
    tot = 0.0
    for _ in range(steps):
        if flush is not None:
            flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        e1.synchronize()
        tot += e0.elapsed_time(e1)
    return tot / steps


def measure_config(torch, lt, inp, peaks, flush, steps=5, warmup=3, unfused=True):
    """One configuration through lt_indexer_topk_ex: ms per step, pairs/s, the scan's roofline fraction against
    its own dtype's measured peak, fallback rows, and the decoupled path's time."""
    q, w, k, ks = lt.to_device(inp)
    out_idx = torch.empty((inp.T, inp.topk), dtype=torch.int32, device="cuda")
    out_score = torch.empty((inp.T, inp.topk), dtype=torch.float32, device="cuda")
    ws = lt.alloc_workspace(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk)

    def step():
        lt.lt_indexer_topk_ex(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score, ws)

    for _ in range(warmup):
        step()
    phase = []

    def timed_step():
        step()

    ms = 0.0
    for _ in range(steps):
        ms += _timed_ms(torch, timed_step, 1, flush)
        phase.append(lt.lt_read_phase_ms())
    ms /= steps
    status = lt.lt_read_status(ws)
    pairs = inp.valid_pairs()
    rec = {"workload": inp.name, "dtype": inp.dtype, "T": inp.T, "N": inp.N, "topk": inp.topk, "ms_per_step": ms,
           "pairs_per_s": pairs / (ms * 1e-3), "fallback_rows": status[1], "status_bits": status[0],
           "mean_survivors_per_row": status[3] / inp.T, "steps": steps}
    scan_ms = statistics.mean(p[2] for p in phase)
    rec["phases_ms"] = {"sample": statistics.mean(p[0] + p[1] for p in phase), "fused_scan": scan_ms,
                        "final_select": statistics.mean(p[3] for p in phase), "fallback": statistics.mean(p[4] for p in phase)}
    if inp.dtype in ("bf16", "e4m3") and inp.H == 64 and inp.D == 128:
        peak = peaks["bf16_tflops"] * (2.0 if inp.dtype == "e4m3" else 1.0)
        achieved = 2.0 * inp.H * inp.D * pairs / (scan_ms * 1e-3) / 1e12
        rec["roofline"] = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak}
    else:
        rec["roofline"] = None  # generic SIMT path (a correctness configuration): no phase events either
        rec["phases_ms"] = None
    if unfused:
        buf = torch.empty(256 + (1024 << 20), dtype=torch.uint8, device="cuda")

        def unf():
            lt.lt_unfused_topk(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score, buf)

        unf()
        rec["unfused_ms"] = _timed_ms(torch, unf, 2, flush)
        del buf
    return rec


def measure_other_configs(torch, lt, peaks, flush):
    """tiny_f32, dsa_bf16, fp8_ar1 and the adversarial recipes x topk in {64, 512, 2048, 4096}."""
    import dataclasses

    from workloads import make_config

    out = []
    for name in ("tiny_f32", "dsa_bf16", "fp8_ar1"):
        out.append(measure_config(torch, lt, make_config(name), peaks, flush))
    for name in ("adv_planted", "adv_cluster", "adv_ties", "adv_ties_exact"):
        base = make_config(name)
        for topk in (64, 512, 2048, 4096):
            out.append(measure_config(torch, lt, dataclasses.replace(base, topk=topk), peaks, flush, unfused=(topk == 2048)))
    return out


def measure_next_rows(torch, lt, peaks, peak_kind, flush, main):
    """The "next" operations: paged key cache against the dense layout, the integer ops on the chunk's result,
    the previous-chunk sampler's survivors, and the k-NN variant's scan against the HBM roofline."""
    import dataclasses

    from workloads import make_config

    inp, q, w, k, ks, out_idx, out_score, ws = main
    res = {}
    # ---- paged key cache, random page order, same keys
    n_pages = inp.N // 64
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234)
    table = torch.randperm(n_pages, device="cuda", generator=gen).to(torch.int32)
    k_pool = torch.empty_like(k)
    k_pool.view(n_pages, 64, inp.D)[table.long()] = k.view(n_pages, 64, inp.D)
    ks_pool = torch.empty_like(ks)
    ks_pool.view(n_pages, 64)[table.long()] = ks.view(n_pages, 64)
    pws = torch.empty(lt.lt_indexer_topk_paged_workspace_bytes(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk),
                      dtype=torch.uint8, device="cuda")
    p_idx = torch.empty_like(out_idx)

    def paged():
        lt.lt_indexer_topk_paged(inp.dtype, q, w, k_pool, ks_pool, table, inp.N, inp.topk, inp.causal_offset, p_idx, None, pws)

    def dense():
        lt.lt_indexer_topk_ex(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score, ws)

    paged()
    dense()
    d_ms, p_ms = _timed_ms(torch, dense, 3, flush), _timed_ms(torch, paged, 3, flush)
    res["paged_key_cache"] = {"workload": inp.name, "dense_ms": d_ms, "paged_ms": p_ms, "delta": p_ms / d_ms - 1.0,
                              "same_indices": bool(torch.equal(p_idx, out_idx))}
    del k_pool, ks_pool, pws, p_idx
    # ---- integer ops on the chunk's index matrix
    res.update(time_aux_ops(torch, lt, out_idx, inp, peaks["hbm_gbs"], peak_kind))
    # ---- previous-chunk sampler on two consecutive (shorter) chunks of the structured workload
    T = 1024
    both = make_config("hot_fp8", T=2 * T)
    n_prev = both.causal_offset + T
    prev = dataclasses.replace(both, q=both.q[:T], w=both.w[:T], k=both.k[:n_prev], k_scale=both.k_scale[:n_prev])
    cur = dataclasses.replace(both, q=both.q[T:], w=both.w[T:], causal_offset=both.causal_offset + T)
    pq, pw, pk, pks = lt.to_device(prev)
    cq, cw, ck, cks = lt.to_device(cur)
    idx1 = torch.empty((T, prev.topk), dtype=torch.int32, device="cuda")
    ws1 = lt.alloc_workspace(prev.dtype, T, prev.N, prev.H, prev.D, prev.topk)
    lt.lt_indexer_topk_ex(prev.dtype, pq, pw, pk, pks, prev.topk, prev.causal_offset, idx1, None, ws1)
    n_sample = min(3 * prev.topk, lt.LT_MAX_TOPK)
    sample = torch.empty(n_sample, dtype=torch.int32, device="cuda")
    fws = torch.empty(lt.lt_topk_frequent_workspace_bytes(prev.N), dtype=torch.uint8, device="cuda")
    lt.lt_topk_frequent(idx1, prev.N, sample, None, fws)
    idx2 = torch.empty((T, cur.topk), dtype=torch.int32, device="cuda")
    ws2 = lt.alloc_workspace(cur.dtype, T, cur.N, cur.H, cur.D, cur.topk)
    lt.lt_indexer_topk_ex(cur.dtype, cq, cw, ck, cks, cur.topk, cur.causal_offset, idx2, None, ws2)
    surv_default = lt.lt_read_status(ws2)[3] / T
    ws3 = torch.empty(lt.lt_indexer_topk_sampled_workspace_bytes(cur.dtype, T, cur.N, cur.H, cur.D, cur.topk, n_sample),
                      dtype=torch.uint8, device="cuda")
    idx3 = torch.empty_like(idx2)
    lt.lt_indexer_topk_sampled(cur.dtype, cq, cw, ck, cks, cur.topk, cur.causal_offset, sample, idx3, None, ws3)
    st3 = lt.lt_read_status(ws3)
    res["previous_chunk_sampler"] = {"workload": "hot_fp8, two chunks of 1024 rows", "n_sample": n_sample,
                                     "survivors_per_row": st3[3] / T, "survivors_per_row_default_sampler": surv_default,
                                     "fallback_rows": st3[1], "same_indices": bool(torch.equal(idx2, idx3))}
    del pq, pw, pk, pks, cq, cw, ck, cks, ws1, ws2, ws3, fws
    # ---- k-NN variant: 64 queries x 2^20 x 768 bf16, unit vectors around 64 centres, generated on the device with
    # the recipe of the CPU generator (the parity tests use the CPU generator; this line only times)
    Tq, Nc, Dk, kk = 64, 1 << 20, 768, 1024
    g = torch.Generator(device="cuda")
    g.manual_seed(20)
    centres = torch.nn.functional.normalize(torch.randn(64, Dk, device="cuda", generator=g), dim=1)

    def draw(rows):
        which = torch.randint(0, 64, (rows,), device="cuda", generator=g)
        out = torch.empty((rows, Dk), dtype=torch.bfloat16, device="cuda")
        for r0 in range(0, rows, 1 << 17):
            r1 = min(rows, r0 + (1 << 17))
            v = 0.7 * centres[which[r0:r1]] + torch.randn(r1 - r0, Dk, device="cuda", generator=g) / Dk ** 0.5
            out[r0:r1] = torch.nn.functional.normalize(v, dim=1).to(torch.bfloat16)
        return out

    xq, xc = draw(Tq), draw(Nc)
    kidx = torch.empty((Tq, kk), dtype=torch.int32, device="cuda")
    kws = torch.empty(lt.lt_knn_topk_workspace_bytes(Tq, Nc, Dk, kk), dtype=torch.uint8, device="cuda")

    def knn():
        lt.lt_knn_topk(xq, xc, kk, kidx, None, kws)

    for _ in range(3):
        knn()
    ph = []
    kms = 0.0
    for _ in range(10):
        kms += _timed_ms(torch, knn, 1, flush)
        ph.append(lt.lt_read_phase_ms())
    kms /= 10
    kst = lt.lt_read_status(kws)
    scan_ms = statistics.mean(p[2] for p in ph)
    nbytes = Nc * Dk * 2 + Tq * Dk * 2 + kst[3] * 8
    res["knn"] = {"T": Tq, "N": Nc, "D": Dk, "topk": kk, "ms_per_step": kms, "pairs_per_s": Tq * Nc / (kms * 1e-3),
                  "scan_ms": scan_ms, "fallback_rows": kst[1],
                  "roofline": {"bound": "hbm", "achieved": nbytes / scan_ms / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": nbytes / scan_ms / 1e6 / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                               "algorithmic_bytes": nbytes}}
    return res


def run_knn(args, rank: int, local_rank: int, world: int):
    """k-NN (inner-product) variant: one step = exact top-k of a batch of queries over the whole corpus."""
    import torch
    import torch.distributed as dist

    from paper_2607_11976_b200 import binding as lt
    from paper_2607_11976_b200 import build as lt_build
    from workloads import make_knn

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    args.warmup = max(args.warmup, 3)
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        lt_build.build()
    if world > 1:
        dist.barrier()
    lt.load()
    inp = make_knn(args.workload, N=args.knn_corpus or None)
    pairs = inp.valid_pairs()
    q = torch.from_numpy(inp.q.view("int16")).cuda().view(torch.bfloat16)
    x = torch.from_numpy(inp.x.view("int16")).cuda().view(torch.bfloat16)
    out_idx = torch.empty((inp.T, inp.topk), dtype=torch.int32, device="cuda")
    out_score = torch.empty((inp.T, inp.topk), dtype=torch.float32, device="cuda")
    ws = torch.empty(lt.lt_knn_topk_workspace_bytes(inp.T, inp.N, inp.D, inp.topk), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        lt.lt_knn_topk(q, x, inp.topk, out_idx, out_score, ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    lt.lt_set_profiling(True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    # a step lasts well under the clock sampler's period: keep the same load up for half a second (untimed) so
    # that the sampled clocks and throttle reasons describe the state the timed steps run in
    t_load = time.perf_counter()
    while time.perf_counter() - t_load < 0.5:
        step()
        torch.cuda.synchronize()
    status = lt.lt_read_status(ws)
    if status[0] & lt.LT_STATUS_TIMEOUT:
        raise SystemExit("device-side wait timed out; results invalid")
    barrier()
    launches0 = lt.lt_launch_count()
    step_ms, phase_ms = [], []
    for _ in range(args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        step()
        e1.record(stream)
        e1.synchronize()
        step_ms.append(e0.elapsed_time(e1))
        phase_ms.append(lt.lt_read_phase_ms())
    launches = lt.lt_launch_count() - launches0
    barrier()
    clocks = sampler.stop()
    total_ms = max_over_ranks(sum(step_ms), world, "cuda")
    ms_per_step = total_ms / args.steps
    value = aggregate_throughput(pairs, args.steps, total_ms, world)
    status = lt.lt_read_status(ws)

    host = [q.cpu().pin_memory(), x.cpu().pin_memory()]
    h_idx = torch.empty_like(out_idx, device="cpu").pin_memory()
    h_score = torch.empty_like(out_score, device="cpu").pin_memory()

    def e2e_step():
        q.copy_(host[0], non_blocking=True)
        x.copy_(host[1], non_blocking=True)
        step()
        h_idx.copy_(out_idx, non_blocking=True)
        h_score.copy_(out_score, non_blocking=True)

    e2e_step()
    barrier()
    e2e_steps = min(args.steps, 3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    e1.synchronize()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks, peak_kind = load_peaks()
    scan_ms = statistics.mean(p[2] for p in phase_ms)
    # algorithmic bytes of the scan: the corpus once per block of 64 queries, the queries, the survivors
    n_qblocks = -(-inp.T // 64)
    alg_bytes = n_qblocks * inp.N * inp.D * 2 + inp.T * inp.D * 2 + status[3] * 8
    achieved = alg_bytes / (scan_ms * 1e-3) / 1e9
    names = ["sample_scan", "sample_stats", "fused_scan", "final_select", "fallback"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "T": inp.T, "N": inp.N, "D": inp.D, "topk": inp.topk, "valid_pairs": pairs,
                   "parallelism": f"replicas x{world}", "l2": "inputs larger than L2 (corpus streamed once per step)",
                   "workspace_bytes": int(ws.numel())},
        "clocks": clocks,
        "e2e": {"value": aggregate_throughput(pairs, e2e_steps, e2e_ms, world), "unit": UNIT,
                "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in host),
                "d2h_bytes_per_step": h_idx.numel() * 4 + h_score.numel() * 4, "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "knn_scan_kernel (fused score + filter)", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                     "kernel_ms": scan_ms, "algorithmic_bytes": alg_bytes,
                     # dram__bytes_read.sum + dram__bytes_write.sum of one launch at the default shape
                     # (profiles/knn_scan_kernel_T64_N1M_D768.md)
                     "traffic": 1.613026e9 + 11.56e6 if (inp.T, inp.N, inp.D) == (64, 1 << 20, 768) else None},
        "phases_ms": {n: statistics.mean(p[i] for p in phase_ms) for i, n in enumerate(names)},
        "status": {"bits": status[0], "fallback_rows": status[1], "max_survivors_per_row": status[2],
                   "mean_survivors_per_row": status[3] / inp.T, "overflow_rows": status[4]},
    }
    if args.knn_sweep and world == 1:
        sweep = []
        sizes = [n for n in (1 << 20, 2 << 20, 4 << 20, 5 * 1000 * 1000) if n <= inp.N] or [inp.N]
        for n_sub in sizes:
            xs = x[:n_sub]
            for k_sub in (128, 1024, 4096, 8192):
                oi = torch.empty((inp.T, k_sub), dtype=torch.int32, device="cuda")
                ws2 = torch.empty(lt.lt_knn_topk_workspace_bytes(inp.T, n_sub, inp.D, k_sub), dtype=torch.uint8, device="cuda")
                for _ in range(3):
                    lt.lt_knn_topk(q, xs, k_sub, oi, None, ws2)
                torch.cuda.synchronize()
                ts, sc = [], []
                for _ in range(10):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    lt.lt_knn_topk(q, xs, k_sub, oi, None, ws2)
                    e1.record(stream)
                    e1.synchronize()
                    ts.append(e0.elapsed_time(e1))
                    sc.append(lt.lt_read_phase_ms()[2])
                st2 = lt.lt_read_status(ws2)
                sweep.append({"N": n_sub, "topk": k_sub, "ms_per_step": statistics.median(ts), "scan_ms": statistics.median(sc),
                              "scan_gbs": n_sub * inp.D * 2 / statistics.median(sc) / 1e6, "fallback_rows": st2[1],
                              "mean_survivors_per_row": st2[3] / inp.T})
                del ws2, oi
        line["sweep"] = sweep
    if not args.no_graph:
        line["graph_replay"] = time_graph_replay(torch, lt, step, None, max(args.steps, 20))
    if not args.no_cpu_baseline and world == 1:
        from oracle import knn_topk

        np.matmul(np.ones((64, 64)), np.ones((64, 64)))
        t0 = time.perf_counter()
        rows_done = 0
        for r in range(0, inp.T, 4):
            knn_topk(inp.q, inp.x, inp.topk, rows=list(range(r, min(inp.T, r + 4))))
            rows_done += min(inp.T, r + 4) - r
            if time.perf_counter() - t0 > args.cpu_budget:
                break
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": rows_done * inp.N / dt, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": f"{rows_done} query rows x the whole corpus ({rows_done * inp.N} pairs, {dt:.1f} s)"}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="fp8_1m")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=20.0, help="seconds of CPU work for the oracle baseline")
    ap.add_argument("--rows", type=int, default=0, help="profiling aid: shrink the chunk to this many query rows")
    ap.add_argument("--sampler", default="strided", choices=["strided", "prev_chunk"],
                    help="prev_chunk: the sample is the 3k most frequent top-k positions of the previous chunk "
                         "(computed untimed through lt_topk_frequent; paper Sec. 3.2 'Sampling')")
    ap.add_argument("--paged", action="store_true",
                    help="keep the keys in a paged cache (pages of 64 keys in random order) and call lt_indexer_topk_paged")
    ap.add_argument("--aux", action="store_true",
                    help="also time the auxiliary integer ops on this step's top-k result: lt_topk_frequent and "
                         "lt_dsa_union_mask (group 64); adds an 'aux' object to the JSON line")
    ap.add_argument("--knn-corpus", type=int, default=0, help="k-NN workloads: corpus size (default: the workload's)")
    ap.add_argument("--knn-sweep", action="store_true",
                    help="k-NN workloads: also time prefixes of the corpus (1M, 2M, 4M, ... vectors) x k in {128, 1024, 4096, 8192} "
                         "(the grid of the paper's retrieval benchmark) and add the table as 'sweep'")
    ap.add_argument("--path", default="default", choices=["default", "abs"],
                    help="abs: the alternative fp8 scan (LT_PATH_FUSED_ABS: |x| form of Eq. 1 with linear-term columns)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="default fp8_1m line only: skip the brief measurements of the other configurations and the next-row operations")
    ap.add_argument("--no-unfused", action="store_true")
    ap.add_argument("--graph", action="store_true", help="indexer workloads: also time the step replayed from a CUDA graph")
    ap.add_argument("--no-graph", action="store_true", help="k-NN workloads: skip the CUDA-graph replay of the step")
    ap.add_argument("--no-fp8-gemm", action="store_true", help="skip the library FP8 GEMM measured for roofline context")
    ap.add_argument("--unfused-budget-mb", type=int, default=2048, help="score-matrix budget of the unfused GPU baseline")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    if args.workload.startswith("knn"):
        run_knn(args, rank, local_rank, world)
        return

    import torch
    import torch.distributed as dist

    from paper_2607_11976_b200 import binding as lt
    from paper_2607_11976_b200 import build as lt_build
    from workloads import make_config

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    args.warmup = max(args.warmup, 3)
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        lt_build.build()
    if world > 1:
        dist.barrier()
    lt.load()

    inp = make_config(args.workload, T=args.rows) if args.rows else make_config(args.workload)
    sampler_info = None
    sample_idx = None
    if args.sampler == "prev_chunk":
        # two consecutive chunks of one context: the first one is run once, untimed, to produce the sample
        import dataclasses

        T = inp.T
        both = make_config(args.workload, T=2 * T)
        n_prev = both.causal_offset + T
        prev = dataclasses.replace(both, q=both.q[:T], w=both.w[:T], k=both.k[:n_prev],
                                   k_scale=None if both.k_scale is None else both.k_scale[:n_prev])
        inp = dataclasses.replace(both, q=both.q[T:], w=both.w[T:], causal_offset=both.causal_offset + T)
        pq, pw, pk, pks = lt.to_device(prev)
        p_idx = torch.empty((T, prev.topk), dtype=torch.int32, device="cuda")
        p_ws = lt.alloc_workspace(prev.dtype, T, prev.N, prev.H, prev.D, prev.topk)
        lt.lt_indexer_topk_ex(prev.dtype, pq, pw, pk, pks, prev.topk, prev.causal_offset, p_idx, None, p_ws)
        n_sample = min(3 * prev.topk, lt.LT_MAX_TOPK, prev.N)
        sample_idx = torch.empty(n_sample, dtype=torch.int32, device="cuda")
        f_ws = torch.empty(lt.lt_topk_frequent_workspace_bytes(prev.N), dtype=torch.uint8, device="cuda")
        lt.lt_topk_frequent(p_idx, prev.N, sample_idx, None, f_ws)
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(torch.cuda.current_stream())
        for _ in range(5):
            lt.lt_topk_frequent(p_idx, prev.N, sample_idx, None, f_ws)
        f1.record(torch.cuda.current_stream())
        f1.synchronize()
        sampler_info = {"kind": "prev_chunk", "n_sample": n_sample, "previous_chunk_rows": T,
                        "lt_topk_frequent_ms": f0.elapsed_time(f1) / 5, "timed_in_step": False}
        del pq, pw, pk, pks, p_ws, f_ws
    pairs = inp.valid_pairs()
    flops = 2.0 * inp.H * inp.D * pairs
    q, w, k, ks = lt.to_device(inp)
    out_idx = torch.empty((inp.T, inp.topk), dtype=torch.int32, device="cuda")
    out_score = torch.empty((inp.T, inp.topk), dtype=torch.float32, device="cuda")
    tun = lt.Tunables(path=lt.LT_PATH_FUSED_ABS) if args.path == "abs" else None
    if tun is not None and (args.paged or sample_idx is not None):
        raise SystemExit("--path abs is timed on the dense layout with the default sampler")
    if sample_idx is None:
        ws = lt.alloc_workspace(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk, tun)
    else:
        ws = torch.empty(lt.lt_indexer_topk_sampled_workspace_bytes(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk,
                                                                    sample_idx.numel()), dtype=torch.uint8, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")  # larger than the 126 MB L2
    stream = torch.cuda.current_stream()

    page_table = None
    if args.paged:
        if sample_idx is not None or inp.N % 64 != 0:
            raise SystemExit("--paged needs the default sampler and a context that is a multiple of 64 keys")
        n_pages = inp.N // 64
        gen = torch.Generator(device="cuda")
        gen.manual_seed(1234)
        page_table = torch.randperm(n_pages, device="cuda", generator=gen).to(torch.int32)
        k_pool = torch.empty_like(k)
        k_pool.view(n_pages, 64, inp.D)[page_table.long()] = k.view(n_pages, 64, inp.D)
        ks_pool = None
        if ks is not None:
            ks_pool = torch.empty_like(ks)
            ks_pool.view(n_pages, 64)[page_table.long()] = ks.view(n_pages, 64)
        k, ks = k_pool, ks_pool
        ws = torch.empty(lt.lt_indexer_topk_paged_workspace_bytes(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk),
                         dtype=torch.uint8, device="cuda")

    def step(src=None, dst=None):
        q_, w_, k_, ks_ = src if src is not None else (q, w, k, ks)
        idx_, score_ = dst if dst is not None else (out_idx, out_score)
        if page_table is not None:
            lt.lt_indexer_topk_paged(inp.dtype, q_, w_, k_, ks_, page_table, inp.N, inp.topk, inp.causal_offset, idx_, score_, ws)
        elif sample_idx is None:
            lt.lt_indexer_topk_ex(inp.dtype, q_, w_, k_, ks_, inp.topk, inp.causal_offset, idx_, score_, ws, tun)
        else:
            lt.lt_indexer_topk_sampled(inp.dtype, q_, w_, k_, ks_, inp.topk, inp.causal_offset, sample_idx, idx_, score_, ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    lt.lt_set_profiling(True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    status = lt.lt_read_status(ws)
    if status[0] & lt.LT_STATUS_TIMEOUT:
        raise SystemExit("device-side wait timed out; results invalid")
    barrier()
    launches0 = lt.lt_launch_count()
    step_ms, phase_ms = [], []
    for _ in range(args.steps):
        flush.fill_(1)  # evict L2 between timed iterations (untimed)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        step()
        e1.record(stream)
        e1.synchronize()
        step_ms.append(e0.elapsed_time(e1))
        phase_ms.append(lt.lt_read_phase_ms())
    launches = lt.lt_launch_count() - launches0
    barrier()
    clocks = sampler.stop()
    total_ms = max_over_ranks(sum(step_ms), world, "cuda")
    ms_per_step = total_ms / args.steps
    value = aggregate_throughput(pairs, args.steps, total_ms, world)
    status = lt.lt_read_status(ws)

    # ---- end to end through the public API with host buffers: H2D of the inputs, D2H of the result
    host = [t.cpu().pin_memory() for t in (q, w, k)] + ([ks.cpu().pin_memory()] if ks is not None else [])
    dev = [q, w, k] + ([ks] if ks is not None else [])
    h_idx = torch.empty_like(out_idx, device="cpu").pin_memory()
    h_score = torch.empty_like(out_score, device="cpu").pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host)
    d2h = h_idx.numel() * 4 + h_score.numel() * 4

    def e2e_step():
        for d, h in zip(dev, host):
            d.copy_(h, non_blocking=True)
        step()
        h_idx.copy_(out_idx, non_blocking=True)
        h_score.copy_(out_score, non_blocking=True)

    e2e_step()
    barrier()
    e2e_steps = min(args.steps, 20)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    e1.synchronize()
    e2e_serial_ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")

    # The same with the copies taken off the compute stream, as a serving loop would run it: two sets of device
    # input and output buffers, the H2D copy of step i + 1 and the D2H read of step i - 1 on side streams while
    # step i computes.  Every step still copies all of its inputs in and its results out inside the timed region.
    h2d_stream, d2h_stream = torch.cuda.Stream(), torch.cuda.Stream()
    dev2 = [dev, [torch.empty_like(t) for t in dev]]
    outs2 = [(out_idx, out_score), (torch.empty_like(out_idx), torch.empty_like(out_score))]
    h_outs2 = [(h_idx, h_score), (torch.empty_like(h_idx).pin_memory(), torch.empty_like(h_score).pin_memory())]

    def e2e_pipelined(n):
        copied = [torch.cuda.Event() for _ in range(n)]
        computed = [torch.cuda.Event() for _ in range(n)]
        read = [torch.cuda.Event() for _ in range(n)]
        for i in range(n):
            b = i & 1
            with torch.cuda.stream(h2d_stream):
                if i >= 2:
                    h2d_stream.wait_event(computed[i - 2])  # the step that last read this input set
                for d, h in zip(dev2[b], host):
                    d.copy_(h, non_blocking=True)
                copied[i].record(h2d_stream)
            stream.wait_event(copied[i])
            if i >= 2:
                stream.wait_event(read[i - 2])  # the read that last drained this output set
            src = tuple(dev2[b]) + ((None,) if ks is None else ())
            step(src, outs2[b])
            computed[i].record(stream)
            with torch.cuda.stream(d2h_stream):
                d2h_stream.wait_event(computed[i])
                h_outs2[b][0].copy_(outs2[b][0], non_blocking=True)
                h_outs2[b][1].copy_(outs2[b][1], non_blocking=True)
                read[i].record(d2h_stream)
        for ev in read[-2:]:
            stream.wait_event(ev)

    e2e_pipelined(2)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    h2d_stream.wait_event(e0)
    e2e_pipelined(e2e_steps)
    e1.record(stream)
    e1.synchronize()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
    e2e_value = aggregate_throughput(pairs, e2e_steps, e2e_ms, world)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_peaks()
    fp8 = inp.dtype == "e4m3"
    # measured dense peak for this dtype: the measured bf16 burst figure x the nominal fp8:bf16 ratio (2)
    peak_tflops = peaks["bf16_tflops"] * (2.0 if fp8 else 1.0)
    scan_ms = statistics.mean(p[2] for p in phase_ms)
    achieved = flops / (scan_ms * 1e-3) / 1e12
    roofline = {
        "bound": "tensor", "kernel": "scan_fp8_kernel (alternative |x| form)" if tun is not None else "scan_kernel (fused score + filter)",
        "achieved": achieved, "peak": peak_tflops,
        "unit": "TFLOP/s", "frac": achieved / peak_tflops, "peak_kind": f"of {peak_kind} (bf16 burst x {2 if fp8 else 1})",
        "frac_of_nominal": achieved / (NOMINAL_FP8_TFLOPS if fp8 else NOMINAL_BF16_TFLOPS),
        # context: the same kernel against the power-capped (seconds-long) cuBLAS figure; the timed loop of
        # this benchmark runs back to back and shows sw_power_cap on the large workloads
        "frac_of_sustained": achieved / (peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * (2.0 if fp8 else 1.0)),
        "flops_per_launch": flops, "kernel_ms": scan_ms,
        "traffic": (SCAN_TRAFFIC[args.workload]["fixed_bytes"] + SCAN_TRAFFIC[args.workload]["bytes_per_row"] * inp.T)
        if args.workload in SCAN_TRAFFIC else None,
        "algorithmic_bytes": algorithmic_bytes(inp),
    }
    names = ["sample_scan", "sample_stats", "fused_scan", "final_select", "fallback"]
    phases = {n: statistics.mean(p[i] for p in phase_ms) for i, n in enumerate(names)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "ms_per_step_median": statistics.median(step_ms), "ms_per_step_min": min(step_ms),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp8_e4m3" if fp8 else inp.dtype, "data": "synthetic",
        "config": {"workload": args.workload, "T": inp.T, "N": inp.N, "H": inp.H, "D": inp.D, "topk": inp.topk,
                   "causal_offset": inp.causal_offset, "valid_pairs": pairs, "parallelism": f"replicas x{world}",
                   "l2": "flushed between timed iterations (256 MiB write)", "workspace_bytes": int(ws.numel()),
                   "key_layout": "paged (64-key pages, random order)" if page_table is not None else "dense",
                   "path": args.path},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
                "how": "double-buffered: H2D of the next step and D2H of the previous one on side streams",
                "serial_ms_per_step": e2e_serial_ms / e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "phases_ms": phases,
        "tensor_tflops_whole_step": flops / (ms_per_step * 1e-3) / 1e12,
        "sampler": sampler_info or {"kind": "strided"},
        "status": {"bits": status[0], "fallback_rows": status[1], "max_survivors_per_row": status[2],
                   "mean_survivors_per_row": status[3] / inp.T, "overflow_rows": status[4]},
    }

    if fp8 and not args.no_fp8_gemm:
        g = measure_fp8_gemm(torch)
        if g and "burst_tflops" in g:
            g["frac_of_burst"] = achieved / g["burst_tflops"]
            g["frac_of_sustained"] = achieved / g["sustained_tflops"]
        roofline["fp8_gemm_measured"] = g
        if not args.no_extras:
            u = measure_umma_stream(torch, lt, local_rank)
            if "single" in u:
                u["frac_of_single"] = achieved / u["single"]["tflops"]
            roofline["fp8_umma_stream_measured"] = u

    if args.aux:
        line["aux"] = time_aux_ops(torch, lt, out_idx, inp, peaks["hbm_gbs"], peak_kind)

    default_line = (args.workload == "fp8_1m" and not args.rows and page_table is None and sample_idx is None and world == 1
                    and tun is None)
    if default_line and not args.no_extras:
        # the other four configurations and the "next" operations, a few timed steps each, in the same process
        del dev2, outs2, h_outs2, host
        line["configs"] = measure_other_configs(torch, lt, peaks, flush)
        line["next"] = measure_next_rows(torch, lt, peaks, peak_kind, flush, (inp, q, w, k, ks, out_idx, out_score, ws))

    if not args.no_unfused and page_table is None:
        # in-repo unfused GPU baseline: dense scores to HBM in row sub-chunks, then a full-row radix select
        buf = torch.empty(256 + (args.unfused_budget_mb << 20), dtype=torch.uint8, device="cuda")

        def unfused():
            lt.lt_unfused_topk(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score, buf)

        unfused()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        n_unf = 2
        for _ in range(n_unf):
            unfused()
        e1.record(stream)
        e1.synchronize()
        ums = e0.elapsed_time(e1) / n_unf
        line["unfused_gpu_baseline"] = {"value": pairs / (ums * 1e-3), "unit": UNIT, "ms_per_step": ums,
                                        "score_buffer_mb": args.unfused_budget_mb}
        del buf

    if args.graph:
        # off by default here: the step is one 39 ms kernel plus a few small ones, launch overhead is not what it
        # waits for, and a figure taken this late in the process runs at the lower clocks of a warmed-up GPU
        line["graph_replay"] = time_graph_replay(torch, lt, step, flush, min(args.steps, 10))

    if not args.no_cpu_baseline and world == 1:
        v, rows, npairs, dt = time_oracle(inp, budget_s=args.cpu_budget)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": f"{rows} evenly spaced rows x all visible keys ({npairs} pairs, {dt:.1f} s)"}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
