#!/usr/bin/env python
"""Benchmark of the BRACE ring aggregation on B200.

A step is one pass of the whole path over one batch of synthetic updates:
Byzantine injection into the update matrix, then one aggregation round
(sign quantisation, share-reduce, consensus, share-only) that leaves every
client with the packed aggregate.  Inputs are resident in HBM for `value`;
`e2e` repeats the step through the host-buffer entry point (pinned host memory,
copies inside the timed region).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

Prints one JSON line on rank 0.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2501_17392_b200 import workloads as W  # noqa: E402

METRIC = "aggregated update elements/s"
UNIT = "elements/s"
L2_BYTES = 126 * 1024 * 1024


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def replica_seed_round(rank: int) -> int:
    """Replicas draw different inputs: rank r uses round index 1000*r as its stream offset."""
    return 1000 * rank


def max_over_ranks(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, n: int, d: int, steps: int, total_ms: float) -> float:
    """Elements all replicas aggregated, divided by the slowest rank's time."""
    return world * n * d * steps / (total_ms * 1e-3)


def algorithmic_bytes_fused(n: int, d: int, entry_bytes: int) -> int:
    """Bytes the fused round must move: every update read once, the last two hops'
    partials written to the mailboxes, every client's packed row written once."""
    words = (d + 31) // 32
    hops_kept = 2 if n > 2 else 1
    return 4 * n * d + hops_kept * d * entry_bytes + 4 * n * words


# ----------------------------------------------------------------------------- CPU oracle timing
def oracle_sample_run(w, sample_d: int, round_idx: int = 0):
    """Time the CPU oracle (injection + hop-by-hop ring) on a coordinate slab of the workload."""
    from oracle import brace_oracle as O
    ws = W.scaled(w, sample_d, name=w.name)
    H = W.honest_updates(ws, round_idx, device="cpu").numpy()[:, :sample_d]
    noise, unif = W.attack_draws(ws, round_idx, device="cpu")
    noise = None if noise is None else noise.numpy()[:, :sample_d]
    unif = None if unif is None else unif.numpy()[:, :sample_d]
    t0 = time.perf_counter()
    U = O.inject_attack(w.attack, H, list(range(w.f)), scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob,
                        noise=noise, uniform=unif)
    tr = O.ring_round(U, lam=w.lam, keep_states=False)
    O.pack_bits_fast(tr.outputs[0])
    dt = time.perf_counter() - t0
    return dt, w.n * sample_d


def oracle_cores() -> int:
    # numpy element-wise kernels run on the calling thread
    return 1


def sample_dim(w, target_elements: float) -> int:
    d = int(min(w.d, max(1024, target_elements // w.n)))
    return d


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    sd = sample_dim(w, 3.0e8)
    for i in range(args.warmup):
        oracle_sample_run(w, max(1024, sd // 16), i)
    total_t, total_e = 0.0, 0
    for i in range(args.steps):
        dt, ne = oracle_sample_run(w, sd, i)
        total_t += dt
        total_e += ne
    value = total_e / total_t
    sample = f"coordinate slab of {sd} of {w.d} coordinates, all {w.n} clients, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32 sign-sums over f32 inputs", "data": "synthetic",
        "config": {"workload": w.name, "n": w.n, "f": w.f, "d": w.d, "lambda": w.lam, "sample_d": sd},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_cores(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- the CUDA arm
def run_cuda(args, w):
    from paper_2501_17392_b200 import brace as B
    from paper_2501_17392_b200 import build as brace_build

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the aggregation has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    if rank == 0:
        brace_build.build()
    if world > 1:
        dist.barrier()
    B.lib()

    n, f, d = w.n, w.f, w.d
    base_round = replica_seed_round(rank)
    H = W.honest_updates(w, base_round, device=device)
    noise, unif = W.attack_draws(w, base_round, device=device)
    U = H.clone()
    mode = {"fused": B.AGG_FUSED, "stepwise": B.AGG_STEPWISE, "auto": B.AGG_AUTO}[args.mode]
    ctx = B.Brace(n, f, d, B.default_params(lam=w.lam, agg_mode=mode), device=device)
    if args.variant or args.grid:
        ctx.set_tuning(args.variant, args.grid)
    out = ctx.new_output(device=device)
    atk = B.make_attack(w.attack, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob, noise=noise, uniform=unif)
    stream = torch.cuda.current_stream()
    input_bytes = 4 * n * w.ld
    flush = None
    if input_bytes < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)

    def step():
        ctx.inject_attack(atk, H, U, stream)
        ctx.aggregate(U, out, stream)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    torch.cuda.synchronize()
    for k in range(args.steps):
        if flush is not None:
            flush.fill_(k & 0xFF)
        ev[k][0].record(stream)
        ctx.inject_attack(atk, H, U, stream)
        ev[k][1].record(stream)
        ctx.aggregate(U, out, stream)
        ev[k][2].record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    step_ms = [ev[k][0].elapsed_time(ev[k][2]) for k in range(args.steps)]
    agg_ms = [ev[k][1].elapsed_time(ev[k][2]) for k in range(args.steps)]
    inj_ms = [ev[k][0].elapsed_time(ev[k][1]) for k in range(args.steps)]
    total_ms = max_over_ranks(float(sum(step_ms)), world, device)
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end: host buffers through the C ABI, copies inside the timed region
    e2e = None
    out_ref = out.clone()
    if not args.no_e2e:
        hH = torch.empty(H.shape, dtype=torch.float32, pin_memory=True)
        hH.copy_(H)
        h_noise = h_unif = None
        if noise is not None:
            h_noise = torch.empty(noise.shape, dtype=torch.float32, pin_memory=True)
            h_noise.copy_(noise)
        if unif is not None:
            h_unif = torch.empty(unif.shape, dtype=torch.float32, pin_memory=True)
            h_unif.copy_(unif)
        h_out = torch.empty(out.shape, dtype=out.dtype, pin_memory=True)
        atk_h = B.make_attack(w.attack, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob, noise=h_noise,
                              uniform=h_unif)
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        ctx.aggregate_host(atk_h, hH, h_out, U, out, noise, unif, stream)      # warm-up
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            ctx.aggregate_host(atk_h, hH, h_out, U, out, noise, unif, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(float(e0.elapsed_time(e1)), world, device)
        h2d = 4 * n * w.ld + (0 if noise is None else noise.numel() * 4) + (0 if unif is None else unif.numel() * 4)
        d2h = out.numel() * 4
        e2e = {"value": whole_job_value(world, n, d, e2e_steps, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps}
        same = bool(torch.equal(h_out.to(device), out_ref))
        e2e["matches_device_result"] = same
        del hH, h_noise, h_unif, h_out

    # ---- hop-by-hop launches for comparison (same final state, one launch per hop)
    stepwise = None
    if args.mode != "stepwise" and not args.no_stepwise and rank == 0:
        ctx_s = B.Brace(n, f, d, B.default_params(lam=w.lam, agg_mode=B.AGG_STEPWISE), device=device)
        out_s = ctx_s.new_output(device=device)
        for _ in range(2):
            ctx_s.aggregate(U, out_s, stream)
        torch.cuda.synchronize()
        reps = 3
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ts = []
        for _ in range(reps):
            if flush is not None:
                flush.fill_(1)
            a.record(stream)
            ctx_s.aggregate(U, out_s, stream)
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ms = float(np.median(ts))
        words = (d + 31) // 32
        b_ring = 4 * n * d + (n - 2) * d + (n - 1) * d + d + 4 * words + (n - 1) * 2 * 4 * words
        stepwise = {"ms_per_round": ms, "launches_per_round": 2 * (n - 1) + 1,
                    "elements_per_s": n * d / (ms * 1e-3), "algorithmic_gbs": b_ring / (ms * 1e-3) / 1e9,
                    "same_result": bool(torch.equal(out_s, out_ref))}
        # the same launches replayed from a CUDA graph (removes host launch cost; matters for short hops)
        try:
            side = torch.cuda.Stream(device=device)
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                ctx_s.aggregate(U, out_s)
            stream.wait_stream(side)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                ctx_s.aggregate(U, out_s)
            graph.replay()
            torch.cuda.synchronize()
            ts = []
            for _ in range(reps):
                if flush is not None:
                    flush.fill_(1)
                a.record(stream)
                graph.replay()
                b.record(stream)
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            gms = float(np.median(ts))
            stepwise["graph_ms_per_round"] = gms
            stepwise["graph_algorithmic_gbs"] = b_ring / (gms * 1e-3) / 1e9
            stepwise["graph_same_result"] = bool(torch.equal(out_s, out_ref))
            del graph
        except RuntimeError as exc:                  # capture unsupported: report, do not fail the bench
            stepwise["graph_error"] = str(exc)[:200]
        ctx_s.close()

    # ---- the step after the round (model update) and the plain-sum rule, timed on their own
    extras = None
    if not args.no_extras and rank == 0:
        extras = {}
        reps = 3
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def timed(fn):
            ts = []
            for _ in range(reps):
                if flush is not None:
                    flush.fill_(2)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            return float(np.median(ts))

        weights = torch.zeros((n, w.ld), dtype=torch.float32, device=device)
        ctx.aggregate(U, out, stream)
        ctx.apply_update(out, weights, 0.01, stream)
        ms = timed(lambda: ctx.apply_update(out, weights, 0.01, stream))
        alg = 8 * n * d + 4 * n * ((d + 31) // 32)
        extras["model_update"] = {"ms": ms, "algorithmic_gbs": alg / (ms * 1e-3) / 1e9, "elements_per_s": n * d / (ms * 1e-3)}
        del weights
        ctx_sum = B.Brace(n, f, d, B.default_params(rule=B.RULE_SUM, agg_mode=B.AGG_FUSED), device=device)
        out_sum = ctx_sum.new_output(device=device)
        ctx_sum.aggregate(U, out_sum, stream)
        ms = timed(lambda: ctx_sum.aggregate(U, out_sum, stream))
        alg = 8 * n * d + 2 * 4 * d
        extras["sum_rule_fused"] = {"ms": ms, "algorithmic_gbs": alg / (ms * 1e-3) / 1e9, "elements_per_s": n * d / (ms * 1e-3)}
        ctx_sum.close()
        del out_sum
        torch.cuda.empty_cache()
        if n <= 128:
            # coordinate-wise median / trimmed mean: arithmetic-bound (bitonic network of min/max pairs on the
            # ALU pipe: 64 lanes per clock per SM, 148 SMs, at the maximum SM clock of the peaks file)
            res = torch.empty(d, dtype=torch.float32, device=device)
            npad = 4
            while npad < n:
                npad *= 2
            lg = npad.bit_length() - 1
            alu_ops = 2 * (npad * lg * (lg + 1) // 4)                    # min + max per compare-exchange
            peaks_now, _ = measured_peaks()
            alu_peak = 148 * 64 * peaks_now.get("sm_max_mhz", 1965.0) * 1e6
            for label, kind, trim in (("median", B.STAT_MEDIAN, 0), ("trimmed_mean", B.STAT_TRIMMED_MEAN, f)):
                ctx.coordinate_stat(kind, trim, U, res, stream)
                ms = timed(lambda: ctx.coordinate_stat(kind, trim, U, res, stream))
                extras["coordinate_" + label] = {
                    "ms": ms, "elements_per_s": n * d / (ms * 1e-3), "bound": "alu",
                    "alu_ops_per_coordinate": alu_ops, "achieved_ops_per_s": alu_ops * d / (ms * 1e-3),
                    "peak_ops_per_s": alu_peak, "frac": alu_ops * d / (ms * 1e-3) / alu_peak,
                    "hbm_gbs": (4 * n * d + 4 * d) / (ms * 1e-3) / 1e9}
            del res

    if rank != 0:
        # replicas have nothing to report; leave together with rank 0 so that no rank tears the
        # process group down while another still holds it
        ctx.close()
        dist.barrier()
        dist.destroy_process_group()
        return
    peaks, peak_kind = measured_peaks()
    entry_bytes = 1 if n <= 127 else 2
    fused_used = (args.mode != "stepwise")
    agg_avg_ms = float(np.mean(agg_ms))
    inj_avg_ms = float(np.mean(inj_ms))
    words = (d + 31) // 32
    if fused_used:
        agg_alg = algorithmic_bytes_fused(n, d, entry_bytes)
        spread = n * d >= (1 << 27)                 # the library adds one share-only launch on large problems
        agg_kernel = "fused_sign_kernel + ag_all_bits_kernel" if spread else "fused_sign_kernel"
        agg_alg += 4 * words if spread else 0       # the owners' rows are read back once
        launches_per_step = 3 if spread else 2
    else:
        agg_alg = 4 * n * d + (n - 2) * d + (n - 1) * d + d + 4 * words + (n - 1) * 2 * 4 * words
        agg_kernel = "rs_step_sign_kernel x(n-1) + consensus_sign_kernel + ag_step_bits_kernel x(n-1)"
        launches_per_step = 1 + 2 * (n - 1) + 1
    inj_alg, inj_kernel = injection_bytes(w)

    def roof(kernel, alg, ms, traffic_key):
        achieved = alg / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"{peak_kind} device copy",
                "algorithmic_bytes_per_launch": alg, "ms_per_launch": ms,
                "traffic": TRAFFIC_BYTES.get((w.name, traffic_key)) if not args.d else None}

    roof_agg = roof(agg_kernel, agg_alg, agg_avg_ms, "aggregate")
    roof_inj = roof(inj_kernel, inj_alg, inj_avg_ms, "inject")
    # the roofline entry is the kernel that takes the larger share of the step
    roofline = roof_inj if inj_avg_ms > agg_avg_ms else roof_agg
    roofline["other_kernel"] = roof_agg if roofline is roof_inj else roof_inj

    cpu_baseline = None
    if not args.no_cpu:
        sd = sample_dim(w, 3.0e8)
        oracle_sample_run(w, max(1024, sd // 16))
        slabs, tot_t, tot_e = 4, 0.0, 0
        for i in range(slabs):                       # fresh draws per slab; about 10 s of CPU work in all
            dt, ne = oracle_sample_run(w, sd, round_idx=i)
            tot_t += dt
            tot_e += ne
        cpu_baseline = {"value": tot_e / tot_t, "unit": UNIT, "cores": oracle_cores(), "kind": "oracle",
                        "sample": f"{slabs} coordinate slabs of {sd} of {d} coordinates, all {n} clients, one step "
                                  f"each ({tot_t:.1f} s in all)"}

    line = {
        "metric": METRIC, "value": whole_job_value(world, n, d, args.steps, total_ms), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32 sign-sums over f32 inputs", "data": "synthetic",
        "config": {"workload": w.name, "n": n, "f": f, "d": d, "lambda": w.lam, "rounds_per_step": 1,
                   "attack_kind": w.attack, "aggregate_mode": args.mode,
                   "l2": "flushed between steps" if flush is not None else "inputs larger than L2",
                   "replicas": world, "parallelism": "replicas only"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "phases_ms": {"inject": inj_avg_ms, "aggregate": agg_avg_ms},
        "aggregate_only_elements_per_s": n * d / (agg_avg_ms * 1e-3),
        "stepwise": stepwise, "extras": extras,
    }
    print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def injection_bytes(w):
    """(algorithmic bytes, kernel name) of one injection launch."""
    n, f, d = w.n, w.f, w.d
    if w.attack == W.ATTACK_SCALE_OWN:
        return 8 * f * d, "inject_elementwise_vec_kernel"
    if w.attack == W.ATTACK_GAUSSIAN:
        return 8 * f * d, "inject_elementwise_vec_kernel"
    if w.attack == W.ATTACK_SPARSE_NOISE:
        return 12 * f * d, "inject_elementwise_vec_kernel"
    if w.attack == W.ATTACK_SCALED_MEAN:
        return 4 * (n - f) * d + 4 * f * d, "inject_stats_smem_kernel"
    return 4 * (n - f) * d + 4 * f * d, "inject_stats_reg_kernel"


# DRAM bytes (read + write) per launch from ncu captures of the full-size workload
# (profiles/), keyed by (workload, phase); absent where no capture of the current kernel exists.
TRAFFIC_BYTES: dict = {
    ("cfg4", "aggregate"): 10_222_916_000 + 45_473_000 + 3_302_000 + 254_037_000,   # fused_sign_kernel<int8,1,8> + ag_all_bits_kernel, profiles/fused_sign_kernel_cfg4.md
    ("cfg4", "inject"): 8_178_365_000 + 1_988_146_000,     # inject_stats_reg_kernel<80>, profiles/inject_stats_reg_kernel_cfg4.md
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(W.WORKLOADS))
    ap.add_argument("--mode", default="fused", choices=["fused", "stepwise", "auto"])
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--grid", type=int, default=0)
    ap.add_argument("--d", type=int, default=0, help="override the workload's vector length (profiling on a small case)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-stepwise", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "cuda":
        args.warmup = 3
    w = W.WORKLOADS[args.workload]
    if args.d:
        w = W.scaled(w, args.d)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_cuda(args, w)


if __name__ == "__main__":
    main()
