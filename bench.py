#!/usr/bin/env python
"""Benchmark of the BRACE ring aggregation on B200.

A step is one pass of the whole path over one batch of synthetic updates:
Byzantine injection into the update matrix, then one aggregation round
(sign quantisation, share-reduce, consensus, share-only) that leaves every
client with the packed aggregate.  Inputs are resident in HBM for `value`;
`e2e` repeats the step through the host-buffer entry point (pinned host memory,
copies inside the timed region).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

Prints one JSON line on rank 0.  The headline numbers are those of --workload
(default cfg4); `per_config` carries the same measurements for all five
workloads.
"""

from __future__ import annotations

import argparse
import json
import multiprocessing as mp
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
DTYPE = "int32 sign-sums over f32 inputs"
ALL_WORKLOADS = ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5")

# DRAM bytes (read + write) per aggregated element, from ncu captures of the current kernels on a
# small case (n = 100, f = 20, d = 4,000,000; two DRAM counters, one kernel per capture): a full
# launch moves this many bytes per element times n * d (traffic grows with n * d: every element is
# read once).  None where the kernel has changed since its counters were taken.
TRAFFIC_BYTES_PER_ELEMENT: dict = {
    ("cfg4", "aggregate"): 4.0196,   # fused_sign_kernel<int8,1,8,256> 1.60003 GB read + 7.27 MB written, ag_all_bits_kernel 0.53 MB
    ("cfg4", "inject"): 3.8583,      # inject_stats_reg_kernel<80,3,strided> 1.28007 GB read + 263.2 MB written (rest still in L2)
}


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run."""

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
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def mark(self) -> int:
        """Index of the next sample: two marks bracket a region of interest."""
        return len(self.lines)

    def summary(self, lo: int = 0, hi: int | None = None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines[lo:hi]:
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

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()


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


def entry_bytes_of(n: int) -> int:
    return 1 if n <= 127 else 2


def algorithmic_bytes_fused(n: int, d: int) -> int:
    """Bytes the fused round must move: every update read once, the last two hops'
    partials written to the mailboxes, every client's packed row written once; on large
    problems the owners' rows are read back once by the share-only launch."""
    words = (d + 31) // 32
    hops_kept = 2 if n > 2 else 1
    spread = n * d >= (1 << 27)
    return 4 * n * d + hops_kept * d * entry_bytes_of(n) + 4 * n * words + (4 * words if spread else 0)


def algorithmic_bytes_ring(n: int, d: int) -> int:
    """Bytes of the hop-by-hop schedule: updates read once (sign fused into the read), mailboxes
    written and re-read every hop, consensus to packed bits, 1-bit share-only hops."""
    words = (d + 31) // 32
    p = entry_bytes_of(n)
    return 4 * n * d + (n - 2) * d * p + (n - 1) * d * p + d * p + 4 * words + (n - 1) * 2 * 4 * words


def injection_bytes(w, generated: bool):
    """(algorithmic bytes, kernel name) of one injection launch."""
    n, f, d = w.n, w.f, w.d
    if w.attack == W.ATTACK_SCALE_OWN:
        return 8 * f * d, "inject_elementwise_vec_kernel"
    if w.attack == W.ATTACK_GAUSSIAN:
        return (4 * f * d, "inject_generated_kernel") if generated else (8 * f * d, "inject_elementwise_vec_kernel")
    if w.attack == W.ATTACK_SPARSE_NOISE:
        return (4 * f * d, "inject_generated_kernel") if generated else (12 * f * d, "inject_elementwise_vec_kernel")
    if w.attack == W.ATTACK_SCALED_MEAN:
        return 4 * (n - f) * d + 4 * f * d, "inject_stats_smem_kernel"
    return 4 * (n - f) * d + 4 * f * d, "inject_stats_reg_kernel"


def sort_network_pairs(n: int, outputs=None) -> int:
    """Compare-exchanges per coordinate of the library's sorting network for n values: Batcher's
    odd-even merge sort for the next power of two, restricted to indices below n rounded up to a
    multiple of 8 (4 for n <= 4).  With `outputs` (sorted positions that are read afterwards) only the
    comparators those positions depend on are counted -- the rest is dead code the compiler removes."""
    nb = 4 if n <= 4 else (n + 7) // 8 * 8
    npow = 1
    while npow < nb:
        npow *= 2
    net, p = [], 1
    while p < npow:
        k = p
        while k >= 1:
            first = k % p
            for i in range(nb):
                hi = i + k
                if i >= first and ((i - first) % (2 * k)) < k and hi < nb and i // (2 * p) == hi // (2 * p):
                    net.append((i, hi))
            k //= 2
        p *= 2
    if outputs is None:
        return len(net)
    live, needed = set(outputs), 0
    for i, hi in reversed(net):
        if i in live or hi in live:
            needed += 1
            live.update((i, hi))
    return needed


def median_positions(n: int):
    """Sorted positions the library's median kernel may read for this n (its bucket's candidates)."""
    nb = 4 if n <= 4 else (n + 7) // 8 * 8
    return range((nb - 8) // 2 if nb > 8 else 0, min(nb // 2, nb - 1) + 1)


def attack_seed(w) -> int:
    return W.BASE_SEED + sum(ord(ch) for ch in w.name.split("_")[0])


def uses_draws(w) -> bool:
    return w.attack in (W.ATTACK_GAUSSIAN, W.ATTACK_SPARSE_NOISE)


# ----------------------------------------------------------------------------- CPU oracle timing
def oracle_inputs(w, sample_d: int, round_idx: int):
    ws = W.scaled(w, sample_d, name=w.name)
    return W.honest_updates(ws, round_idx, device="cpu").numpy()[:, :sample_d]


def oracle_step(w, H: np.ndarray, round_idx: int) -> float:
    """One step of the oracle as it stands: draws (where the attack consumes them), injection,
    hop-by-hop ring, packing of one client's result.  Returns seconds."""
    from oracle import brace_oracle as O
    sample_d = H.shape[1]
    t0 = time.perf_counter()
    noise = unif = None
    if uses_draws(w):
        noise, unif = O.attack_draws(w.attack, attack_seed(w), round_idx, list(range(w.f)), sample_d)
    U = O.inject_attack(w.attack, H, list(range(w.f)), scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob,
                        noise=noise, uniform=unif)
    tr = O.ring_round(U, lam=w.lam, keep_states=False)
    O.pack_bits_fast(tr.outputs[0])
    return time.perf_counter() - t0


def _oracle_worker(w, H, idx, barrier, queue):
    # runs in a forked child: numpy only (the inputs were drawn by the parent before the fork)
    oracle_step(w, H[:, : max(1024, H.shape[1] // 16)], 0)     # warm numpy up
    barrier.wait(timeout=120)
    t0 = time.perf_counter()
    oracle_step(w, H, 100 + idx)
    queue.put((t0, time.perf_counter(), w.n * H.shape[1]))


def sample_dim(w, target_elements: float) -> int:
    return int(min(w.d, max(1024, target_elements // w.n)))


def cpu_baseline_legs(w):
    """The oracle on the host: one core, then one process per core of the affinity mask, each on
    its own coordinate slab (Eq. (1) is per coordinate, so slabs are independent problems).
    Must run before this process touches CUDA or starts a thread pool: the second leg forks."""
    threads_before = torch.get_num_threads()
    torch.set_num_threads(1)                         # no thread pool in this process before it forks
    sd = sample_dim(w, 3.0e8)
    oracle_step(w, oracle_inputs(w, max(1024, sd // 16), 0), 0)
    slabs, tot_t, tot_e = 3, 0.0, 0
    for i in range(slabs):
        H = oracle_inputs(w, sd, i)
        tot_t += oracle_step(w, H, i)
        tot_e += w.n * sd
    one = {"value": tot_e / tot_t, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"{slabs} coordinate slabs of {sd} of {w.d} coordinates, all {w.n} clients, one step each "
                     f"({tot_t:.1f} s in all)"}
    cores = len(os.sched_getaffinity(0))
    workers = max(1, min(cores, 64))
    sd_all = int(min(sd, max(4096, 6.0e9 // (workers * w.n * 4 * 4))))     # bounded host memory
    inputs = [oracle_inputs(w, sd_all, 100 + i) for i in range(workers)]
    ctx = mp.get_context("fork")
    barrier, queue = ctx.Barrier(workers), ctx.Queue()
    procs = [ctx.Process(target=_oracle_worker, args=(w, inputs[i], i, barrier, queue), daemon=True)
             for i in range(workers)]
    for p in procs:
        p.start()
    try:
        res = [queue.get(timeout=240) for _ in procs]
        wall = max(r[1] for r in res) - min(r[0] for r in res)
        one["all_cores"] = {"value": sum(r[2] for r in res) / wall, "unit": UNIT, "cores": workers,
                            "cores_in_affinity_mask": cores,
                            "sample": f"{workers} processes, one coordinate slab of {sd_all} coordinates each, all "
                                      f"{w.n} clients, one step each ({wall:.1f} s wall)"}
    except Exception as exc:                         # a worker died or never answered: report, do not hang
        one["all_cores"] = {"value": None, "cores": workers, "error": repr(exc)[:200]}
    for p in procs:
        p.join(timeout=5)
        if p.is_alive():
            p.terminate()
    del inputs
    torch.set_num_threads(threads_before)
    return one


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    sd = sample_dim(w, 3.0e8)
    for i in range(min(args.warmup, 2)):
        oracle_step(w, oracle_inputs(w, max(1024, sd // 16), i), i)
    total_t, total_e = 0.0, 0
    for i in range(args.steps):
        H = oracle_inputs(w, sd, i)
        total_t += oracle_step(w, H, i)
        total_e += w.n * sd
    value = total_e / total_t
    sample = f"coordinate slab of {sd} of {w.d} coordinates, all {w.n} clients, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": w.name, "n": w.n, "f": w.f, "d": w.d, "lambda": w.lam, "sample_d": sd},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- one workload on the GPU
class Timer:
    def __init__(self, stream, flush):
        self.stream, self.flush = stream, flush
        self.a, self.b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def median_ms(self, fn, reps: int) -> float:
        ts = []
        for r in range(reps):
            if self.flush is not None:
                self.flush.fill_(r & 0xFF)
            self.a.record(self.stream)
            fn()
            self.b.record(self.stream)
            torch.cuda.synchronize()
            ts.append(self.a.elapsed_time(self.b))
        return float(np.median(ts))


def sampled_oracle_check(w, U: torch.Tensor, out: torch.Tensor, seed: int = 0) -> bool:
    """Eq. (1) by the oracle on sampled columns of the matrix the round consumed, against row 0 of the
    result; every other client's row must equal row 0."""
    from oracle import brace_oracle as O
    d, n = w.d, w.n
    rng = np.random.default_rng(seed + n)
    idx_np = np.unique(np.concatenate([np.arange(0, min(d, 1024)), np.arange(max(0, d - 1024), d),
                                       rng.integers(0, d, size=16384)])).astype(np.int64)
    idx = torch.as_tensor(idx_np, device=U.device)
    cols = U[:, idx].cpu().numpy()
    exp = O.gar_direct(cols, w.lam) > 0
    words = out[0][idx // 32].to(torch.int64) & 0xFFFFFFFF
    got = ((words >> (idx % 32)) & 1).cpu().numpy().astype(bool)
    nwords = (d + 31) // 32
    same_rows = all(bool(torch.equal(out[c, :nwords], out[0, :nwords])) for c in range(1, n))
    return bool(np.array_equal(got, exp)) and same_rows


def measure_workload(B, w, args, device, stream, world, rank, sampler):
    """All device-side measurements of one workload.  Returns (results, live buffers or None)."""
    n, f, d = w.n, w.f, w.d
    peaks, peak_kind = measured_peaks()
    base_round = replica_seed_round(rank)
    H = W.honest_updates(w, base_round, device=device)
    U = H.clone()
    generated = uses_draws(w) and not args.supplied_draws
    noise = unif = None
    if uses_draws(w) and not generated:
        noise, unif = W.attack_draws(w, base_round, device=device)
    mode = {"fused": B.AGG_FUSED, "stepwise": B.AGG_STEPWISE, "auto": B.AGG_AUTO}[args.mode]
    ctx = B.Brace(n, f, d, B.default_params(lam=w.lam, agg_mode=mode), device=device)
    if args.variant or args.grid:
        ctx.set_tuning(args.variant, args.grid)
    out = ctx.new_output(device=device)
    rounds = w.rounds

    def attack_for(r):
        return B.make_attack(w.attack, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob, noise=noise,
                             uniform=unif, seed=attack_seed(w) if generated else None, round_idx=base_round + r)

    atks = [attack_for(r) for r in range(rounds)]
    flush = None
    if 4 * n * w.ld < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)

    steps = args.steps
    for _ in range(args.warmup):
        for r in range(rounds):
            ctx.inject_attack(atks[r], H, U, stream)
            ctx.aggregate(U, out, stream)
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(rounds)] for _ in range(steps)]
    lo = sampler.mark() if sampler else 0
    torch.cuda.synchronize()
    for k in range(steps):
        for r in range(rounds):
            if flush is not None:
                flush.fill_(k & 0xFF)
            ev[k][r][0].record(stream)
            ctx.inject_attack(atks[r], H, U, stream)
            ev[k][r][1].record(stream)
            ctx.aggregate(U, out, stream)
            ev[k][r][2].record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    step_ms = [sum(ev[k][r][0].elapsed_time(ev[k][r][2]) for r in range(rounds)) for k in range(steps)]
    inj_ms = [ev[k][r][0].elapsed_time(ev[k][r][1]) for k in range(steps) for r in range(rounds)]
    agg_ms = [ev[k][r][1].elapsed_time(ev[k][r][2]) for k in range(steps) for r in range(rounds)]
    res = {
        "n": n, "f": f, "d": d, "lambda": w.lam, "rounds_per_step": rounds, "attack_kind": w.attack,
        "draws": "generated in the kernel" if generated else ("supplied matrices" if uses_draws(w) else "none"),
        "steps": steps, "l2": "flushed between rounds" if flush is not None else "inputs larger than L2",
        "step_ms_median": max_over_ranks(float(np.median(step_ms)), world, device),
        "step_ms_mean": max_over_ranks(float(np.mean(step_ms)), world, device),
        "inject_ms": float(np.median(inj_ms)), "round_ms": float(np.median(agg_ms)),
    }
    res["elements_per_s"] = world * rounds * n * d / (res["step_ms_median"] * 1e-3)
    res["round_only_elements_per_s"] = n * d / (res["round_ms"] * 1e-3)
    if sampler:
        time.sleep(0.12)                              # let the sampler see the end of the region
        res["clocks"] = sampler.summary(lo, sampler.mark())
    live = {"H": H, "U": U, "out": out, "ctx": ctx, "noise": noise, "unif": unif, "generated": generated,
            "round0": base_round}
    if rank != 0:
        return res, live

    fused_used = args.mode != "stepwise"
    peak = peaks["hbm_gbs"]

    def roof(kernel, alg, ms, key):
        achieved = alg / (ms * 1e-3) / 1e9
        per_el = TRAFFIC_BYTES_PER_ELEMENT.get((w.name, key)) if not args.d else None
        return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"{peak_kind} device copy",
                "algorithmic_bytes_per_launch": alg, "ms_per_launch": ms,
                "traffic": None if per_el is None else int(per_el * n * d)}

    if fused_used:
        spread = n * d >= (1 << 27)                 # the library adds one share-only launch on large problems
        agg_kernel = "fused_sign_kernel + ag_all_bits_kernel" if spread else "fused_sign_kernel"
        agg_alg = algorithmic_bytes_fused(n, d)
        launches_per_round = 3 if spread else 2
    else:
        agg_kernel = "rs_step_sign_kernel x(n-1) + consensus_sign_kernel + ag_step_bits_kernel x(n-1)"
        agg_alg = algorithmic_bytes_ring(n, d)
        launches_per_round = 1 + 2 * (n - 1) + 1
    inj_alg, inj_kernel = injection_bytes(w, generated)
    res["gpu_launches_per_step"] = launches_per_round * rounds
    res["roofline_round"] = roof(agg_kernel, agg_alg, res["round_ms"], "aggregate")
    res["roofline_inject"] = roof(inj_kernel, inj_alg, res["inject_ms"], "inject")
    if generated:
        res["roofline_inject"]["note"] = ("arithmetic-bound, not HBM-bound: the kernel draws its random numbers "
                                          "(Philox4x32-10, Box-Muller) and only writes the Byzantine rows")
    res["frac_of_nominal_8tbs"] = {"round": res["roofline_round"]["achieved"] / 8000.0,
                                   "inject": res["roofline_inject"]["achieved"] / 8000.0}

    # parity flag: the oracle's Eq. (1) on sampled columns of the matrix the last round consumed
    res["same_result"] = sampled_oracle_check(w, U, out)
    out_ref = out.clone()
    timer = Timer(stream, flush)

    # hop-by-hop launches (same final state, one launch per hop), eager and replayed from a CUDA graph
    if fused_used and not args.no_stepwise:
        ctx_s = B.Brace(n, f, d, B.default_params(lam=w.lam, agg_mode=B.AGG_STEPWISE), device=device)
        out_s = ctx_s.new_output(device=device)
        for _ in range(2):
            ctx_s.aggregate(U, out_s, stream)
        torch.cuda.synchronize()
        ms = timer.median_ms(lambda: ctx_s.aggregate(U, out_s, stream), 5)
        b_ring = algorithmic_bytes_ring(n, d)
        launches = 2 * (n - 1) + 1
        sw = {"ms_per_round": ms, "launches_per_round": launches, "us_per_launch": 1e3 * ms / launches,
              "elements_per_s": n * d / (ms * 1e-3), "algorithmic_bytes": b_ring,
              "algorithmic_gbs": b_ring / (ms * 1e-3) / 1e9, "frac": b_ring / (ms * 1e-3) / 1e9 / peak,
              "same_result": bool(torch.equal(out_s, out_ref))}
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
            gms = timer.median_ms(graph.replay, 5)
            sw["graph_ms_per_round"] = gms
            sw["graph_algorithmic_gbs"] = b_ring / (gms * 1e-3) / 1e9
            sw["graph_frac"] = sw["graph_algorithmic_gbs"] / peak
            sw["graph_same_result"] = bool(torch.equal(out_s, out_ref))
            del graph
        except RuntimeError as exc:                  # capture unsupported: report, do not fail the bench
            sw["graph_error"] = str(exc)[:200]
        res["stepwise"] = sw
        ctx_s.close()
        del out_s

    # small problems: many rounds enqueued back to back between one event pair (launch cost amortised;
    # the inputs stay in L2 where they fit, so this is a latency figure, not an HBM one)
    if fused_used and 4 * n * w.ld < 2 * L2_BYTES:
        k_rounds = 100
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ts = []
        for _ in range(3):
            a.record(stream)
            for _ in range(k_rounds):
                ctx.aggregate(U, out, stream)
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / k_rounds)
        ms = float(np.median(ts))
        res["back_to_back"] = {"rounds": k_rounds, "ms_per_round": ms, "elements_per_s": n * d / (ms * 1e-3),
                               "algorithmic_gbs": agg_alg / (ms * 1e-3) / 1e9, "l2": "not flushed"}

    live["out_ref"] = out_ref
    live["timer"] = timer
    return res, live


def e2e_leg(B, w, args, device, stream, world, live):
    """The step through the host-buffer entry point, copies inside the timed region; every rank runs it."""
    n, f, d = w.n, w.f, w.d
    H, U, out, ctx = live["H"], live["U"], live["out"], live["ctx"]
    noise, unif, generated = live["noise"], live["unif"], live["generated"]
    e2e = None
    if not args.no_e2e:
        ctx.aggregate(U, out, stream)
        out_ref = out.clone()
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
                              uniform=h_unif, seed=attack_seed(w) if generated else None,
                              round_idx=live["round0"] + w.rounds - 1)
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        ctx.aggregate_host(atk_h, hH, h_out, U, out, noise, unif, stream)      # warm-up
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
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
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
               "rounds_per_step": 1, "matches_device_result": bool(torch.equal(h_out.to(device), out_ref))}
        del hH, h_noise, h_unif, h_out
    return e2e


def extras_leg(B, w, args, device, stream, live):
    """The kernels beside the path (model update, plain-sum rule, coordinate-wise statistics), rank 0."""
    n, f, d = w.n, w.f, w.d
    U, out, ctx, timer = live["U"], live["out"], live["ctx"], live["timer"]
    extras = None
    if not args.no_extras:
        extras = {}
        weights = torch.zeros((n, w.ld), dtype=torch.float32, device=device)
        ctx.aggregate(U, out, stream)
        ctx.apply_update(out, weights, 0.01, stream)
        ms = timer.median_ms(lambda: ctx.apply_update(out, weights, 0.01, stream), 3)
        alg = 8 * n * d + 4 * n * ((d + 31) // 32)
        extras["model_update"] = {"ms": ms, "algorithmic_gbs": alg / (ms * 1e-3) / 1e9,
                                  "elements_per_s": n * d / (ms * 1e-3)}
        del weights
        ctx_sum = B.Brace(n, f, d, B.default_params(rule=B.RULE_SUM, agg_mode=B.AGG_FUSED), device=device)
        out_sum = ctx_sum.new_output(device=device)
        ctx_sum.aggregate(U, out_sum, stream)
        ms = timer.median_ms(lambda: ctx_sum.aggregate(U, out_sum, stream), 3)
        alg = 8 * n * d + 2 * 4 * d
        extras["sum_rule_fused"] = {"ms": ms, "algorithmic_gbs": alg / (ms * 1e-3) / 1e9,
                                    "elements_per_s": n * d / (ms * 1e-3)}
        ctx_sum.close()
        del out_sum
        torch.cuda.empty_cache()
        if n <= 128:
            # coordinate-wise median / trimmed mean: arithmetic-bound (sorting network of min/max pairs)
            res = torch.empty(d, dtype=torch.float32, device=device)
            # peak: the min/max rate of this GPU, measured now with the library's register-only probe kernel
            sms = torch.cuda.get_device_properties(device).multi_processor_count
            probe_out = torch.empty(sms * 8 * 256, dtype=torch.float32, device=device)
            B.minmax_rate_probe(sms * 8, 2000, probe_out, stream)
            pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            rates = []
            for _ in range(3):
                pa.record(stream)
                probe_ops = B.minmax_rate_probe(sms * 8, 20000, probe_out, stream)
                pb.record(stream)
                torch.cuda.synchronize()
                rates.append(probe_ops / (pa.elapsed_time(pb) * 1e-3))
            alu_peak = float(np.median(rates))
            del probe_out
            for label, kind, trim in (("median", B.STAT_MEDIAN, 0), ("trimmed_mean", B.STAT_TRIMMED_MEAN, f)):
                # the median reads a few middle positions only: comparators nothing of that depends on are not run
                pairs = sort_network_pairs(n, median_positions(n) if kind == B.STAT_MEDIAN else None)
                ctx.coordinate_stat(kind, trim, U, res, stream)
                ms = timer.median_ms(lambda: ctx.coordinate_stat(kind, trim, U, res, stream), 3)
                extras["coordinate_" + label] = {
                    "ms": ms, "elements_per_s": n * d / (ms * 1e-3), "bound": "alu",
                    "compare_exchanges_per_coordinate": pairs, "alu_ops_per_coordinate": 2 * pairs,
                    "achieved_ops_per_s": 2 * pairs * d / (ms * 1e-3), "peak_ops_per_s": alu_peak,
                    "peak_kind": "measured: min/max operations per second of a register-only probe kernel in this run",
                    "frac": 2 * pairs * d / (ms * 1e-3) / alu_peak, "hbm_gbs": (4 * n * d + 4 * d) / (ms * 1e-3) / 1e9}
            del res
    return extras


# ----------------------------------------------------------------------------- the CUDA arm
def run_cuda(args, head):
    rank, world, local = dist_env()
    # the CPU legs fork worker processes: run them before this process touches CUDA
    cpu_baseline = None
    if rank == 0 and not args.no_cpu:
        cpu_baseline = cpu_baseline_legs(head)

    from paper_2501_17392_b200 import brace as B
    from paper_2501_17392_b200 import build as brace_build

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
    stream = torch.cuda.current_stream()
    sampler = None
    if rank == 0:
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.3)

    head_res, live = measure_workload(B, head, args, device, stream, world, rank, sampler)
    e2e = e2e_leg(B, head, args, device, stream, world, live)
    extras = extras_leg(B, head, args, device, stream, live) if rank == 0 else None
    live["ctx"].close()
    live.clear()
    torch.cuda.empty_cache()

    per_config = None
    if rank == 0 and world == 1 and not args.no_per_config and not args.d:
        per_config = {}
        sub = argparse.Namespace(**vars(args))
        sub.steps = max(10, min(args.steps, 20))
        for name in ALL_WORKLOADS:
            if name == head.name:
                per_config[name] = head_res
                continue
            res, lv = measure_workload(B, W.WORKLOADS[name], sub, device, stream, 1, 0, sampler)
            if lv is not None:
                lv["ctx"].close()
                lv.clear()
            del lv
            torch.cuda.empty_cache()
            per_config[name] = res

    if rank != 0:
        dist.barrier()
        dist.destroy_process_group()
        return
    sampler.stop()
    n, f, d = head.n, head.f, head.d
    inj, rnd = head_res["roofline_inject"], head_res["roofline_round"]
    roofline = dict(inj if head_res["inject_ms"] > head_res["round_ms"] else rnd)
    roofline["other_kernel"] = rnd if roofline["kernel"] == inj["kernel"] else inj
    line = {
        "metric": METRIC, "value": head_res["elements_per_s"], "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": head_res["step_ms_median"],
        "ms_per_step_mean": head_res["step_ms_mean"], "timing": "median of the timed steps, CUDA events per step",
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": head.name, "n": n, "f": f, "d": d, "lambda": head.lam,
                   "rounds_per_step": head.rounds, "attack_kind": head.attack, "aggregate_mode": args.mode,
                   "l2": head_res["l2"], "replicas": world, "parallelism": "replicas only"},
        "clocks": head_res.get("clocks"), "e2e": e2e,
        "gpu_launches": head_res["gpu_launches_per_step"] * args.steps,
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "phases_ms": {"inject": head_res["inject_ms"], "aggregate": head_res["round_ms"]},
        "aggregate_only_elements_per_s": head_res["round_only_elements_per_s"],
        "same_result": head_res["same_result"], "stepwise": head_res.get("stepwise"),
        "back_to_back": head_res.get("back_to_back"), "extras": extras, "per_config": per_config,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(W.WORKLOADS))
    ap.add_argument("--mode", default="fused", choices=["fused", "stepwise", "auto"])
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--grid", type=int, default=0)
    ap.add_argument("--d", type=int, default=0, help="override the workload's vector length (profiling on a small case)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--supplied-draws", action="store_true",
                    help="attacks 2 and 5 read pre-drawn matrices instead of drawing in the kernel")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-stepwise", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
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
