#!/usr/bin/env python
"""Benchmark of the majority-vote sparse DSGD step.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c1] [--impl ours|reference]

A step is one whole pass of the hot path (error feedback, per-worker top-K, vote count, shared
mask, aggregate, residual) over one batch of synthetic gradients; the residual is carried from
step to step and every step gets fresh gradients from a pool that was generated before the timed
region.  Before the warm-up the residuals are carried through 300 untimed steps, so that the timed
steps are those of a run in progress (every chunk of every worker holds candidates) and not of its
first iterations.  One JSON line is printed by rank 0; with the default workload it also carries the
other two ResNet-scale configurations under "also".  With --gpus N > 1 (launched through torchrun) every
rank runs an independent replica of the same workload (the one-GPU step does not shard); `--sharded` instead
spreads the workload's N workers over the ranks and all-reduces the votes and the partial sums.
"""
from __future__ import annotations

import argparse
import contextlib
import hashlib
import json
import os
import re
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2011_06495_b200 import workloads as WL  # noqa: E402

RS_SEED = 201106495
METRIC = "majority-vote sparse steps/s"
UNIT = "steps/s"
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


STREAM_KERNEL_FUNCTIONS = ("pdl_enter", "fkey", "lanemask_lt", "chunk_geom", "load_keys", "load_extra", "iter_ranks",
                           "ge_mask", "emit_candidates", "k_acc_compact")


def function_text(text: str, name: str) -> str:
    """Source text of the first __device__/__global__ function called `name` (signature through closing brace)."""
    for m in re.finditer(r"^[^\n;{}]*\b" + re.escape(name) + r"\s*\(", text, flags=re.M):
        line_start = text.rfind("\n", 0, m.start()) + 1
        head = text[max(0, line_start - 200):m.end()]
        if "__device__" not in head and "__global__" not in head:
            continue
        i = text.index("{", m.end())
        depth, j = 1, i + 1
        while depth:
            depth += {"{": 1, "}": -1}.get(text[j], 0)
            j += 1
        return text[line_start:j]
    raise KeyError(name)


def kernel_source_hash():
    """Hash of the streaming kernel and of the device functions it calls (the counters in
    profiles/traffic.json belong to exactly this text)."""
    src = os.path.join(ROOT, "paper_2011_06495_b200", "csrc", "mv_sparse.cu")
    text = open(src).read()
    consts = "".join(re.findall(r"^constexpr[^\n]*\n", text, flags=re.M))
    body = consts + "".join(function_text(text, f) for f in STREAM_KERNEL_FUNCTIONS)
    return hashlib.sha256(body.encode()).hexdigest()[:16]


def recorded_traffic(workload: str, n_units: int):
    """DRAM bytes per launch of the streaming kernel from the committed ncu summary, scaled to this
    launch by the elements processed; None if the kernel source changed since the capture."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        rec = json.load(open(path))
        if rec.get("source_sha256_16") != kernel_source_hash():
            return None
        if n_units * 4 <= l2_bytes():        # an L2-resident case moves other bytes than a streaming one
            return None
        # captured on c2; the streaming pass moves the same bytes per element on any input larger than L2
        return float(rec["dram_bytes_per_element"]) * n_units
    except Exception:
        return None


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def rows_so_far(self) -> int:
        try:
            return sum(1 for r in open(self.file.name) if r.strip())
        except Exception:
            return 0

    def wait_for_first_sample(self, limit_s: float = 3.0):
        t0 = time.time()
        while self.proc is not None and self.rows_so_far() == 0 and time.time() - t0 < limit_s:
            time.sleep(0.02)

    def stop(self, first_row: int = 0):
        """Median SM clock and the throttle reasons seen in the rows from `first_row` on."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        try:
            self.file.flush()
            rows = [r.strip().split(", ") for r in open(self.file.name) if r.strip()]
            rows = rows[max(0, min(first_row, len(rows) - 1)):]
            os.unlink(self.file.name)
        except Exception:
            rows = []
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[4:8]):
                if val.strip().lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_run(w: WL.Workload, steps: int, warmup: int, threads: int, method: str = "mv"):
    """Times the CPU oracle as it stands on the whole workload (all N workers, full d and K): `warmup`
    untimed steps, then `steps` timed ones, the residual carried.  `threads` host threads work on
    different workers' rows at the same time (the oracle's own option; its arithmetic is the same).
    Returns (seconds per step, steps timed)."""
    from oracle import mv_oracle as O
    err = WL.initial_err(w).numpy()
    prev = np.zeros((w.N, w.d), dtype=bool)
    times = []
    for s in range(warmup + steps):
        g = WL.gradients(w, s).numpy()
        t0 = time.perf_counter()
        if method == "ad":
            r = O.mv_ad_step(g, err, prev, w.K, max(1, w.K // 10))
            prev = r["prev"]
        elif method == "rs":
            from oracle import rs_oracle as R
            r = R.mv_rs_step(g, err, w.K, RS_SEED, s)
        else:
            r = O.mv_sparse_step(g, err, w.K, threads=threads)
        dt = time.perf_counter() - t0
        err = r["err"]
        if s >= warmup:
            times.append(dt)
    return float(np.mean(times)), len(times)


def oracle_budget_steps(w: WL.Workload, asked: int, seconds: float) -> int:
    """How many whole steps of the oracle fit a budget of `seconds`, by its cost of roughly 10 ns per
    element and thread plus the generation of the inputs; at least 1, at most `asked`."""
    per_step = 25e-9 * w.N * w.d + 0.05
    return int(max(1, min(asked, seconds // per_step)))


def run_reference(args, w: WL.Workload):
    """The reference arm: the CPU oracle on the host cores (rank 0 only), whole steps of the whole
    workload.  `steps` and `warmup` in the line are the ones that ran."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cores = host_cores()
    threads = max(1, min(cores, w.N)) if args.method == "mv" else 1
    steps = oracle_budget_steps(w, args.steps, 90.0)
    warmup = 1 if args.warmup >= 1 else 0
    sec, ran = oracle_run(w, steps, warmup, threads, method=args.method)
    sps = 1.0 / sec
    sample = (f"whole workload: all {w.N} workers, d={w.d}, K={w.K}; {ran} consecutive step(s) timed after {warmup} "
              f"untimed, residual carried; {threads} host thread(s) over the workers' rows")
    line = {
        "impl": "reference", "metric": METRIC, "value": sps, "unit": UNIT, "n_gpus": args.gpus, "steps": ran,
        "warmup": warmup, "steps_asked": args.steps, "warmup_asked": args.warmup,
        "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": sps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                         "host_cores_available": cores},
        "e2e": {"value": sps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """The sweep of the configuration list: N in {4,16,64} x d in {2^20,2^24,2^27} x K/d in {1e-2,1e-3,2.5e-4},
    gradients with cross-worker correlation 0.3, residuals ~ N(0, 0.01^2).  Per cell: 3 warm-up steps, then
    `reps` single steps, each from the same saved residual (the restore is outside the timed region); the
    candidate threshold is carried from the step before (the default mode, --mode track: the warm-up steps
    leave it; --mode auto samples it in every step instead); the median is reported.  One GPU."""
    from paper_2011_06495_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak()
    reps = 10
    for w in WL.sweep_cells():
        grads = WL.gradients(w, 0, device=dev)
        err0 = WL.initial_err(w, device=dev)
        err = torch.empty_like(err0)
        out_idx = torch.empty(w.K, dtype=torch.int32, device=dev)
        out_val = torch.empty(w.K, dtype=torch.float32, device=dev)
        ctx = B.MvContext(w.N, w.d, w.K, device=dev,
                          mode={"auto": B.MV_MODE_AUTO, "general": B.MV_MODE_GENERAL, "track": B.MV_MODE_TRACK}[args.mode])
        times = []
        for it in range(3 + reps):
            err.copy_(err0)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            ctx.mv_sparse_step(grads, err, out_idx, out_val)
            ev1.record()
            torch.cuda.synchronize()
            if it >= 3:
                times.append(ev0.elapsed_time(ev1))
        ms = float(np.median(times))
        nbytes = w.N * w.d * 4
        line = {"metric": METRIC, "value": 1000.0 / ms, "unit": UNIT, "ms_per_step": ms, "ms_min": float(min(times)),
                "config": {"workload": f"sweep cell N={w.N} d={w.d} K={w.K}", "N": w.N, "d": w.d, "K": w.K,
                           "l2": "inputs larger than L2" if 2 * nbytes > l2_bytes() else "inputs fit in L2"},
                "effective_gradient_gbs": nbytes / ms / 1e6, "step_roofline_frac": 3 * nbytes / ms / 1e6 / peak,
                "peak": peak, "peak_kind": "of " + peak_kind, "launches_per_step": ctx.last_launches(),
                "fallback_workers": int((ctx.read_diag(w.N)[:, 2] != 0).sum()), "repeats": reps, "dtype": "f32", "data": "synthetic",
                "threshold": args.mode}
        print(json.dumps(line), flush=True)
        ctx.close()
        del grads, err0, err, out_idx, out_val, ctx
        torch.cuda.empty_cache()


def max_over_ranks(value: float, dist, device) -> float:
    """Largest value over all ranks (the job is as slow as its slowest replica)."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_steps_per_s(ms_total_max: float, world: int, steps: int) -> float:
    """Whole-job throughput of `world` independent replicas that each ran `steps` steps."""
    return world * steps / (ms_total_max * 1e-3)


def l2_bytes() -> int:
    """L2 capacity of the current CUDA device (what decides whether a workload streams from HBM)."""
    if torch.cuda.is_available():
        return int(torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size)
    return 126 * 1024 * 1024      # no device to ask (the reference arm on a host without one): B200's data-sheet size


def workload_config(w: WL.Workload):
    nbytes = w.N * w.d * 4
    return {"workload": f"{w.name}: N={w.N} workers, d={w.d} fp32, K={w.K} ({w.note}), error feedback carried, "
                        f"fresh gradients every step",
            "N": w.N, "d": w.d, "K": w.K,
            "l2": "inputs larger than L2" if nbytes > l2_bytes() else "L2-resident",
            "parallelism": "replicas only"}


PREHEAT_STEPS = 300      # untimed steps that carry the residuals into the error-feedback steady state
POOL_BYTES = 32e9        # gradient tensors generated before the timed region (cycled if the run is longer)
NOMINAL_HBM_GBS = 7700.0


def measure(w: WL.Workload, args, B, dev, dist, world, local_rank, with_e2e: bool):
    """Runs one workload: inputs resident in HBM, `preheat` untimed steps on fresh gradients so that the
    residuals are those of a run in progress, `--warmup` untimed steps, `--steps` timed ones (CUDA events
    on the launching stream, barrier and synchronize on both sides, max over ranks).  Returns the fields
    of the JSON line that depend on the workload."""
    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    nbytes = w.N * w.d * 4
    pool_n = int(max(2, min(args.steps + args.warmup, POOL_BYTES // nbytes, 64)))
    std = WL.std_vector(w, dev) if w.segments > 1 else None
    err = WL.initial_err(w, device=dev)
    out_idx = torch.empty(w.K, dtype=torch.int32, device=dev)
    out_val = torch.empty(w.K, dtype=torch.float32, device=dev)
    mode = {"auto": B.MV_MODE_AUTO, "general": B.MV_MODE_GENERAL, "track": B.MV_MODE_TRACK}[args.mode]
    ctx = B.MvContext(w.N, w.d, w.K, device=dev, mode=mode)

    if args.method == "ad":
        K_ad = max(1, w.K // 10)
        prev_bits = torch.zeros((w.N, (w.d + 31) // 32), dtype=torch.int32, device=dev)

        def one_step(g):
            ctx.mv_ad_step(g, err, prev_bits, K_ad, out_idx, out_val)
    elif args.method == "rs":
        draw = [0]

        def one_step(g):
            ctx.mv_rs_step(g, err, RS_SEED, draw[0], out_idx, out_val)
            draw[0] += 1
    else:
        def one_step(g):
            ctx.mv_sparse_step(g, err, out_idx, out_val)

    # ---- the state of a run in progress: residuals built up over `preheat` steps of fresh gradients
    preheat = args.preheat if args.preheat >= 0 else (PREHEAT_STEPS if w.steps > 1 else 0)
    scratch = torch.empty((w.N, w.d), dtype=torch.float32, device=dev)
    for s in range(preheat):
        one_step(WL.gradients(w, 100_000 + s, out=scratch, std=std))
    torch.cuda.synchronize()
    del scratch
    # ---- inputs resident in HBM before the timed region: gradient tensors not seen so far
    pool = [WL.gradients(w, s, device=dev, std=std) for s in range(pool_n)]

    sampler = ClockSampler(visible_gpu_index(local_rank))
    sampler.start()
    step_no = 0
    for _ in range(args.warmup):
        one_step(pool[step_no % pool_n])
        step_no += 1
    # CUDA events around the streaming kernel on one step in eight (each pair costs a few microseconds)
    ctx.set_kernel_timing(8 if args.steps >= 8 else 1)
    fb_before = ctx.fallback_count()
    sampler.wait_for_first_sample()
    barrier()
    first_row = sampler.rows_so_far()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        one_step(pool[step_no % pool_n])
        step_no += 1
    ev1.record()
    barrier()
    time.sleep(0.03)
    clocks = sampler.stop(first_row)
    ms_total = ev0.elapsed_time(ev1)
    launches_per_step = ctx.last_launches()
    k_ms, k_cnt = ctx.read_kernel_timing()
    ctx.set_kernel_timing(0)
    fallbacks = ctx.fallback_count() - fb_before
    diag = ctx.read_diag(w.N)
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms_step = ms_total / args.steps

    # ---- end to end through the host entry point: gradients start in pinned host memory
    e2e = None
    if with_e2e:
        h_pool = [pool[i].cpu().pin_memory() for i in range(2)]
        h_idx = torch.empty(w.K, dtype=torch.int32).pin_memory()
        h_val = torch.empty(w.K, dtype=torch.float32).pin_memory()
        d_grads = pool[-1]
        e_steps = max(3, min(args.steps, 10))
        for i in range(2):
            ctx.mv_sparse_step_host(h_pool[i % 2], h_idx, h_val, d_grads, err, out_idx, out_val)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(e_steps):
            ctx.mv_sparse_step_host(h_pool[i % 2], h_idx, h_val, d_grads, err, out_idx, out_val)
        e1.record()
        barrier()
        te = max_over_ranks(e0.elapsed_time(e1), dist, dev)
        e2e = {"value": job_steps_per_s(te, world, e_steps), "unit": UNIT,
               "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": 8 * w.K, "steps": e_steps,
               "note": "mv_sparse_step_host: gradients copied from pinned host memory every step, indices and "
                       "values copied back; the residual stays on the device"}
        del h_pool

    peak, peak_kind = measured_peak()
    alg_bytes = 12.0 * w.N * w.d                      # read grads, read err, write acc: 12 B per element
    k_ms_avg = k_ms / max(k_cnt, 1)
    achieved = alg_bytes / (k_ms_avg * 1e-3) / 1e9 if k_cnt else None
    step_gbs = alg_bytes / (ms_step * 1e-3) / 1e9
    frac = (achieved / peak) if achieved else None
    roofline = {"bound": "hbm", "kernel": "k_acc_compact" if args.mode != "general" else "k_hist<1,true>",
                "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": frac, "traffic": recorded_traffic(w.name, w.N * w.d),
                "kernel_ms": k_ms_avg, "kernel_launches_timed": k_cnt, "algorithmic_bytes_per_launch": alg_bytes,
                "peak_nominal": NOMINAL_HBM_GBS, "frac_of_nominal": (achieved / NOMINAL_HBM_GBS) if achieved else None}
    if frac is not None and frac > 1.0:
        roofline["note"] = ("above 1: the peak is the bandwidth of a plain device copy, which this kernel outruns; "
                            "frac_of_nominal is the fraction of the HBM3e data-sheet figure")
    out = {
        "value": job_steps_per_s(ms_total, world, args.steps), "ms_per_step": ms_step,
        "config": workload_config(w),
        "setup": dict(method={"ad": "add-drop voting, K_ad=K/10", "rs": "random selection proportional to the votes",
                              "mv": "majority voting"}[args.method],
                      threshold={"track": "candidate threshold carried from the previous step's key histogram",
                                 "auto": "candidate threshold sampled every step",
                                 "general": "no candidate threshold (multi-pass select)"}[args.mode],
                      preheat_steps=preheat, gradient_pool=pool_n),
        "effective_gradient_gbs": w.N * w.d * 4 / (ms_step * 1e-3) / 1e9,
        "step_roofline_frac": step_gbs / peak, "step_roofline_frac_of_nominal": step_gbs / NOMINAL_HBM_GBS,
        "roofline": roofline, "clocks": clocks,
        "gpu_launches": launches_per_step * args.steps, "launches_per_step": launches_per_step,
        "fallback_workers": int(fallbacks),
        "candidates_over_K_last_step": float(diag[:, 0].double().mean() / w.K),
    }
    if e2e is not None:
        out["e2e"] = e2e
    ctx.close()
    del pool, err, ctx
    torch.cuda.empty_cache()
    return out


@contextlib.contextmanager
def stdout_to_stderr():
    """File descriptor 1 points at stderr inside the block (libraries that print while they start up write there)."""
    sys.stdout.flush()
    saved = os.dup(1)
    os.dup2(2, 1)
    try:
        yield
    finally:
        sys.stdout.flush()
        os.dup2(saved, 1)
        os.close(saved)


def shard_rows(N: int, world: int, rank: int):
    """Rows [lo, hi) of the N workers that rank `rank` of `world` holds in the worker-sharded step."""
    return rank * N // world, (rank + 1) * N // world


def run_sharded(args, w: WL.Workload):
    """The worker-sharded step (launched through torchrun, one rank per GPU): the N workers of the workload are
    spread over the ranks, every rank streams and selects its own rows, the vote counts (d bytes) and the
    binary64 partial sums on the shared mask (8K bytes) are all-reduced over NCCL, every rank ends up with
    the same mask and values.  Total work is fixed, so scaling is strong; the step time is the slowest
    rank's (CUDA events on the context's stream, barrier and synchronize on both sides)."""
    import torch.distributed as dist
    from paper_2011_06495_b200 import binding as B
    from paper_2011_06495_b200.sharded import ShardedStep
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if world > w.N:
        raise SystemExit(f"--sharded: {world} ranks for {w.N} workers (every rank needs at least one)")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29655")
    with stdout_to_stderr():     # (the NCCL version banner must not share stdout with the JSON line)
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
        dist.barrier()
        torch.cuda.synchronize()

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    lo, hi = shard_rows(w.N, world, rank)
    n_local = hi - lo
    std = WL.std_vector(w, dev) if w.segments > 1 else None
    mode = {"auto": B.MV_MODE_AUTO, "general": B.MV_MODE_GENERAL, "track": B.MV_MODE_TRACK}[args.mode]
    ctx = B.MvContext(w.N, w.d, w.K, device=dev, mode=mode)
    step = ShardedStep(ctx, w.N, w.d, w.K, dev)
    err = WL.initial_err(w, device=dev)[lo:hi].clone()
    out_idx = torch.empty(w.K, dtype=torch.int32, device=dev)
    out_val = torch.empty(w.K, dtype=torch.float32, device=dev)
    full = torch.empty((w.N, w.d), dtype=torch.float32, device=dev)
    preheat = args.preheat if args.preheat >= 0 else (PREHEAT_STEPS if w.steps > 1 else 0)
    for s in range(preheat):                       # every rank draws the whole step's gradients and keeps its rows
        step.step(WL.gradients(w, 100_000 + s, out=full, std=std)[lo:hi], err, out_idx, out_val)
    nbytes_local = n_local * w.d * 4
    pool_n = int(max(2, min(args.steps + args.warmup, POOL_BYTES // max(nbytes_local, 1), 64)))
    pool = [WL.gradients(w, s, out=full, std=std)[lo:hi].clone() for s in range(pool_n)]
    del full
    torch.cuda.synchronize()
    # kernels per step, counted once outside the timed region
    # (one whole step written out call by call, as ShardedStep.step makes them)
    launches = 0
    ctx.mv_vote(pool[0], err, votes=step.votes, K=w.K)
    launches += ctx.last_launches()
    dist.all_reduce(step.votes, op=dist.ReduceOp.SUM)
    ctx.mv_select(step.votes, w.N, out_idx, K=w.K)
    launches += ctx.last_launches()
    ctx.mv_aggregate_partial(err, out_idx, step.partial)
    launches += ctx.last_launches() + 1            # + the kernel of mv_finish_mean
    dist.all_reduce(step.partial, op=dist.ReduceOp.SUM)
    ctx.mv_finish_mean(step.partial, w.N, out_val)
    sampler = ClockSampler(visible_gpu_index(local_rank))
    sampler.start()
    k = 0
    for _ in range(args.warmup):
        step.step(pool[k % pool_n], err, out_idx, out_val)
        k += 1
    ctx.set_kernel_timing(8 if args.steps >= 8 else 1)
    sampler.wait_for_first_sample()
    barrier()
    first_row = sampler.rows_so_far()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step.step(pool[k % pool_n], err, out_idx, out_val)
        k += 1
    ev1.record()
    barrier()
    time.sleep(0.03)
    clocks = sampler.stop(first_row)
    k_ms, k_cnt = ctx.read_kernel_timing()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), dist, dev)
    checksum = int(out_idx.sum(dtype=torch.int64).item())
    sums = torch.tensor([checksum], dtype=torch.int64, device=dev)
    gathered = [torch.zeros_like(sums) for _ in range(world)]
    dist.all_gather(gathered, sums)
    same_mask = all(int(g.item()) == checksum for g in gathered)
    if rank == 0:
        peak, peak_kind = measured_peak()
        ms_step = ms_total / args.steps
        alg_local = 12.0 * n_local * w.d
        k_ms_avg = k_ms / max(k_cnt, 1)
        achieved = alg_local / (k_ms_avg * 1e-3) / 1e9 if k_cnt else None
        line = {
            "metric": METRIC, "value": args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(w), parallelism="workers sharded over ranks: all-reduce of u8 votes (d B) and "
                                                           "of binary64 partial sums (8K B)"),
            "setup": {"workers_per_rank": [shard_rows(w.N, world, r)[1] - shard_rows(w.N, world, r)[0] for r in range(world)],
                      "preheat_steps": preheat, "gradient_pool": pool_n, "collectives": "NCCL all_reduce x 2 per step",
                      "collective_bytes_per_step": w.d + 8 * w.K},
            "effective_gradient_gbs": w.N * w.d * 4 / (ms_step * 1e-3) / 1e9,
            "step_roofline_frac": 12.0 * w.N * w.d / world / (ms_step * 1e-3) / 1e9 / peak,
            "roofline": {"bound": "hbm", "kernel": "k_acc_compact", "achieved": achieved, "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": (achieved / peak) if achieved else None,
                         "traffic": None, "kernel_ms": k_ms_avg, "algorithmic_bytes_per_launch": alg_local,
                         "note": "rank 0's streaming pass over its own workers' rows"},
            "clocks": clocks, "gpu_launches": launches * args.steps, "launches_per_step": launches,
            "same_mask_on_every_rank": same_mask,
        }
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c1", "c1_ties", "c2", "c3", "c4"])
    ap.add_argument("--mode", default="track", choices=["auto", "general", "track"],
                    help="how the per-worker candidate threshold is found: sampled every step (auto), carried from "
                         "the previous step's key histogram (track), or none (general)")
    ap.add_argument("--method", default="mv", choices=["mv", "ad", "rs"],
                    help="mv: plain majority voting (Algorithm 1); ad: add-drop voting (Algorithm 2) with K_ad = K/10; "
                         "rs: random selection proportional to the votes (Algorithm 1, second variant)")
    ap.add_argument("--preheat", type=int, default=-1,
                    help="untimed steps on fresh gradients before warm-up, so that the timed steps see the residuals of a "
                         f"run in progress (default: {PREHEAT_STEPS} for the multi-step workloads, 0 for c1)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-also", action="store_true",
                    help="with the default workload c2 the line also carries c3 and c4 (the other two ResNet-scale "
                         "configurations) under \"also\"; this switches that off")
    ap.add_argument("--sharded", action="store_true",
                    help="the worker-sharded step: the workload's N workers spread over the ranks (torchrun), votes and "
                         "partial sums all-reduced; strong scaling.  Without it, N GPUs run N replicas")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the one bench line: time the 27 cells of the sweep (N x d x K/d), one JSON line per "
                         "cell, a single step timed after warm-up with the residual restored before every repeat")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    w = WL.resnet_like(args.workload)

    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.sharded:
        run_sharded(args, w)
        return

    from paper_2011_06495_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        with stdout_to_stderr():     # (the NCCL version banner must not share stdout with the JSON line)
            dist.init_process_group("nccl", device_id=dev)
            dist.barrier()
            torch.cuda.synchronize()

    res = measure(w, args, B, dev, dist, world, local_rank, with_e2e=not args.no_e2e and args.method == "mv")
    also = {}
    if args.workload == "c2" and args.method == "mv" and not args.no_also:
        # the other two ResNet-scale configurations, same process, same flags
        for name in ("c3", "c4"):
            r = measure(WL.resnet_like(name), args, B, dev, dist, world, local_rank, with_e2e=False)
            also[name] = {"value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"],
                          "step_roofline_frac": r["step_roofline_frac"],
                          "step_roofline_frac_of_nominal": r["step_roofline_frac_of_nominal"],
                          "effective_gradient_gbs": r["effective_gradient_gbs"],
                          "roofline": {k: r["roofline"][k] for k in ("kernel", "achieved", "peak", "peak_kind", "frac", "frac_of_nominal", "kernel_ms")},
                          "clocks": r["clocks"], "launches_per_step": r["launches_per_step"],
                          "fallback_workers": r["fallback_workers"],
                          "config": r["config"], "setup": r["setup"]}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    line = {"metric": METRIC, "value": res.pop("value"), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic"}
    line.update(res)
    if also:
        line["also"] = also
    if world == 1 and not args.no_cpu_baseline:
        # the oracle as it stands on this machine's host cores: whole steps of the whole workload, on one
        # core and with its rows spread over the cores (a reported baseline, not a target)
        cores = host_cores()
        threads = max(1, min(cores, w.N)) if args.method == "mv" else 1
        n1 = oracle_budget_steps(w, 3, 12.0)
        sec1, ran1 = oracle_run(w, n1, 0, 1, method=args.method)
        line["cpu_baseline"] = {
            "value": 1.0 / sec1, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"whole workload: all {w.N} workers, d={w.d}, K={w.K}; {ran1} consecutive step(s) from zero "
                      f"residuals, one host thread", "host_cores_available": cores}
        if threads > 1:
            secn, rann = oracle_run(w, oracle_budget_steps(w, 3, 12.0), 0, threads, method=args.method)
            line["cpu_baseline"]["all_cores"] = {
                "value": 1.0 / secn, "unit": UNIT, "cores": threads,
                "sample": f"the same {rann} step(s) with {threads} host threads over the workers' rows"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
