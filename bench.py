#!/usr/bin/env python
"""Benchmark of the CADA hot path (one "step" = one full CADA iteration over all M workers).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2] [--also C5,C3,C1] [--impl ours|reference]

Prints ONE JSON line.  `value` is CADA iterations/s with all inputs resident in device memory
(timed with CUDA events on the library's stream around cada_step(K), repeated `repeats` times between
the same two events so that the region lasts at least 60 ms: `ms_per_step` = region / (repeats * K)); `e2e` is the same
metric through cada_step_host_n, i.e. with every step's minibatch copied from pinned host memory
and theta / the upload mask copied back inside the timed region (the copy of step i+1 overlaps step i).  `roofline` describes the
two-point gradient kernel (per-launch CUDA-event timing in a second pass of the same K steps).
`cpu_baseline` is the fp64 oracle timed on the host cores on a bounded sample of the same
workload.  `also` repeats the measurement for the other workloads (C5 is the bandwidth case).

With --gpus N > 1 (one process per GPU under torchrun) the workload's M workers are dealt over the
ranks (worker m on rank m mod N) and the ranks exchange one all-reduce of p floats per iteration
(Eq. 2a's sum); the total work is fixed, so the line reports strong scaling.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2012_15469_b200 import synth  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# small workloads finish their paper-sized run in a few milliseconds; time more iterations by default
DEFAULT_MIN_STEPS = {"C1": 20000, "C2": 20000, "C3": 5000}
MIN_REGION_MS = 60.0        # shortest timed region (several 20 ms clock samples fit)
MAX_REPEATS = 100000
METRIC = "cada_iterations_per_s"
UNIT = "iterations/s"


# ----------------------------------------------------------------------------------------------
# bookkeeping helpers (no GPU needed; covered by CPU tests)
# ----------------------------------------------------------------------------------------------

def algorithmic_bytes_per_iteration(w: synth.Workload, rule: int, uploads_per_iter: float) -> dict:
    """Bytes one CADA iteration must move (X rows once for both iterates; no padding counted)."""
    elt = 2 if w.x_bf16 else 4
    x_rows = w.M * w.batch * w.n_features * elt
    labels = w.M * w.batch * 4
    iterates = w.p * 4 * (2 if rule == synth.RULE_CADA1 else 1 + w.M)
    grad = x_rows + labels + iterates                       # the two-point gradient kernel
    trigger = w.M * w.p * 4 if rule == synth.RULE_CADA1 else 0
    replace = uploads_per_iter * w.p * 4 * 2
    aggregate = w.M * w.p * 4
    optimiser = 24 * w.p
    return {"grad_kernel": grad, "total": grad + trigger + replace + aggregate + optimiser}


def workload_label(w: synth.Workload) -> str:
    """The `config.workload` string both arms of the bench report."""
    kind = {synth.MODEL_LOGISTIC: "binary logistic", 1: "softmax regression", 2: "2-layer MLP"}.get(w.model, "model")
    return f"{w.name}: {kind} p={w.p}, M={w.M} workers x {w.n_samples} samples, batch {w.batch}"


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "source": "fallback"}


def kernel_source_hash(files) -> str:
    """Hash of the named kernel sources (files of csrc/): a traffic record is valid only for the sources it was taken with."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2012_15469_b200", "csrc")
    for name in sorted(files):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, kernel: str, iterations_per_launch: float = 1.0):
    """DRAM bytes per launch from the committed ncu summary, or None if the kernel's sources changed since."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        d = json.load(f)
    rec = d.get(f"{workload}:{kernel}")
    if not rec or rec.get("source_hash") != kernel_source_hash(rec.get("sources", [])):
        return None
    if "dram_bytes_per_iteration" in rec:
        return rec["dram_bytes_per_iteration"] * iterations_per_launch
    return rec["dram_bytes_per_launch"]


def aggregate_over_ranks(local_iters: int, local_ms: float, dist=None) -> tuple:
    """Whole-job units and the slowest rank's time (replicas: units add, time is the max)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_iters, local_ms
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    n = torch.tensor([local_iters], dtype=torch.int64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return int(n.item()), float(t.item())


def shard_workers(M: int, rank: int, world: int) -> dict:
    """Workers of rank `rank` when the M workers of Algorithm 1 are dealt round-robin over `world` ranks: worker m goes to
    rank m mod world.  Returns the cada_config fields of that rank's handle and the list of its workers."""
    mine = list(range(rank, M, world))
    return {"M_total": M, "m_first": rank, "m_stride": world, "workers": mine}


def sharded_step(solver, local_sum, dist) -> None:
    """One iteration with the workers split over the ranks: worker side on this rank's workers, ONE all-reduce of the
    p-vector of partial sums (Eq. 2a's sum is the only exchange of the method), server side on every rank."""
    solver.step_local(local_sum)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(local_sum, op=dist.ReduceOp.SUM)
    solver.step_apply(local_sum)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.rows, self.proc = gpu_index, [], None
        self.t_begin = self.t_end = None

    def start(self):
        """Launches the sampler and waits (up to 5 s) for its first sample."""
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            t0 = time.perf_counter()
            while not self.rows and time.perf_counter() - t0 < 5.0:
                time.sleep(0.01)
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [s.strip() for s in line.split(",")]))

    def begin(self):
        self.t_begin = time.perf_counter()

    def end(self):
        self.t_end = time.perf_counter()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.03)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [r for t, r in self.rows if self.t_begin is not None and self.t_begin <= t <= (self.t_end or 1e300)]
        window = "timed region"
        if not inside:      # region shorter than the sampling period: take the samples nearest to it
            inside = [r for _, r in self.rows[-3:]]
            window = "nearest samples (timed region shorter than the 20 ms sampling period)"
        for r in inside:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "window": window, "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# workloads
# ----------------------------------------------------------------------------------------------

def build_inputs(w: synth.Workload, device):
    """Returns (X list, y list, theta0) as CUDA tensors, plus host copies where they exist."""
    import torch
    if w.name in ("C5", "C5S"):
        X, y, t0 = synth.make_device_logistic(w, device)
        return [X[m] for m in range(w.M)], [y[m] for m in range(w.M)], t0, None
    Xs, ys, t0 = synth.make_host_data(w)
    if w.x_bf16:
        Xd = [torch.from_numpy(x).to(device).to(torch.bfloat16).contiguous() for x in Xs]
    else:
        Xd = [torch.from_numpy(x).to(device) for x in Xs]
    yd = [torch.from_numpy(y).to(device) for y in ys]
    return Xd, yd, torch.from_numpy(t0).to(device), (Xs, ys, t0)


def make_solver(w, rule, Xd, yd, t0, *, seed, host_step=False, shard=None):
    from paper_2012_15469_b200 import binding as B
    kw = {}
    if shard is not None:
        Xd, yd = [Xd[m] for m in shard["workers"]], [yd[m] for m in shard["workers"]]
        kw = {k: shard[k] for k in ("M_total", "m_first", "m_stride")}
    return B.Cada(model=w.model, rule=rule, X=Xd, y=yd, theta0=t0, batch=w.batch, alpha=w.alpha, beta1=w.beta1,
                  beta2=w.beta2, eps=w.eps, c=w.c, d_max=w.d_max, D=w.D, lam=w.lam, n_features=w.n_features,
                  n_classes=w.n_classes, n_hidden=w.n_hidden, has_bias=w.has_bias, seed=seed, host_step=host_step, **kw)


def oracle_for(w, rule, Xs, ys, t0, seed):
    from oracle import cada_oracle as O
    model = O.Model(w.model, w.n_features, w.n_classes, w.n_hidden, w.has_bias, w.lam, bf16=w.x_bf16)
    f32 = lambda v: float(np.float32(v))
    return O.CadaOracle(model, rule, Xs, ys, t0, batch=w.batch, alpha=f32(w.alpha), beta1=f32(w.beta1),
                        beta2=f32(w.beta2), eps=f32(w.eps), c=f32(w.c), d_max=w.d_max, D=w.D, seed=seed)


def time_oracle(w, rule, host, Xd, seed, budget_s: float, max_iters: int) -> dict:
    """The oracle, as it stands, on the host cores: iterations/s over a bounded number of iterations."""
    from oracle import cada_oracle as O
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    if host is not None:
        Xs, ys, t0 = host
        orc = oracle_for(w, rule, Xs, ys, t0, seed)
        idx_fn = lambda k: None
        sample = "first iterations of the full workload"
    else:
        # data live on the device only: bring over exactly the rows the first iterations sample
        import torch
        n_it = min(max_iters, 2)
        idx = [O.sample_indices(seed, k, w.M, w.batch, [w.n_samples] * w.M) for k in range(n_it)]
        Xs, ys, remap = [], [], [np.empty((w.M, w.batch), dtype=np.int64) for _ in range(n_it)]
        yd = host_y_device = None
        for m in range(w.M):
            rows = np.unique(np.concatenate([ix[m] for ix in idx]))
            pos = {int(r): i for i, r in enumerate(rows)}
            sel = torch.from_numpy(rows).to(Xd[0][m].device)
            Xs.append(Xd[0][m].index_select(0, sel).cpu().numpy())
            ys.append(Xd[1][m].index_select(0, sel).cpu().numpy())
            for k in range(n_it):
                remap[k][m] = [pos[int(r)] for r in idx[k][m]]
        orc = oracle_for(w, rule, Xs, ys, np.zeros(w.p, dtype=np.float32), seed)
        idx_fn = lambda k: remap[k]
        max_iters = n_it
        sample = f"first {n_it} iterations (their sampled rows copied from the device)"
    t_start = time.perf_counter()
    done = 0
    while done < max_iters and (time.perf_counter() - t_start) < budget_s:
        orc.step(idx_fn(done))
        done += 1
    dt = time.perf_counter() - t_start
    return {"value": done / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{done} iterations, {sample}, rule CADA{rule}", "seconds": round(dt, 2)}


def run_workload(name: str, rule: int, steps, warmup: int, *, device, rank: int, dist, with_e2e: bool,
                 cpu_budget_s: float, clocks: bool) -> dict:
    import torch
    from paper_2012_15469_b200 import binding as B

    w = synth.workload(name)
    K = steps if steps else max(w.iters, DEFAULT_MIN_STEPS.get(name, 0))
    seed = w.sample_seed + 7919 * rank
    Xd, yd, t0, host = build_inputs(w, device)
    stream = torch.cuda.current_stream()
    solver = make_solver(w, rule, Xd, yd, t0, seed=seed)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- resident timing ---------------------------------------------------------------------
    # The timed region is the K-step call repeated R times between the same two events, R chosen so that the region
    # lasts at least MIN_REGION_MS: a single call of a small workload is over before a clock sample can be taken.
    solver.step(warmup)
    barrier()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record(stream)
    solver.step(K)
    c1.record(stream)
    barrier()
    R = max(1, min(MAX_REPEATS, int(math.ceil(MIN_REGION_MS / max(c0.elapsed_time(c1), 1e-3)))))
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        r_t = torch.tensor([R], dtype=torch.int64, device=device)
        dist.all_reduce(r_t, op=dist.ReduceOp.MAX)
        R = int(r_t.item())
    st0 = solver.stats()
    sampler = ClockSampler(torch.cuda.current_device()) if clocks else None
    if sampler:
        sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler:
        sampler.begin()
    e0.record(stream)
    for _ in range(R):
        solver.step(K)
    e1.record(stream)
    barrier()
    if sampler:
        sampler.end()
    ms = e0.elapsed_time(e1)
    clk = sampler.stop() if sampler else None
    st1 = solver.stats()
    launches = st1.kernel_launches - st0.kernel_launches
    uploads = st1.uploads_total - st0.uploads_total
    KR = K * R
    total_iters, max_ms = aggregate_over_ranks(KR, ms, dist)
    value = total_iters / (max_ms / 1e3)

    # ---- per-launch timing of the gradient kernel (second pass of K steps) --------------------
    solver.profile(True)
    p0 = solver.stats()
    solver.step(K)
    p1 = solver.stats()
    solver.profile(False)
    n_l = p1.grad_kernel_launches - p0.grad_kernel_launches
    n_it = p1.profiled_iterations - p0.profiled_iterations
    fused = launches * 2 <= KR         # whole iterations inside one launch (small logistic problems)
    grad_ms = (p1.grad_kernel_ms - p0.grad_kernel_ms) / max(n_l, 1)
    ab = algorithmic_bytes_per_iteration(w, rule, uploads / KR)
    peaks = measured_peaks()
    per_launch_bytes = (ab["total"] if fused else ab["grad_kernel"]) * (n_it / max(n_l, 1))
    achieved = per_launch_bytes / (grad_ms * 1e-3) / 1e9 if grad_ms > 0 else 0.0
    roofline = {"kernel": "fused iteration kernel (all steps of the path)" if fused else "two-point gradient",
                "bound": "hbm", "achieved": round(achieved, 1),
                "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                "frac": round(achieved / peaks["hbm_gbs"], 4), "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                "bytes_per_launch": per_launch_bytes, "us_per_launch": round(grad_ms * 1e3, 2),
                "iterations_per_launch": n_it / max(n_l, 1),
                "launches_timed": int(n_l), "traffic": recorded_traffic(name, "fused" if fused else "grad", n_it / max(n_l, 1)),
                "whole_iteration_GBs": round(ab["total"] / (ms / KR * 1e-3) / 1e9, 1)}
    solver.close()

    out = {"workload": name, "rule": f"CADA{rule}", "value": value, "ms_per_step": max_ms / KR, "steps": K,
           "repeats": R, "timed_region_ms": max_ms,
           "worker_grads_per_s": value * w.M, "point_gradients_per_s": 2 * value * w.M,
           "gpu_launches": int(launches), "uploads_per_iteration": uploads / KR,
           "roofline": roofline, "clocks": clk, "M": w.M, "batch": w.batch, "p": w.p}

    # ---- end to end: minibatch from pinned host memory every step ---------------------------
    if with_e2e and host is not None:
        Ke = min(max(K, 200), 2000)
        Xs, ys, _ = host
        rng = np.random.default_rng(seed)
        elt_dtype = torch.bfloat16 if w.x_bf16 else torch.float32
        hx = torch.empty((Ke, w.M, w.batch, w.ldx), dtype=elt_dtype).pin_memory()
        hy = torch.empty((Ke, w.M, w.batch), dtype=torch.float32 if w.model == synth.MODEL_LOGISTIC else torch.int32).pin_memory()
        for k in range(Ke):
            for m in range(w.M):
                rows = rng.integers(0, Xs[m].shape[0], size=w.batch)
                hx[k, m] = torch.from_numpy(Xs[m][rows]).to(elt_dtype)
                hy[k, m] = torch.from_numpy(ys[m][rows])
        th = torch.empty((Ke, w.p), dtype=torch.float32).pin_memory()
        mk = torch.empty((Ke, w.M), dtype=torch.uint8).pin_memory()
        s2 = make_solver(w, rule, Xd, yd, t0, seed=seed, host_step=True)
        s2.step_host_n(min(max(warmup, 3), Ke), hx, hy, th, mk)
        barrier()
        t_0 = time.perf_counter()
        s2.step_host_n(Ke, hx, hy, th, mk)          # every step: minibatch H2D, the iteration, theta and mask D2H; one sync at the end
        torch.cuda.synchronize()
        dt = time.perf_counter() - t_0
        tot, mx = aggregate_over_ranks(Ke, dt * 1e3, dist)
        streamed_by_kernel = s2.stats().path == B.CADA_PATH_ONE_LAUNCH_CLUSTER
        out["e2e"] = {"value": tot / (mx / 1e3), "unit": UNIT, "steps": Ke, "api": "cada_step_host_n",
                      "transport": ("one launch per call; the kernel's fetching warps read every step's minibatch from the pinned host "
                                    "buffers over the bus and store theta and the mask of every step into pinned host memory")
                      if streamed_by_kernel else "per step: cudaMemcpyAsync H2D on a copy stream into a double-buffered staging area, results D2H",
                      "h2d_bytes_per_step": int(hx[0].numel() * hx.element_size() + hy[0].numel() * 4),
                      "d2h_bytes_per_step": int(w.p * 4 + w.M)}
        s2.close()
    elif with_e2e:
        out["e2e"] = None

    if rank == 0 and cpu_budget_s > 0:
        out["cpu_baseline"] = time_oracle(w, rule, host, (Xd, yd), seed, cpu_budget_s, K)
    del Xd, yd
    torch.cuda.empty_cache()
    return out


def run_sharded(name: str, rule: int, steps, warmup: int, *, device, rank: int, world: int, dist) -> dict:
    """N > 1: the M workers of the workload are dealt over the ranks (worker m on rank m mod N); per iteration every rank runs
    the worker side for its workers, the ranks all-reduce ONE p-vector (NCCL, on the library's stream), and every rank applies
    the server update to its replica of theta, h, vhat and the window.  Total work is fixed: strong scaling."""
    import torch
    w = synth.workload(name)
    if w.name in ("C5", "C5S"):
        raise SystemExit("the sharded mode builds its inputs on the host: use --workload C1..C4")
    K = steps if steps else w.iters
    Xs, ys, t0 = synth.make_host_data(w)            # same seed on every rank: the ranks hold disjoint workers of ONE problem
    shard = shard_workers(w.M, rank, world)
    if w.x_bf16:
        Xd = {m: torch.from_numpy(Xs[m]).to(device).to(torch.bfloat16).contiguous() for m in shard["workers"]}
    else:
        Xd = {m: torch.from_numpy(Xs[m]).to(device) for m in shard["workers"]}
    yd = {m: torch.from_numpy(ys[m]).to(device) for m in shard["workers"]}
    solver = make_solver(w, rule, Xd, yd, torch.from_numpy(t0).to(device), seed=w.sample_seed, shard=shard)
    local_sum = torch.zeros(w.p, dtype=torch.float32, device=device)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        sharded_step(solver, local_sum, dist)
    barrier()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record(stream)
    for _ in range(K):
        sharded_step(solver, local_sum, dist)
    c1.record(stream)
    barrier()
    r_t = torch.tensor([max(1, min(MAX_REPEATS, int(math.ceil(MIN_REGION_MS / max(c0.elapsed_time(c1), 1e-3)))))],
                       dtype=torch.int64, device=device)
    dist.all_reduce(r_t, op=dist.ReduceOp.MAX)
    R = int(r_t.item())
    st0 = solver.stats()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.begin()
    e0.record(stream)
    for _ in range(R * K):
        sharded_step(solver, local_sum, dist)
    e1.record(stream)
    barrier()
    sampler.end()
    ms = e0.elapsed_time(e1)
    clk = sampler.stop()
    st1 = solver.stats()
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    max_ms = float(t.item())
    counts = torch.tensor([st1.uploads_total - st0.uploads_total, st1.kernel_launches - st0.kernel_launches], dtype=torch.int64, device=device)
    dist.all_reduce(counts, op=dist.ReduceOp.SUM)
    KR = K * R
    value = KR / (max_ms / 1e3)                      # every rank walks the same KR iterations of the one problem
    solver.close()
    return {"workload": name, "rule": f"CADA{rule}", "value": value, "ms_per_step": max_ms / KR, "steps": K, "repeats": R,
            "timed_region_ms": max_ms, "worker_grads_per_s": value * w.M, "point_gradients_per_s": 2 * value * w.M,
            "gpu_launches": int(counts[1].item()), "uploads_per_iteration": float(counts[0].item()) / KR, "clocks": clk,
            "allreduce_bytes_per_iteration": w.p * 4, "workers_per_rank": [len(range(r, w.M, world)) for r in range(world)]}


def run_reference(args) -> None:
    """--impl reference: the oracle on the host cores, same workload / metric / unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.workload(args.workload)
    rule = args.rule
    if w.name in ("C5", "C5S"):
        print(json.dumps({"impl": "reference", "unavailable": "C5 lives in device memory only; use --workload C1..C4"}))
        return
    host = synth.make_host_data(w)
    K, W = args.steps or 50, args.warmup
    orc = oracle_for(w, rule, host[0], host[1], host[2], w.sample_seed)
    for _ in range(W):
        orc.step()
    t0 = time.perf_counter()
    for _ in range(K):
        orc.step()
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    value = K / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
            "warmup": W, "ms_per_step": dt / K * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_label(w), "rule": f"CADA{rule}", "c": w.c, "d_max": w.d_max, "D": w.D,
                       "parallelism": "host cores (oracle)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"{K} iterations of the full workload after {W} warm-up iterations"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed iterations (0 = the workload's full run)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C2")
    ap.add_argument("--rule", type=int, default=2, choices=[1, 2])
    ap.add_argument("--also", default="C5,C4,C3,C1", help="comma list of extra workloads reported under 'also' (N=1 only)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--sharded", action="store_true",
                    help="use the worker-sharded stepping (cada_step_local / all-reduce / cada_step_apply) even on one GPU")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1 or args.sharded:
        if world == 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29655")
            dist.init_process_group("nccl", device_id=device, rank=0, world_size=1)
        else:
            dist.init_process_group("nccl", device_id=device)
    from paper_2012_15469_b200 import build as build_mod
    build_mod.build()

    if world > 1 or args.sharded:
        res = run_sharded(args.workload, args.rule, args.steps, args.warmup, device=device, rank=rank, world=world, dist=dist)
        if rank == 0:
            w = synth.workload(args.workload)
            print(json.dumps({
                "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": res["steps"], "warmup": args.warmup,
                "ms_per_step": res["ms_per_step"], "repeats": res["repeats"], "timed_region_ms": res["timed_region_ms"],
                "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": workload_label(w), "rule": res["rule"], "c": w.c, "d_max": w.d_max, "D": w.D,
                           "parallelism": f"workers sharded over {world} GPUs (worker m on rank m mod {world}); one NCCL all-reduce of "
                                          f"{w.p} floats per iteration; server state replicated",
                           "l2": "no flush: every iteration samples fresh random rows"},
                "worker_grads_per_s": res["worker_grads_per_s"], "point_gradients_per_s": res["point_gradients_per_s"],
                "uploads_per_iteration": res["uploads_per_iteration"], "clocks": res["clocks"], "gpu_launches": res["gpu_launches"],
                "allreduce_bytes_per_iteration": res["allreduce_bytes_per_iteration"], "workers_per_rank": res["workers_per_rank"],
                "e2e": None, "e2e_note": "the host-minibatch entry points are not offered for worker-sharded handles",
                "roofline": None, "cpu_baseline": None}))
        dist.destroy_process_group()
        return
    main_res = run_workload(args.workload, args.rule, args.steps, args.warmup, device=device, rank=rank,
                            dist=None, with_e2e=True, cpu_budget_s=args.cpu_seconds, clocks=True)
    also = []
    if world == 1 and args.also:
        for name in [s for s in args.also.split(",") if s and s != args.workload]:
            r = run_workload(name, args.rule, 0 if not args.steps else args.steps, args.warmup, device=device, rank=0,
                             dist=None, with_e2e=False, cpu_budget_s=min(args.cpu_seconds, 8.0), clocks=True)
            also.append(r)

    if rank == 0:
        w = synth.workload(args.workload)
        line = {"metric": METRIC, "value": main_res["value"], "unit": UNIT, "n_gpus": world, "steps": main_res["steps"],
                "warmup": args.warmup, "ms_per_step": main_res["ms_per_step"], "higher_is_better": True,
                "repeats": main_res["repeats"], "timed_region_ms": main_res["timed_region_ms"],
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": workload_label(w),
                           "rule": main_res["rule"], "c": w.c, "d_max": w.d_max, "D": w.D,
                           "parallelism": "single GPU",
                           "l2": "no flush: every iteration samples fresh random rows from a dataset larger than L2 "
                                 f"({w.M * w.n_samples * w.ldx * 4 / 1e6:.0f} MB)"},
                "worker_grads_per_s": main_res["worker_grads_per_s"],
                "point_gradients_per_s": main_res["point_gradients_per_s"],
                "uploads_per_iteration": main_res["uploads_per_iteration"],
                "clocks": main_res["clocks"], "e2e": main_res.get("e2e"), "gpu_launches": main_res["gpu_launches"],
                "roofline": main_res["roofline"], "cpu_baseline": main_res.get("cpu_baseline"), "also": also}
        # the bandwidth-bound configuration (C5) carries the HBM-roofline figure of the path; repeat it at the top level
        for r in also:
            if r["workload"] == "C5":
                line["roofline_hbm_bound_workload"] = dict(r["roofline"], workload="C5", ms_per_step=r["ms_per_step"],
                                                           iterations_per_s=r["value"])
        print(json.dumps(line))


if __name__ == "__main__":
    main()
