#!/usr/bin/env python
"""Benchmark of the cb-DyBW round: simulated worker-rounds/s on one B200 (replicas on N GPUs).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

A step is one round of the whole hot path over one batch of synthetic input: backup counts
(threshold rule, where the workload is dynamic), mini-batch gradients (where the workload has a
model), fastest-neighbour selection, weights, fused mix + SGD.  One JSON line is printed by
rank 0.  `value` is timed with everything resident in HBM; `e2e` is the same loop through
dbw_round_host with the per-round inputs in pinned host memory and the per-round results read
back.  `roofline` is the mix kernel: 12 bytes per parameter element (read x, read g, write x')
over its own CUDA-event time inside the timed loop, against the measured copy bandwidth.
`cpu_baseline` times the double-precision CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import configs as wl  # noqa: E402

METRIC = "simulated worker-rounds/sec"
UNIT = "worker-rounds/s"
DEFAULT_CONFIG = 4
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the mix kernel, from the ncu captures summarised
# under profiles/ (config 4: the d = 65,536 case scaled by 16, the traffic being proportional to the columns
# processed; configs 2 and 3: their mix at full size).  Reported only for the kernel the capture was taken of;
# None = not captured for this workload.
MIX_TRAFFIC_BYTES = {4: ("mix_staged_kernel", (537.05e6 + 220.89e6) * 16),
                     3: ("mix_panel_kernel", 4.316048e9 + 3.227908e9),
                     2: ("mix_panel_kernel", 875.2448e6 + 612.1979e6)}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------
# workload set-up shared by the bench and the full-size parity tests
# ------------------------------------------------------------------------------------------

class Job:
    """One workload resident on one GPU, stepped through the C ABI."""

    def __init__(self, config: int, device: int = 0, rounds: int | None = None, col_range=None, consensus_only=False, **overrides):
        """col_range = (c0, c1): this job owns only those columns of a mix-only workload's matrices (one column
        shard of several; the update is independent per column, see paper_2102_06280_b200/sharding.py)."""
        import torch
        import paper_2102_06280_b200 as p
        self.torch, self.p = torch, p
        torch.cuda.set_device(device)
        self.dev = torch.device("cuda", device)
        w = self.w = wl.make_workload(config, **overrides)
        self.n_rounds = rounds or w.rounds
        flags = (p.WEIGHT_UNIFORM if w.weight_rule == "uniform" else 0) | (p.GEMM_BF16 if w.precision == "bf16" else 0)
        if w.layers is not None:
            self.m = p.model_layout(w.layers, w.batch)
            self.h = p.Dbw(w.rowptr, w.col, d=self.m.d, model=self.m, flags=flags, device=device)
            means = wl.class_means(w)
            feat = torch.empty((w.N, w.samples, w.layers[0]), dtype=torch.float32, device=self.dev)
            labels = torch.empty((w.N, w.samples), dtype=torch.int32, device=self.dev)
            for i in range(w.N):
                f, l = wl.worker_dataset(w, i, means)
                feat[i].copy_(torch.from_numpy(f))
                labels[i].copy_(torch.from_numpy(l))
            self.feat, self.labels = feat, labels
            self.h.set_dataset(feat, labels, w.samples)
            self.h.set_param_tracking(True)      # X is updated in place and never modified between rounds
            X0 = np.stack([wl.init_params(w, i) for i in range(w.N)])
            self.X = torch.from_numpy(self.m.pack(X0)).to(self.dev)
            self.G = None
            self.h_idx = torch.from_numpy(np.stack([wl.batch_indices(w, k) for k in range(self.n_rounds)])).pin_memory()
            self.d_idx = self.h_idx.to(self.dev)
            self.ld = self.m.ld
        else:
            self.m = None
            c0, c1 = col_range if col_range is not None else (0, w.d)
            self.ld = c1 - c0
            self.h = p.Dbw(w.rowptr, w.col, d=self.ld, ld=self.ld, flags=flags, device=device)
            self.X = torch.empty((w.N, self.ld), dtype=torch.float32, device=self.dev)
            self.G = torch.empty((w.N, self.ld), dtype=torch.float32, device=self.dev)
            step = 64
            for r0 in range(0, w.N, step):
                rows = range(r0, min(w.N, r0 + step))
                self.X[r0:r0 + step].copy_(torch.from_numpy(np.ascontiguousarray(wl.gaussian_rows(w.init_seed, rows, w.d)[:, c0:c1])))
                self.G[r0:r0 + step].copy_(torch.from_numpy(np.ascontiguousarray(
                    wl.gaussian_rows(wl.external_gradient_seed(w), rows, w.d, scale=0.01)[:, c0:c1])))
            self.h_idx = self.d_idx = None
            if consensus_only:      # the truncated model's tail (Section 3.2.1): G = 0, no gradient matrix is read
                self.G = None
        self.consensus_only = consensus_only and w.layers is None
        self.h_t = torch.from_numpy(wl.arrival_times(w, self.n_rounds)).pin_memory()
        self.d_t = self.h_t.to(self.dev)
        if w.backups == "fixed":
            hb = np.tile(wl.fixed_backups(w), (self.n_rounds, 1))
        elif w.backups == "uniform":
            hb = wl.uniform_backups(w, self.n_rounds)
        else:
            hb = np.zeros((self.n_rounds, w.N), dtype=np.int32)     # round 1: everyone waits for everyone
        self.h_b = torch.from_numpy(np.ascontiguousarray(hb)).pin_memory()
        self.d_b = self.h_b.to(self.dev)
        n, nnz = w.N, len(w.col)
        self.kept = torch.zeros(nnz, dtype=torch.uint8, device=self.dev)
        self.Tw = torch.zeros(n, dtype=torch.float64, device=self.dev)
        self.Tr = torch.zeros(1, dtype=torch.float64, device=self.dev)
        self.loss = torch.zeros(n, dtype=torch.float32, device=self.dev)
        self.b_dyn = torch.zeros(n, dtype=torch.int32, device=self.dev)
        self.hk = torch.zeros(nnz, dtype=torch.uint8).pin_memory()
        self.hTw = torch.zeros(n, dtype=torch.float64).pin_memory()
        self.hTr = torch.zeros(1, dtype=torch.float64).pin_memory()
        self.hloss = torch.zeros(n, dtype=torch.float32).pin_memory()
        self.hb_out = torch.zeros(n, dtype=torch.int32).pin_memory()
        self.k = 0
        torch.cuda.synchronize()

    def step(self):
        """One round, every input already on the device (in place on X)."""
        w, r = self.w, self.k % self.n_rounds
        b = self.d_b[r]
        if w.backups == "dtur" and self.k > 0:
            self.h.update_backups(self.d_t[r], self.b_dyn)
            b = self.b_dyn
        out = self._out()
        self.h.round(self.X, self.d_t[r], b, wl.learning_rate(w, self.k % self.n_rounds), out, self.kept,
                     batch_idx=None if self.d_idx is None else self.d_idx[r], G_ext=self.G,
                     T_worker=self.Tw, T_round=self.Tr, loss=self.loss)
        self._swap(out)
        self.k += 1

    def _out(self):
        """X itself where the selected mix kernel may run in place, else a second buffer (ping-pong)."""
        if self.h.mix_in_place_ok():
            return self.X
        if getattr(self, "X2", None) is None:
            self.X2 = self.torch.empty_like(self.X)
        return self.X2

    def _swap(self, out):
        if out is not self.X:
            self.X, self.X2 = out, self.X

    def capture(self, rounds_per_graph: int):
        """Capture `rounds_per_graph` consecutive rounds into one CUDA graph (launch-bound workloads).

        The graph bakes in the inputs of the rounds it was captured on, so replays cycle through
        those rounds' arrival times and batches; parameters and the threshold rule's state keep
        evolving.  Call after the warm-up rounds (one-time allocations happen there)."""
        torch = self.torch
        torch.cuda.synchronize()
        k0 = self.k
        self._graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self._graph):
            for _ in range(rounds_per_graph):
                self.step()
        self.k = k0
        self._graph_rounds = rounds_per_graph

    def step_graph(self):
        """`rounds_per_graph` rounds by one graph launch."""
        self._graph.replay()
        self.k += self._graph_rounds

    def step_host(self):
        """One round with the per-round inputs in pinned host memory and the results read back."""
        w, r = self.w, self.k % self.n_rounds
        dyn = w.backups == "dtur" and self.k > 0
        out = self._out()
        self.h.round_host(self.X, self.h_t[r], None if dyn else self.h_b[r], wl.learning_rate(w, self.k % self.n_rounds), out,
                          h_batch_idx=None if self.h_idx is None else self.h_idx[r], G_ext=self.G,
                          h_kept=self.hk, h_T_worker=self.hTw, h_T_round=self.hTr,
                          h_loss=None if self.h_idx is None else self.hloss, h_b_out=self.hb_out if dyn else None)
        self.torch.cuda.current_stream().synchronize()      # the caller reads the round's results
        self._swap(out)
        self.k += 1

    def host_bytes_per_step(self):
        w = self.w
        h2d = w.N * 8 + (0 if w.backups == "dtur" else w.N * 4) + (0 if self.h_idx is None else w.N * w.batch * 4)
        d2h = len(w.col) + w.N * 8 + 8 + (0 if self.h_idx is None else w.N * 4) + (w.N * 4 if w.backups == "dtur" else 0)
        return h2d, d2h

    def mix_bytes_per_launch(self):
        return (8 if self.consensus_only else 12) * self.w.N * self.ld

    def close(self):
        self.h.close()


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device: int):
        self.device, self.proc, self.path = device, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.device), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if not sm:
            return None
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(np.max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------
# CPU oracle timing (baseline leg and the reference arm)
# ------------------------------------------------------------------------------------------

def _one_thread():
    """Context manager pinning the BLAS / OpenMP pools of this process to one thread (no-op without threadpoolctl)."""
    try:
        from threadpoolctl import threadpool_limits
        return threadpool_limits(limits=1)
    except Exception:
        import contextlib
        return contextlib.nullcontext()


def _mix_block_seconds(job):
    """Worker of the all-core leg: the oracle's mix on all rows x one block of columns, one thread; returns seconds."""
    rowptr, col, ws, we, lr, n, cols, seed = job
    from oracle import dbw_oracle as orc
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, cols)).astype(np.float32)
    G = (0.01 * rng.standard_normal((n, cols))).astype(np.float32)
    with _one_thread():
        t0 = time.perf_counter()
        orc.mix_update(rowptr, col, X, G, ws, we, lr)
        return time.perf_counter() - t0


def _grad_block_seconds(job):
    """Worker of the all-core leg: the oracle's gradient of a few workers, one thread; returns seconds."""
    config, overrides, k, workers = job
    from oracle import dbw_oracle as orc
    w = wl.make_workload(config, **overrides)
    means = wl.class_means(w)
    idx = wl.batch_indices(w, k)
    data = [(wl.worker_dataset(w, i, means), wl.init_params(w, i)) for i in workers]
    with _one_thread():
        t0 = time.perf_counter()
        for i, ((f, l), x) in zip(workers, data):
            orc.mlp_grad(x, w.layers, f[idx[i]], l[idx[i]])
        return time.perf_counter() - t0


def oracle_sample_seconds(w, k: int = 0, budget_s: float = 12.0, pool=None, procs: int = 1, config=None, overrides=None):
    """Times the oracle, as it stands, on a bounded sample of round k; returns (estimated s per full round, description).

    Selection, times, weights (and the threshold rule) run whole.  Gradients run for a few workers and scale
    by N / sampled.  The mix runs on all rows x a block of columns and scales by d / sampled columns (the
    update is independent per column).  The timed code runs on ONE thread (BLAS pools pinned to one).  With a
    process pool (`pool`, `procs` processes started with spawn) the gradient workers and the mix's column blocks
    are spread over the processes, one thread each, and the slowest process counts: the all-core figure.
    """
    from oracle import dbw_oracle as orc
    rng = np.random.default_rng(123)
    t = wl.arrival_times(w, max(k + 1, 2))[k]
    with _one_thread():
        t0 = time.perf_counter()
        if w.backups == "dtur":
            b, _ = orc.Dtur(w.rowptr, w.col).update_backups(t)
        elif w.backups == "uniform":
            b = wl.uniform_backups(w, k + 1)[k]
        else:
            b = wl.fixed_backups(w)
        kept = orc.select_fastest(w.rowptr, w.col, t, b)
        orc.round_times(w.rowptr, w.col, t, b, kept)
        ws, we = orc.mixing_weights(w.rowptr, w.col, b, kept, w.weight_rule)
        t_discrete = time.perf_counter() - t0
    t_grad, n_grad = 0.0, 0
    if w.layers is not None and pool is None:
        means = wl.class_means(w)
        idx = wl.batch_indices(w, k)
        while n_grad < w.N and t_grad < budget_s / 2:
            i = n_grad
            f, l = wl.worker_dataset(w, i, means)
            x = wl.init_params(w, i)
            with _one_thread():
                t0 = time.perf_counter()
                orc.mlp_grad(x, w.layers, f[idx[i]], l[idx[i]])
                t_grad += time.perf_counter() - t0
            n_grad += 1
        t_grad_full = t_grad * w.N / n_grad
    elif w.layers is not None:
        per = max(1, min(w.N // procs, 2))
        jobs = [(config, overrides or {}, k, list(range(p * per, min(w.N, (p + 1) * per)))) for p in range(procs) if p * per < w.N]
        t_grad = max(pool.map(_grad_block_seconds, jobs))
        n_grad = sum(len(j[3]) for j in jobs)
        t_grad_full = t_grad * w.N / n_grad
    else:
        t_grad_full = 0.0
    cols = 1024
    t_mix, t_mix_full = 0.0, 0.0
    while True:
        cols = min(cols, w.d)
        if pool is None:
            X = rng.standard_normal((w.N, cols)).astype(np.float32)
            G = (0.01 * rng.standard_normal((w.N, cols))).astype(np.float32)
            with _one_thread():
                t0 = time.perf_counter()
                orc.mix_update(w.rowptr, w.col, X, G, ws, we, w.lr)
                t_mix = time.perf_counter() - t0
            done_cols = cols
        else:
            t_mix = max(pool.map(_mix_block_seconds, [(w.rowptr, w.col, ws, we, w.lr, w.N, cols, 1000 + p) for p in range(procs)]))
            done_cols = cols * procs
        t_mix_full = t_mix * w.d / min(done_cols, w.d)
        if done_cols >= w.d or t_mix > budget_s / 4:
            break
        cols *= 4
    desc = ("round %d on %s: selection/times/weights%s whole (%.3fs); gradients of %d of %d workers (%.2fs, scaled); "
            "mix on all %d rows x %d of %d columns (%.2fs, scaled)" %
            (k, "1 thread" if pool is None else "%d processes x 1 thread" % procs,
             "/threshold rule" if w.backups == "dtur" else "", t_discrete, n_grad, w.N, t_grad, w.N, min(done_cols, w.d), w.d, t_mix))
    return t_discrete + t_grad_full + t_mix_full, desc


def cpu_baseline(w, config, overrides, budget_s):
    """The oracle on this host: on one thread, and spread over all cores (processes started with spawn, since the
    CUDA context of this process must not be forked)."""
    import multiprocessing as mp
    sec1, desc1 = oracle_sample_seconds(w, 0, budget_s=budget_s)
    out = {"value": w.N / sec1, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc1}
    procs = max(1, min(os.cpu_count() or 1, 64))
    if procs > 1:
        try:
            with mp.get_context("spawn").Pool(procs) as pool:
                secp, descp = oracle_sample_seconds(w, 0, budget_s=budget_s, pool=pool, procs=procs, config=config, overrides=overrides)
            out["all_cores"] = {"value": w.N / secp, "unit": UNIT, "cores": procs, "sample": descp}
        except Exception as e:  # a host that cannot start the pool still reports the one-thread figure
            out["all_cores"] = {"error": repr(e)}
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.make_workload(args.config)
    # the whole run (warm-up included) is bounded to a minute or two of CPU work
    budget = min(args.ref_budget, 60.0 / (args.steps + args.warmup))
    for _ in range(args.warmup):
        oracle_sample_seconds(w, 0, budget_s=budget)
    est = []
    desc = ""
    for k in range(args.steps):
        s, desc = oracle_sample_seconds(w, k % w.rounds, budget_s=budget)
        est.append(s)
    sec = float(np.mean(est))
    value = w.N / sec
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "N": w.N, "d": w.d, "note": "CPU oracle, each step a bounded sample scaled to a full round"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# the GPU arm
# ------------------------------------------------------------------------------------------

def max_over_ranks(ms, dist, device="cuda"):
    """Slowest rank's time (every rank gets it); `dist` is torch.distributed or None."""
    if dist is None:
        return float(ms)
    import torch
    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def aggregate_value(units_per_rank_step, steps, ms_max, world, sharded=False):
    """Whole-job throughput: `world` replicas (all units processed / slowest rank's time), or, column-sharded,
    ONE simulation split over the ranks (its units / slowest rank's time)."""
    return (1 if sharded else world) * units_per_rank_step * steps / (ms_max * 1e-3)


def timed_loop(job, steps, fn, dist):
    import torch
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    return max_over_ranks(e0.elapsed_time(e1), dist)


def run_ours(args):
    import torch
    from paper_2102_06280_b200 import build, binding
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        torch.cuda.set_device(local)
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod
    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()
    overrides = {}
    if args.samples:
        overrides["samples"] = args.samples
    if args.width:
        overrides["d"] = args.width
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    col_range = None
    if args.shard == "columns":
        from paper_2102_06280_b200.sharding import column_shards
        full = wl.make_workload(args.config, **overrides)
        if full.layers is not None:
            raise SystemExit("--shard columns applies to the mix-only workloads (the gradients need whole rows)")
        col_range = column_shards(full.d, world)[rank]
    res = measure(args.config, local, args, dist, overrides, col_range)
    extra = {}
    # the whole hot path with a model (gradients on the tensor cores) next to the mix-only headline
    also = [c for c in (args.also or []) if c != args.config] if world == 1 and not overrides else []
    for c in also:
        extra[wl.CONFIGS[c]["name"]] = summary(measure(c, local, args, dist, {}), world, args)
    clocks = sampler.stop() if rank == 0 else None
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    w = res["w"]
    line = {"metric": METRIC, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "higher_is_better": True, "scaling": "strong" if args.shard == "columns" else "weak", "vs_baseline": None,
            "data": "synthetic"}
    line.update(summary(res, world, args))
    if overrides or col_range is not None or args.consensus_only:
        line["roofline"]["traffic"] = None
    if args.consensus_only:
        line["config"]["gradients"] = "none (consensus-only iterations: 8 B per element)"
    line["clocks"] = clocks
    if extra:
        line["other_workloads"] = extra
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, args.config, overrides, args.ref_budget)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def measure(config, local, args, dist, overrides, col_range=None):
    """Device-resident loop, stage times, launch count and the end-to-end loop of one workload."""
    import torch
    from paper_2102_06280_b200 import binding
    job = Job(config, device=local, col_range=col_range, consensus_only=getattr(args, "consensus_only", False), **overrides)
    if args.mix_panel is not None:
        job.h.set_mix_panel(args.mix_panel)
    for _ in range(args.warmup):
        job.step()
    torch.cuda.synchronize()
    job.h.profile(True)
    job.h.profile_read()
    launches0 = binding.launch_count()
    ms = timed_loop(job, args.steps, job.step, dist)
    launches = binding.launch_count() - launches0
    stage_ms, stage_rounds = job.h.profile_read()
    job.h.profile(False)
    graph_ms = None
    if args.graph and args.steps % args.graph == 0:
        # the same loop replayed from a CUDA graph of args.graph rounds (no stage events inside)
        job.capture(args.graph)
        job.step_graph()
        graph_ms = timed_loop(job, args.steps // args.graph, job.step_graph, dist)
    # end to end: per-round inputs from pinned host memory, results read back every round
    for _ in range(min(args.warmup, 3)):
        job.step_host()
    ms_e2e = timed_loop(job, args.steps, job.step_host, dist)
    out = dict(w=job.w, ld=job.ld, mix_kernel=job.h.mix_kernel(), graph_ms=graph_ms, ms=ms, ms_e2e=ms_e2e, launches=launches, status=job.h.status(),
               stage_ms={k: v / max(stage_rounds, 1) for k, v in stage_ms.items()},
               bytes=job.host_bytes_per_step(), mix_bytes=job.mix_bytes_per_launch(),
               kept_last=int(job.kept.sum().item()), sms=torch.cuda.get_device_properties(local).multi_processor_count)
    job.close()
    del job
    torch.cuda.empty_cache()
    return out


def model_flops_per_round(w):
    """Dense-layer flops of one round: forward + dW (2 each per weight and sample) + dA for layers above the first."""
    if w.layers is None:
        return 0
    dims = wl.layer_dims(w.layers)
    per_sample = sum(4 * o * i for o, i in dims) + sum(2 * o * i for o, i in dims[1:])
    return per_sample * w.batch * w.N


def tensor_core_gemm_work(w):
    """(flops, bytes) of the tensor-core GEMM launches of one round: forward, dW and (above the first layer) dA of
    every layer but the last.  Bytes = what each launch must move once: its two bf16 operands, its output (bf16
    activations / dZ, fp32 dW into G), the fp32 bias or the bf16 ReLU mask."""
    if w.layers is None or w.precision != "bf16":
        return 0, 0
    dims = wl.layer_dims(w.layers)          # [(out, in)] per layer
    B, flops, nbytes = w.batch, 0, 0
    for l, (o, i) in enumerate(dims[:-1]):
        flops += 2 * B * i * o * 2                                   # forward, dW
        nbytes += (B * i * 2 + i * o * 2 + B * o * 2 + o * 4)        # forward: A_l, W_l, A_{l+1}, bias
        nbytes += (B * o * 2 + B * i * 2 + i * o * 4)                # dW: dZ_{l+1}, A_l, fp32 dW
        if l >= 1:
            flops += 2 * B * i * o                                   # dA
            nbytes += (B * o * 2 + i * o * 2 + B * i * 2 + B * i * 2)  # dA: dZ_{l+1}, W_l, mask A_l, dZ_l
    return flops * w.N, nbytes * w.N


def summary(res, world, args):
    w = res["w"]
    peaks, peak_kind = measured_peaks()
    mix_ms = res["stage_ms"]["mix"]
    achieved = res["mix_bytes"] / (mix_ms * 1e-3) / 1e9 if mix_ms > 0 else 0.0
    h2d, d2h = res["bytes"]
    sharded = getattr(args, "shard", "none") == "columns"
    out = {"value": aggregate_value(w.N, args.steps, res["ms"], world, sharded), "ms_per_step": res["ms"] / args.steps,
           "dtype": "f32" if w.precision == "fp32" else "bf16",
           "config": {"workload": w.name, "N": w.N, "d": w.d, "ld": res["ld"], "nnz": int(len(w.col)),
                      "batch": w.batch, "layers": w.layers, "backups": w.backups, "weights": w.weight_rule,
                      "precision": "fp32" if w.precision == "fp32" else "bf16 operands, fp32 accumulate, fp32 master and mix",
                      "l2": "inputs larger than L2 (X and G each %.2f GB)" % (w.N * res["ld"] * 4 / 1e9)
                            if w.N * res["ld"] * 4 > 126e6 else "working set smaller than L2: cache-resident by design",
                      "multi_gpu": ("one simulation, X split by columns over %d ranks, no exchange (this rank: %d columns)" % (world, res["ld"])
                                    if sharded else "replicas only" if world > 1 else "single GPU")},
           "stage_ms": res["stage_ms"],
           "e2e": {"value": aggregate_value(w.N, args.steps, res["ms_e2e"], world, sharded), "unit": UNIT,
                   "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": res["ms_e2e"] / args.steps},
           "gpu_launches": int(res["launches"]),
           "roofline": {"kernel": res["mix_kernel"], "bound": "hbm",
                        "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                        "peak_kind": "of " + peak_kind, "frac_of_8TBps_nominal": achieved / 8000.0,
                        "traffic": (MIX_TRAFFIC_BYTES[w.index][1] if w.index in MIX_TRAFFIC_BYTES and
                                    MIX_TRAFFIC_BYTES[w.index][0] == res["mix_kernel"] else None),
                        "bytes_per_launch": res["mix_bytes"], "ms_per_launch": mix_ms},
           "device_status": res["status"]}
    # The second roofline of the mix: every output element needs (1 + kept neighbours) fp32 operands out
    # of on-chip storage; shared memory delivers 128 bytes per clock and SM.  With ~30 terms per output
    # (the mix-only workload) this bound, not HBM, is the binding one.
    smem_peak = 128.0 * res["sms"] * peaks.get("sm_max_mhz", 1965.0) * 1e6 / 1e9
    operand_bytes = 4.0 * (w.N + res["kept_last"]) * res["ld"]
    operand_rate = operand_bytes / (mix_ms * 1e-3) / 1e9 if mix_ms > 0 else 0.0
    out["roofline"]["operand_delivery"] = {
        "terms_per_output": 1.0 + res["kept_last"] / w.N, "bytes_per_launch": operand_bytes, "achieved": operand_rate,
        "peak": smem_peak, "unit": "GB/s", "frac": operand_rate / smem_peak,
        "peak_kind": "128 B/clk/SM x %d SMs x %.0f MHz (shared-memory data pipe, nominal)" % (res["sms"], peaks.get("sm_max_mhz", 1965.0))}
    if mix_ms <= 0:   # the whole round was one launch (small fp32 networks): there is no mix stage of its own to rate
        out["roofline"].update({"kernel": "round_fused_kernel", "achieved": None, "frac": None, "frac_of_8TBps_nominal": None,
                                "note": "one cooperative launch per round; launch-bound, no separate mix kernel"})
        out["roofline"]["operand_delivery"].update({"achieved": None, "frac": None})
    if res.get("graph_ms"):
        out["cuda_graph"] = {"rounds_per_graph": args.graph, "ms_per_step": res["graph_ms"] / args.steps,
                             "value": aggregate_value(w.N, args.steps, res["graph_ms"], world, sharded),
                             "note": "same rounds replayed from one CUDA graph per %d rounds" % args.graph}
    flops = model_flops_per_round(w)
    if flops and res["stage_ms"]["grad"] > 0:
        out["gradients"] = {"dense_flop_per_round": flops,
                            "tflops_over_grad_stage": flops / (res["stage_ms"]["grad"] * 1e-3) / 1e12,
                            "note": "grad stage = gather, casts, GEMMs, loss and last layer together"}
    tc_flops, tc_bytes = tensor_core_gemm_work(w)
    gemm_ms = res["stage_ms"].get("gemm", 0.0)
    if tc_flops and gemm_ms > 0:
        # The dense layers' GEMMs (batch 128-256 per worker) stream their weights or their fp32 result once: they sit
        # between the two rooflines, so both are reported: flops over the tensor peak a long step sustains, and
        # the bytes each launch must move over the copy bandwidth.
        tf = tc_flops / (gemm_ms * 1e-3) / 1e12
        gbs = tc_bytes / (gemm_ms * 1e-3) / 1e9
        peak_tf = peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops"))
        out["roofline_gemm"] = {"kernel": "gemm_tc_kernel (all tensor-core launches of a round)", "ms_per_round": gemm_ms,
                                "flop_per_round": tc_flops, "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s",
                                "frac": tf / peak_tf, "peak_kind": "sustained bf16, of " + peak_kind,
                                "hbm_bytes_per_round": tc_bytes, "achieved_gbs": gbs, "frac_hbm": gbs / peaks["hbm_gbs"],
                                "bound": "hbm" if gbs / peaks["hbm_gbs"] > tf / peak_tf else "tensor"}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=DEFAULT_CONFIG, choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-budget", type=float, default=12.0, help="seconds of CPU oracle work per sampled step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--also", type=int, nargs="*", default=[3], choices=sorted(wl.CONFIGS),
                    help="further workloads summarised under other_workloads (single GPU only)")
    ap.add_argument("--graph", type=int, default=0,
                    help="also time the loop replayed from CUDA graphs of this many rounds (must divide --steps)")
    ap.add_argument("--mix-panel", type=int, default=None,
                    help="expert knob passed to dbw_set_mix_panel (1 = staged kernel, 2 = tensor-core kernel, 16..128 = panel width)")
    ap.add_argument("--consensus-only", action="store_true",
                    help="mix-only workloads: consensus-only iterations (G = 0, nothing of G read): 8 bytes per element")
    ap.add_argument("--shard", default="none", choices=["none", "columns"],
                    help="columns: ONE mix-only simulation split over the ranks by columns of X (no exchange; selection "
                         "replicated; strong scaling) instead of one replica per rank")
    ap.add_argument("--samples", type=int, default=0, help="profiling aid: samples per worker instead of the config's")
    ap.add_argument("--width", type=int, default=0, help="profiling aid: columns d of the mix-only config instead of 2^20")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
