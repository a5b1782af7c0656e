"""cb-DyBW against cb-Full on the paper-shaped synthetic workloads (Section 5, Appendix B).

    python -m paper_2102_06280_b200.experiments --config 6 --rounds 60 [--bf16]

Runs the same seeded workload twice on the GPU through the C-ABI library: once with the
backup counts set by the threshold rule (`dbw_update_backups`, cb-DyBW) and once with b = 0
(every worker waits for all its neighbours, cb-Full), and reports what the paper's figures
plot: training loss per iteration, the virtual duration of every iteration (T(k) of Section
3.2.2), the number of backup workers, and the virtual time needed to reach a loss level.
Real MNIST / CIFAR-10 are not available; the data are the Gaussian-mixture stand-ins of
`workloads`, so only the shape of the result is comparable with the paper.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
from typing import Dict, Optional

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def run(config: int, rounds: Optional[int] = None, dynamic: bool = True, bf16: bool = False, device: int = 0,
        lagged: bool = False, **overrides) -> Dict[str, np.ndarray]:
    """One training run; returns per-round arrays: loss (mean over workers), T_round, backups (mean b).

    `lagged`: the backup counts of iteration k come from the arrival times of iteration k-1 (set after
    that iteration, as Algorithm 1 is printed) instead of from the times of the iteration about to run."""
    import torch
    from workloads import configs as wl
    from . import binding as p

    torch.cuda.set_device(device)
    w = wl.make_workload(config, **overrides)
    rounds = rounds or w.rounds
    m = p.model_layout(w.layers, w.batch)
    h = p.Dbw(w.rowptr, w.col, d=m.d, model=m, flags=p.GEMM_BF16 if bf16 else 0, device=device)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    means = wl.class_means(w)
    data = [wl.worker_dataset(w, i, means) for i in range(w.N)]
    feat, labels = dev(np.stack([f for f, _ in data])), dev(np.stack([l for _, l in data]))
    h.set_dataset(feat, labels, w.samples)
    h.set_param_tracking(True)
    X = dev(m.pack(np.stack([wl.init_params(w, i) for i in range(w.N)])))
    times = dev(wl.arrival_times(w, rounds))
    n, nnz = w.N, len(w.col)
    kept = torch.zeros(nnz, dtype=torch.uint8, device="cuda")
    b = torch.zeros(n, dtype=torch.int32, device="cuda")
    Tr = torch.zeros(rounds, dtype=torch.float64, device="cuda")
    loss = torch.zeros(rounds, n, device="cuda")
    bs = torch.zeros(rounds, n, dtype=torch.int32, device="cuda")
    for k in range(rounds):
        if dynamic and k > 0:                 # Algorithm 1: the first iteration waits for every neighbour
            h.update_backups(times[k - 1] if lagged else times[k], b)
        bs[k].copy_(b)
        h.round(X, times[k], b, wl.learning_rate(w, k), X, kept, batch_idx=dev(wl.batch_indices(w, k)),
                T_round=Tr[k:k + 1], loss=loss[k])
    torch.cuda.synchronize()
    status = h.status()
    h.close()
    if status:
        raise RuntimeError("device status %d" % status)
    return {"loss": loss.mean(dim=1).cpu().numpy(), "T_round": Tr.cpu().numpy(),
            "backups": bs.float().mean(dim=1).cpu().numpy(), "X": X.cpu().numpy()}


def time_to_loss(res: Dict[str, np.ndarray], level: float) -> float:
    """Virtual time at which the (running-minimum) training loss first reaches `level` (inf if never)."""
    clock = np.cumsum(res["T_round"])
    hit = np.nonzero(np.minimum.accumulate(res["loss"]) <= level)[0]
    return float(clock[hit[0]]) if len(hit) else float("inf")


def compare(config: int, rounds: Optional[int] = None, bf16: bool = False, **overrides) -> dict:
    dy = run(config, rounds, dynamic=True, bf16=bf16, **overrides)
    full = run(config, rounds, dynamic=False, bf16=bf16, **overrides)
    level = float(max(dy["loss"][-1], full["loss"][-1]) * 1.05)      # a level both runs reach
    t_dy, t_full = time_to_loss(dy, level), time_to_loss(full, level)
    return {"rounds": len(dy["loss"]),
            "mean_round_duration": {"cb-DyBW": float(dy["T_round"].mean()), "cb-Full": float(full["T_round"].mean()),
                                    "reduction": float(1.0 - dy["T_round"].mean() / full["T_round"].mean())},
            "final_loss": {"cb-DyBW": float(dy["loss"][-1]), "cb-Full": float(full["loss"][-1])},
            "mean_backups": float(dy["backups"].mean()),
            "time_to_loss": {"level": level, "cb-DyBW": t_dy, "cb-Full": t_full,
                             "reduction": float(1.0 - t_dy / t_full) if np.isfinite(t_full) and t_full > 0 else None}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=6)
    ap.add_argument("--rounds", type=int, default=0)
    ap.add_argument("--bf16", action="store_true")
    args = ap.parse_args()
    print(json.dumps(compare(args.config, args.rounds or None, args.bf16), indent=1))


if __name__ == "__main__":
    main()
