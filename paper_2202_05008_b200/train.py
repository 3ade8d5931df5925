"""A minimal training loop over the three calls (the paper's trainer, Section 2, reduced to its
core: ask -> rollout -> tell, with the best and mean fitness per generation read back).

    python -m paper_2202_05008_b200.train --workload cfg2 --generations 200
"""
from __future__ import annotations

import argparse
import time
from typing import List, Optional, Tuple

import torch

from . import workloads as W
from .binding import Solver


def run(workload: W.Workload, generations: int, device="cuda:0", log_every: int = 0,
        fixed_batch: bool = False, initial_center: Optional[torch.Tensor] = None,
        target: Optional[torch.Tensor] = None, **cfg_kw) -> Tuple[Solver, List[Tuple[float, float]]]:
    """Runs `generations` generations; returns the solver and [(mean fitness, best fitness)]."""
    s = Solver(workload, device=device, **cfg_kw)
    if initial_center is not None:
        s.set_state(center=initial_center.to(s.device).contiguous())
    if workload.task_kind == W.TASK_PAINT:
        if target is None:
            width, height = int(workload.task_param[0]), int(workload.task_param[1])
            target = torch.tensor(W.paint_target(workload.seed, width, height), device=s.device)
        s.set_target(target)
    history = []
    fitness = torch.empty(workload.pop_size, dtype=torch.float32, device=s.device)
    for g in range(generations):
        if workload.task_kind == W.TASK_SUPERVISED:
            images, labels = W.image_batch(workload.seed, 0 if fixed_batch else g, workload.batch)
            s.set_batch(torch.tensor(images, device=s.device), torch.tensor(labels, device=s.device))
        s.ask()
        s.rollout(fitness=fitness)
        s.tell(fitness)
        mean, best = float(fitness.mean()), float(fitness.max())      # synchronises
        history.append((mean, best))
        if log_every and (g % log_every == 0 or g == generations - 1):
            print(f"generation {g:5d}  mean fitness {mean:12.4f}  best {best:12.4f}")
    status = s.sync_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after training")
    return s, history


def main(argv: Optional[List[str]] = None) -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg2", choices=sorted(W.CONFIGS))
    ap.add_argument("--generations", type=int, default=100)
    ap.add_argument("--log-every", type=int, default=10)
    ap.add_argument("--clipup", action="store_true", help="ClipUp instead of Adam")
    ap.add_argument("--adapt-sigma", action="store_true", help="PGPE sigma update")
    a = ap.parse_args(argv)
    w = W.CONFIGS[a.workload]
    if w.task_kind == W.TASK_NONE:
        raise SystemExit("this workload has no task to train on")
    w = w.with_(optimizer=W.OPT_CLIPUP if a.clipup else W.OPT_ADAM,
                sigma_mode=W.SIGMA_PGPE if a.adapt_sigma else W.SIGMA_CONSTANT)
    t0 = time.perf_counter()
    _, hist = run(w, a.generations, log_every=a.log_every)
    dt = time.perf_counter() - t0
    print(f"{a.generations} generations in {dt:.2f} s ({a.generations / dt:.1f} generations/s incl. read-backs); "
          f"mean fitness {hist[0][0]:.4f} -> {hist[-1][0]:.4f}")


if __name__ == "__main__":
    main()
