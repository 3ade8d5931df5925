#!/usr/bin/env python
"""Benchmark of one evolution-strategy generation (ask -> rollout -> tell) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl ours|reference]

One "step" is one whole generation of the workload.  Prints ONE JSON line (rank 0).
For N > 1 (launched by torch.distributed.run) every rank runs an independent solver on its own
GPU with its own seed (replicas; the generation itself needs no exchange on one GPU), timing is
the max over ranks and the value is the sum of the work of all ranks.

`--impl reference` times the CPU oracle (single-threaded C, fp64) on a bounded sample of the same
workload; it is a deliberately slow, plain program and serves as a baseline only.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

FP32_LANES_PER_SM = 128
L2_FLUSH_BYTES = 256 << 20


# ------------------------------------------------------------------------------------------
# workload arithmetic (algorithmic work per generation)
# ------------------------------------------------------------------------------------------
def mlp_macs(sizes):
    return sum(a * b for a, b in zip(sizes[:-1], sizes[1:]))


def rollout_flops_per_env_step(w):
    from paper_2202_05008_b200 import workloads as W
    if w.task_kind == W.TASK_SUPERVISED:
        return 645120.0                       # conv1 230,400 + conv2 409,600 + fc 5,120 (2 x MAC)
    if w.task_kind == W.TASK_PAINT:               # per member: every pixel against every triangle,
        n_tri = w.param_dim // 10                 # 3 edges x 5 flop + 3 blends x 2 flop
        return 21.0 * n_tri * w.task_param[0] * w.task_param[1]
    if w.task_kind == W.TASK_SEQ2SEQ_ADD:         # per query: every LSTM step + the read-out steps
        h, nd = w.layer_sizes[0], int(w.task_param[0])
        return 2.0 * ((3 * nd + 2) * 4 * h * (h + 12 + 1) + (nd + 1) * 12 * h)
    macs = mlp_macs(w.layer_sizes)
    if w.task_kind == W.TASK_TANH_LINEAR:
        macs += 28 * 28 + 28 * 8              # the task's own x' = tanh(Ax + Ba)
    return 2.0 * macs


def stage_work(w, stored):
    """Algorithmic bytes / flops of each stage of one generation."""
    P, D = w.pop_size, w.param_dim
    H = P // 2
    ask_bytes = 4.0 * P * D + (4.0 * H * D if stored else 0.0) + 4.0 * D
    tell_bytes = (4.0 * H * D if stored else 0.0) + 28.0 * D + 8.0 * P
    rollout_flops = rollout_flops_per_env_step(w) * w.env_steps_per_generation
    return {"ask_bytes": ask_bytes, "tell_bytes": tell_bytes, "rollout_flops": rollout_flops}


# DRAM bytes (read + write) of the dominant kernel per launch, from the ncu captures summarised
# under profiles/ (same workload, same kernel).  An entry is dropped (-> null) when its kernel
# changes after the capture.
NCU_TRAFFIC_BYTES = {
    ("cfg2", "stored"): ("k_rollout_cartpole_ws", 4.783360e6),
    ("cfg2", "regenerated"): ("k_rollout_cartpole_ws", 4.783360e6),
    ("cfg3", "stored"): ("k_cnn_conv2_tc", 152.721664e6 + 3.863040e6),
    ("cfg4", "stored"): ("k_rollout_mlp_tiled", 350.257664e6 + 5.215232e6),
    ("cfg4", "regenerated"): ("k_rollout_mlp_tiled", 350.257664e6 + 5.215232e6),
    ("cfg5", "stored"): ("k_ask", 32 * (3.161160e9 + 0.000273e9)),       # reduced-D capture scaled by D
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls NVML for SM clock and throttle reasons while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index):
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self.h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def sample(self):
        if self.h is None:
            return
        try:
            self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
            self.reason_bits |= int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
        except Exception:
            try:
                self.reason_bits |= int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            except Exception:
                pass

    def _run(self):
        while not self._stop.is_set():
            self.sample()
            time.sleep(0.02)

    def start(self):
        if self.h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------
def _oracle_member_rollout(w, generation):
    """Returns f(row) -> fitness of one member through the oracle's rollout for this workload."""
    import oracle
    from paper_2202_05008_b200 import workloads as W
    if w.task_kind == W.TASK_SUPERVISED:
        images, labels = W.image_batch(w.seed, generation, w.batch)
        return lambda row: oracle.cnn_fitness(row, images, labels, True)
    if w.task_kind == W.TASK_CARTPOLE:
        tp = w.task_param
        p = oracle.cartpole_params(tp[0], tp[1], tp[2], tp[3], tp[4])
        return lambda row: oracle.rollout_cartpole(row, w.layer_sizes, w.action_scale, p, tp[5], w.seed,
                                                   generation, w.episodes, w.horizon)[0]
    if w.task_kind == W.TASK_PAINT:
        width, height, bg = int(w.task_param[0]), int(w.task_param[1]), w.task_param[2]
        target = W.paint_target(w.seed, width, height)
        return lambda row: oracle.paint_fitness(row.reshape(-1, 10), width, height, target, bg)
    if w.task_kind == W.TASK_SEQ2SEQ_ADD:
        h, nd = w.layer_sizes[0], int(w.task_param[0])
        enc, dec, tgt = oracle.seq2seq_queries(w.seed, generation, w.batch, nd)
        return lambda row: oracle.seq2seq_fitness(row, h, nd, enc, dec, tgt, True)[0]
    A, B = oracle.tanh_linear_constants(w.seed)
    return lambda row: oracle.rollout_tanh_linear(row, w.layer_sizes, w.action_scale, A, B, w.seed,
                                                  generation, w.episodes, w.horizon)[0]


def oracle_generation_sample(w, n_members, generation=0, threads=1):
    """Times the oracle on ask + tell for the whole population (a column sample for very wide
    problems) and the rollout of n_members members; returns seconds for a full generation
    extrapolated linearly (members and columns are independent).  threads > 1 spreads the
    members' rollouts (unchanged oracle code, one member per call) over host threads; ask and
    tell stay on one thread."""
    import oracle
    from paper_2202_05008_b200 import workloads as W
    P, D = w.pop_size, w.param_dim
    cols = D if P * D <= 50_000_000 else 4096
    t0 = time.perf_counter()
    theta, eps = oracle.ask(w.seed, generation, P, cols, np.zeros(cols, np.float32), w.sigma)
    t_ask = (time.perf_counter() - t0) * (D / cols)
    t_roll, n_done = 0.0, 0
    fitness = W.synthetic_fitness(w.seed, generation, P)
    if w.task_kind != W.TASK_NONE:
        full = np.zeros((n_members, D), dtype=np.float32)
        if cols == D:
            full[:] = theta[:n_members]
        f = _oracle_member_rollout(w, generation)
        t0 = time.perf_counter()
        if threads > 1:
            from concurrent.futures import ThreadPoolExecutor
            with ThreadPoolExecutor(threads) as pool:      # the C oracle runs without the interpreter lock
                fitness[:n_members] = list(pool.map(f, [full[m] for m in range(n_members)]))
        else:
            for m in range(n_members):
                fitness[m] = f(full[m])
        t_roll = (time.perf_counter() - t0) * (P / n_members)
        n_done = n_members
    t0 = time.perf_counter()
    _, u, _ = oracle.centered_rank(fitness)
    g = oracle.gradient(u, eps, w.sigma)
    oracle.adam(np.zeros(cols), np.zeros(cols), np.zeros(cols), g, 1, w.lr)
    t_tell = (time.perf_counter() - t0) * (D / cols)
    sample = (f"ask+tell on all {P} members x {cols} of {D} columns; rollout of {n_done} of {P} members "
              f"x {w.episodes} episodes x {w.horizon} steps; scaled linearly to one generation")
    return t_ask + t_roll + t_tell, sample


def unit_of(w):
    from paper_2202_05008_b200 import workloads as W
    if w.task_kind == W.TASK_NONE:
        return "generations_per_sec", "generations/s", 1.0
    return "env_steps_per_sec", "env-steps/s", float(w.env_steps_per_generation)


def members_for_budget(w, seconds):
    """Members whose oracle rollout takes about `seconds` (from a one-member probe)."""
    from paper_2202_05008_b200 import workloads as W
    if w.task_kind == W.TASK_NONE:
        return 0
    t, _ = oracle_generation_sample(w.with_(pop_size=2, param_dim=w.param_dim), 1)
    per_member = max(t / 2.0, 1e-4)
    return int(max(1, min(w.pop_size, seconds / per_member)))


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    metric, unit, units_per_gen = unit_of(w)
    # per-step sample sized so that warm-up + timed steps take about two minutes in all
    n = members_for_budget(w, min(1.0, 120.0 / max(1, args.warmup + args.steps)))
    times, sample = [], ""
    for i in range(args.warmup + args.steps):
        t, sample = oracle_generation_sample(w, max(n, 1), generation=i)
        if i >= args.warmup:
            times.append(t)
    t_step = sum(times) / len(times)
    value = units_per_gen / t_step
    line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(w, args, stored=True),
            "generations_per_sec": 1.0 / t_step,
            "cpu_baseline": {"value": value, "unit": unit, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def config_of(w, args, stored):
    from paper_2202_05008_b200 import workloads as W
    task = {W.TASK_NONE: "none", W.TASK_CARTPOLE: "cartpole_swingup", W.TASK_TANH_LINEAR: "tanh_linear",
            W.TASK_SUPERVISED: "supervised_28x28", W.TASK_SEQ2SEQ_ADD: "seq2seq_addition",
            W.TASK_PAINT: f"triangle_painting_{int(w.task_param[0]) if w.task_param else 0}x{int(w.task_param[1]) if len(w.task_param) > 1 else 0}"}[w.task_kind]
    return {"workload": w.name, "pop_size": w.pop_size, "param_dim": w.param_dim, "task": task,
            "policy": "mlp " + "-".join(map(str, w.layer_sizes)) if w.policy_kind == W.POLICY_MLP else
                      {W.POLICY_CNN_28: "cnn_28",
                       W.POLICY_LSTM_SEQ2SEQ: f"lstm_encoder_decoder h={w.layer_sizes[0] if w.layer_sizes else 0}"
                       }.get(w.policy_kind, "none"),
            "episodes": w.episodes, "horizon": w.horizon, "batch": w.batch,
            "noise": "stored" if stored else "regenerated",
            "parallelism": f"{'one population, pair shards' if args.sharded else 'replicas'} x{args.gpus}",
            "l2": "flushed between timed steps (256 MiB write, untimed)"}


# ------------------------------------------------------------------------------------------
# cross-rank plumbing (works with gloo on CPU tensors and nccl on CUDA tensors)
# ------------------------------------------------------------------------------------------
def rank_seed(base_seed: int, rank: int) -> int:
    """Replicas are independent problems: every rank gets its own random streams."""
    return base_seed + 1000 * rank


def max_over_ranks(value_ms: float, device, world: int) -> float:
    """Timing of a multi-rank run is the slowest rank's."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank_step: float, world: int, ms_per_step: float, sharded: bool = False) -> float:
    """Aggregate throughput of all ranks.  Replicas (weak scaling): every rank does one full
    generation.  Pair shards (strong scaling): all ranks together do one generation."""
    return (1 if sharded else world) * units_per_rank_step / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------
def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2202_05008_b200 import Solver, sharded, workloads as W
    from paper_2202_05008_b200.binding import fma_probe

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the GPU arm has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    stored = args.noise == "stored"
    if args.sharded:                                    # one population, rank r owns a range of pairs
        first_pair, n_pairs = sharded.shard_of(w.pop_size // 2, rank, world)
        w_rank = w
        s = Solver(w_rank, device=dev, noise_mode=W.NOISE_STORED if stored else W.NOISE_REGENERATED,
                   shard_first_pair=first_pair, shard_pairs=n_pairs)
    else:
        w_rank = w.with_(seed=rank_seed(w.seed, rank))  # independent replicas
        s = Solver(w_rank, device=dev, noise_mode=W.NOISE_STORED if stored else W.NOISE_REGENERATED)
    P, D = s.P, w.param_dim                             # P = members this rank evaluates
    supervised = w.task_kind == W.TASK_SUPERVISED
    no_task = w.task_kind == W.TASK_NONE
    fitness = torch.empty(P, dtype=torch.float32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    if supervised:
        batches = []
        for g in range(4):
            im, lb = W.image_batch(w_rank.seed, g, w.batch)
            batches.append((torch.tensor(im, device=dev), torch.tensor(lb, device=dev)))
    if w.task_kind == W.TASK_PAINT:
        d_target = torch.tensor(W.paint_target(w_rank.seed, int(w.task_param[0]), int(w.task_param[1])), device=dev)
        s.set_target(d_target)
    if no_task:
        fits = [torch.tensor(W.synthetic_fitness(w_rank.seed, g, s.P_global), device=dev) for g in range(4)]
        if args.sharded:
            fits = [f[2 * first_pair:2 * (first_pair + n_pairs)].contiguous() for f in fits]

    def tell(f):
        if not args.sharded:
            s.tell(f)
            return
        s.tell_begin(sharded.gather_fitness(f, world))
        sharded.reduce_sums(*s.reduce_buffers(), world)
        s.tell_end()

    def generation(i, ev=None):
        if ev: ev[0].record()
        s.ask()
        if ev: ev[1].record()
        if supervised:
            s.set_batch(*batches[i % 4])
        if no_task:
            f = fits[i % 4]
        else:
            f = s.rollout(fitness=fitness)
        if ev: ev[2].record()
        tell(f)
        if ev: ev[3].record()

    for i in range(args.warmup):
        flush.fill_(i & 255)
        generation(i)
    torch.cuda.synchronize()
    if s.sync_status() != 0:
        raise SystemExit("bench.py: device status not ok after warm-up")

    sampler = ClockSampler(local)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    launches0 = s.launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    for i in range(args.steps):
        flush.fill_(i & 255)                            # evict L2 (untimed)
        generation(args.warmup + i, events[i])
    sampler.sample()
    torch.cuda.synchronize()
    sampler.stop()
    if world > 1:
        dist.barrier()
    launches = s.launch_count() - launches0
    status = s.sync_status()
    if status != 0:
        raise SystemExit(f"bench.py: device status {status} after the timed region")

    t_ask = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
    t_roll = sum(e[1].elapsed_time(e[2]) for e in events) / args.steps
    t_tell = sum(e[2].elapsed_time(e[3]) for e in events) / args.steps
    per_step = sorted(e[0].elapsed_time(e[3]) for e in events)
    t_total_ms = sum(per_step)
    t_step_ms = max_over_ranks(t_total_ms, dev, world) / args.steps

    # ---- end to end: host-resident centre in, fitness and centre out, every step -----------
    h_center = torch.zeros(D, dtype=torch.float32).pin_memory()
    h_fit = torch.zeros(P, dtype=torch.float32).pin_memory()
    d_center = torch.zeros(D, dtype=torch.float32, device=dev)
    if supervised:
        h_batches = [(b[0].cpu().pin_memory(), b[1].cpu().pin_memory()) for b in batches]
        d_im = torch.empty_like(batches[0][0]); d_lb = torch.empty_like(batches[0][1])
    if no_task:
        h_fits = [f.cpu().pin_memory() for f in fits]
    h_center.copy_(s.center().cpu())
    gen0, t0_adam = s.counters()
    e2e_steps = max(3, min(args.steps, 50))
    h2d = 4 * D + (w.batch * (784 * 4 + 4) if supervised else 0) + (4 * P if no_task else 0)
    d2h = 4 * D + 4 * P

    def e2e_step(i):
        d_center.copy_(h_center, non_blocking=True)
        s.set_state(center=d_center, generation=gen0 + i, adam_step=t0_adam + i)
        s.ask()
        if supervised:
            d_im.copy_(h_batches[i % 4][0], non_blocking=True)
            d_lb.copy_(h_batches[i % 4][1], non_blocking=True)
            s.set_batch(d_im, d_lb)
        if no_task:
            fitness.copy_(h_fits[i % 4], non_blocking=True)
        else:
            s.rollout(fitness=fitness)
        tell(fitness)
        h_fit.copy_(fitness, non_blocking=True)
        h_center.copy_(s.center(), non_blocking=True)
        torch.cuda.current_stream().synchronize()

    e2e_step(0)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(1, e2e_steps + 1):
        e2e_step(i)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, dev, world)

    # ---- optional: the same generation replayed from a CUDA graph (no host launch cost) ---------
    graph_ms = None
    if args.graph and not args.sharded and not no_task:
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            sg = Solver(w_rank, device=dev, stream=side,
                        noise_mode=W.NOISE_STORED if stored else W.NOISE_REGENERATED)
            if supervised:
                sg.set_batch(*batches[0])
            if w.task_kind == W.TASK_PAINT:
                sg.set_target(d_target)
            gfit = torch.empty(P, dtype=torch.float32, device=dev)
            for _ in range(max(args.warmup, 3)):
                sg.ask(); sg.rollout(fitness=gfit); sg.tell(gfit)
            graph = sg.capture_generation(gfit)
            gev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
            graph.replay()
            side.synchronize()
            for i in range(args.steps):
                flush.fill_(i & 255)
                gev[i][0].record(side)
                graph.replay()
                gev[i][1].record(side)
            side.synchronize()
            if sg.sync_status() != 0:
                raise SystemExit("bench.py: device status not ok after the graph replays")
            graph_ms = max_over_ranks(sum(a.elapsed_time(b) for a, b in gev), dev, world) / args.steps
            sg.close()

    if rank == 0:
        metric, unit, units_per_gen = unit_of(w)
        value = whole_job_value(units_per_gen, world, t_step_ms, args.sharded)
        peaks = measured_peaks()
        clocks = sampler.summary()
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        max_mhz = clocks["sm_max_mhz"] or 1965
        work = stage_work(w.with_(pop_size=P) if args.sharded else w, stored)   # this rank's share
        alu_peak = sm_count * FP32_LANES_PER_SM * 2 * max_mhz * 1e6 / 1e12      # TFLOP/s fp32 FMA
        stages = {
            "ask": {"ms": t_ask, "GB/s": work["ask_bytes"] / (t_ask * 1e-3) / 1e9},
            "rollout": {"ms": t_roll, "TFLOP/s": work["rollout_flops"] / (t_roll * 1e-3) / 1e12 if t_roll > 0 else 0.0},
            "tell": {"ms": t_tell, "GB/s": work["tell_bytes"] / (t_tell * 1e-3) / 1e9},
        }
        traffic_entry = NCU_TRAFFIC_BYTES.get((args.workload, args.noise)) if not (args.pop or args.dim) else None
        if no_task:
            dom = "ask" if t_ask >= t_tell else "tell"
            achieved = stages[dom]["GB/s"]
            roofline = {"kernel": "k_ask" if dom == "ask" else "k_grad_partial", "bound": "hbm",
                        "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                        "traffic": None}
        elif supervised or w.task_kind == W.TASK_SEQ2SEQ_ADD:
            achieved = stages["rollout"]["TFLOP/s"]
            roofline = {"kernel": "k_cnn_conv1_tc + k_cnn_conv2_tc" if supervised else "k_s2s_tc",
                        "bound": "tensor", "achieved": achieved,
                        "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                        "frac": achieved / peaks["bf16_tflops"], "peak_source": peaks["source"],
                        "traffic": None}
        else:
            achieved = stages["rollout"]["TFLOP/s"]
            fma_measured = fma_probe(dev)                 # register-only FMA chains, timed alone
            roofline = {"kernel": "k_paint" if w.task_kind == W.TASK_PAINT else "k_rollout_mlp (tiled / warp-specialised)", "bound": "alu", "achieved": achieved, "peak": alu_peak,
                        "unit": "TFLOP/s", "frac": achieved / alu_peak,
                        "peak_source": f"{sm_count} SMs x 128 fp32 lanes x 2 x {max_mhz} MHz",
                        "peak_measured": fma_measured, "frac_of_measured": achieved / fma_measured,
                        "peak_measured_source": "evo_fma_probe (16 FMA chains per thread, best of 5 launches)",
                        "traffic": None}
            if w.task_kind == W.TASK_PAINT:
                roofline["note"] = ("algorithmic flop = every pixel against every triangle; the kernel skips the pairs "
                                    "outside a triangle's bounding box, so this is an equivalent rate, not pipe utilisation")
        if traffic_entry is not None and (not no_task or roofline["kernel"] == traffic_entry[0]):
            roofline["traffic"] = traffic_entry[1]
            roofline["traffic_kernel"] = traffic_entry[0]
        cpu = None
        if not args.skip_cpu_baseline:
            n = members_for_budget(w, 12.0)
            t_cpu, sample = oracle_generation_sample(w, max(n, 1))
            cpu = {"value": units_per_gen / t_cpu, "unit": unit, "cores": 1, "kind": "oracle",
                   "sample": sample}
            cores = len(os.sched_getaffinity(0))
            if cores > 1 and not no_task:                  # same oracle, members spread over the host's cores
                n_all = min(w.pop_size, max(n, 1) * cores)
                t_all, sample_all = oracle_generation_sample(w, n_all, threads=cores)
                cpu["all_cores"] = {"value": units_per_gen / t_all, "unit": unit, "cores": cores,
                                    "sample": sample_all + f"; rollouts on {cores} threads"}
        line = {"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": t_step_ms, "higher_is_better": True,
                "scaling": "strong" if args.sharded else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": config_of(w, args, stored),
                "generations_per_sec": (1 if args.sharded else world) / (t_step_ms * 1e-3),
                "ms_per_step_median": per_step[len(per_step) // 2], "ms_per_step_best": per_step[0],
                "sm_count": sm_count,
                "e2e": {"value": whole_job_value(units_per_gen, world, e2e_ms, args.sharded), "unit": unit,
                        "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
                "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline,
                "stages": stages, "cpu_baseline": cpu}
        if graph_ms is not None:
            line["graph_replay"] = {"ms_per_step": graph_ms, "value": whole_job_value(units_per_gen, world, graph_ms),
                                    "unit": unit, "note": "ask -> rollout -> tell captured once, replayed per step"}
        print(json.dumps(line))
    s.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "seq2seq", "paint"])
    ap.add_argument("--noise", default="stored", choices=["stored", "regenerated"])
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="omit the oracle timing leg")
    ap.add_argument("--sharded", action="store_true",
                    help="one population split over the ranks by antithetic pairs (strong scaling) "
                         "instead of independent replicas")
    ap.add_argument("--graph", action="store_true",
                    help="also time the generation replayed from a CUDA graph (extra key graph_replay)")
    ap.add_argument("--pop", type=int, default=0, help="override the population size (experiments)")
    ap.add_argument("--dim", type=int, default=0, help="override the parameter count (cfg5 only)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2202_05008_b200 import workloads as W
    w = W.CONFIGS[args.workload]
    if args.pop:
        w = w.with_(pop_size=args.pop)
    if args.dim and args.workload == "cfg5":
        w = w.with_(param_dim=args.dim)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
