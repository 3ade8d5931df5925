#!/usr/bin/env python
"""Benchmark of one evolution-strategy generation (ask -> rollout -> tell) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl ours|reference]

One "step" is one whole generation of the workload.  Prints ONE JSON line (rank 0).

The headline workload is the large-population control configuration (cfg4: 4,096 members,
MLP 28-128-128-8, 4 episodes x 1,000 steps), the largest roll-out that fits one GPU.  At N = 1
the same line carries, under "per_config", a compact record (time per generation, stage times,
roofline, end-to-end, CPU baseline) for the other configurations: cfg1, cfg2, cfg3 and the
update sweep cfg5 with stored and with regenerated noise.

For N > 1 (launched by torch.distributed.run) the ranks share ONE population, split by
antithetic pairs: every rank samples and evaluates its pairs, the fitness is all-gathered and
the gradient sums all-reduced over NCCL (strong scaling; value = one population's units / time
of the slowest rank).  `--replicas` runs N independent solvers instead (weak scaling).

`--impl reference` times the CPU oracle (single-threaded C, fp64) on a bounded sample of the same
workload; it is a deliberately slow, plain program and serves as a baseline only.
"""
from __future__ import annotations

import argparse
import ctypes
import hashlib
import json
import os
import shutil
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

FP32_LANES_PER_SM = 128
L2_FLUSH_BYTES = 256 << 20
HEADLINE = "cfg4"
PER_CONFIG = [("cfg1", "stored"), ("cfg2", "stored"), ("cfg3", "stored"), ("cfg5", "stored"),
              ("cfg5", "regenerated")]


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


# ------------------------------------------------------------------------------------------
# DRAM traffic of the dominant kernel, from ncu captures
# ------------------------------------------------------------------------------------------
# (workload, noise) -> kernel, dram__bytes_read.sum + dram__bytes_write.sum per launch, the source
# files that define the kernel, and the digest of those files when the counters were taken (see
# the matching summary under profiles/).  The figure is printed only while the files still have
# that digest; once a kernel's source changes its entry reads null until it is captured again.
CSRC = os.path.join(ROOT, "paper_2202_05008_b200", "csrc")
NCU_TRAFFIC = {
    ("cfg4", "stored"): {"kernel": "k_rollout_tl_tc", "bytes": 3.490288e+08,
                         "files": ['rollout_tl_tc.cu', 'umma.cuh', 'async.cuh', 'noise.cuh', 'fp32x2.cuh', 'internal.h'],
                         "digest": "6dc95ec37104ccff",
                         "capture": "P = 592 capture scaled by members (the traffic is the parameter rows, proportional to P)"},
    ("cfg2", "stored"): {"kernel": "k_rollout_cartpole_ws", "bytes": 4.788480e+06,
                         "files": ['rollout_mlp_tiled.cu', 'async.cuh', 'tasks.cuh', 'noise.cuh', 'fp32x2.cuh', 'internal.h'],
                         "digest": "43ceffc3a9b4ab42", "capture": "full size"},
    ("cfg3", "stored"): {"kernel": "k_cnn_conv2_tc", "bytes": 1.530819e+08,
                         "files": ['rollout_cnn_tc.cu', 'umma.cuh', 'async.cuh', 'fp32x2.cuh', 'internal.h'],
                         "digest": "9d6c703703822230", "capture": "full size"},
    ("cfg5", "stored"): {"kernel": "k_ask", "bytes": 1.012191e+11,
                         "files": ['solver_kernels.cu', 'noise.cuh', 'internal.h'],
                         "digest": "7c892cd86db089c1",
                         "capture": "D = 32,768 capture scaled by 32 (columns are independent)"},
    ("cfg5", "regenerated"): {"kernel": "k_ask", "bytes": 6.677464e+10,
                              "files": ['solver_kernels.cu', 'noise.cuh', 'internal.h'],
                              "digest": "7c892cd86db089c1", "capture": "D = 32,768 capture scaled by 32"},
}
NCU_TRAFFIC[("cfg4", "regenerated")] = NCU_TRAFFIC[("cfg4", "stored")]
NCU_TRAFFIC[("cfg2", "regenerated")] = NCU_TRAFFIC[("cfg2", "stored")]


def source_digest(files):
    h = hashlib.sha256()
    for f in sorted(files):
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(f.encode() + b"\0" + fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload, noise):
    entry = NCU_TRAFFIC.get((workload, noise))
    if entry is None:
        return None
    try:
        if source_digest(entry["files"]) != entry["digest"]:
            return None
    except OSError:
        return None
    return entry


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------
# fp32 FMA probe (a measurement aid that lives beside this file, not in the library)
# ------------------------------------------------------------------------------------------
PROBE_SRC = os.path.join(ROOT, "bench_fma_probe.cu")
PROBE_LIB = os.path.join(ROOT, "libbench_fma_probe.so")
_probe = None


def build_fma_probe(force=False):
    if not force and os.path.exists(PROBE_LIB) and os.path.getmtime(PROBE_LIB) >= os.path.getmtime(PROBE_SRC):
        return PROBE_LIB
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--shared",
           "-Xcompiler", "-fPIC", "-o", PROBE_LIB, PROBE_SRC]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return PROBE_LIB


def fma_probe(device="cuda:0", iters=1 << 14, repeats=5, threads=1024):
    """Sustained fp32 FMA rate of `device` in TFLOP/s (best of `repeats` launches of the probe
    kernel, timed with CUDA events): the measured denominator for ALU-bound kernels."""
    import torch
    global _probe
    if _probe is None:
        _probe = ctypes.CDLL(build_fma_probe())
        _probe.bench_fma_probe.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                           ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint64)]
        _probe.bench_fma_probe.restype = ctypes.c_int
    dev = torch.device(device)
    with torch.cuda.device(dev):
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        blocks = sms * (2048 // threads) * 4
        sink = torch.empty(blocks * threads, dtype=torch.float32, device=dev)
        st = torch.cuda.current_stream(dev)
        flops = ctypes.c_uint64()
        best = 0.0
        for i in range(repeats + 2):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            rc = _probe.bench_fma_probe(sink.data_ptr(), blocks, threads, iters, st.cuda_stream, ctypes.byref(flops))
            if rc != 0:
                raise RuntimeError(f"bench_fma_probe returned {rc}")
            e1.record(st)
            e1.synchronize()
            if i >= 2:                                   # two warm-up launches
                best = max(best, flops.value / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    return best


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
            self._stop.clear()
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
            self._thread = None

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
    problems) and the rollout of n_members members.  Returns (seconds for a full generation,
    extrapolated linearly -- members and columns are independent --, seconds actually spent, a
    description of the sample).  threads > 1 spreads the members' rollouts (unchanged oracle
    code, one member per call) over host threads; ask and tell stay on one thread."""
    import oracle
    from paper_2202_05008_b200 import workloads as W
    P, D = w.pop_size, w.param_dim
    cols = D if P * D <= 50_000_000 else 4096
    wall0 = time.perf_counter()
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
    spent = time.perf_counter() - wall0
    sample = (f"ask+tell on all {P} members x {cols} of {D} columns; rollout of {n_done} of {P} members "
              f"x {w.episodes} episodes x {w.horizon} steps; scaled linearly to one generation")
    return t_ask + t_roll + t_tell, spent, sample


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
    t, _, _ = oracle_generation_sample(w.with_(pop_size=2, param_dim=w.param_dim), 1)
    per_member = max(t / 2.0, 1e-4)
    return int(max(1, min(w.pop_size, seconds / per_member)))


def cpu_baseline_of(w, seconds, all_cores=False):
    """The oracle, as it stands, on one host core for about `seconds` of work."""
    from paper_2202_05008_b200 import workloads as W
    _, unit, units_per_gen = unit_of(w)
    n = members_for_budget(w, seconds)
    t_cpu, _, sample = oracle_generation_sample(w, max(n, 1))
    cpu = {"value": units_per_gen / t_cpu, "unit": unit, "cores": 1, "kind": "oracle", "sample": sample}
    cores = len(os.sched_getaffinity(0))
    if all_cores and cores > 1 and w.task_kind != W.TASK_NONE:   # same oracle, members spread over the host's cores
        n_all = min(w.pop_size, max(n, 1) * cores)
        t_all, _, sample_all = oracle_generation_sample(w, n_all, threads=cores)
        cpu["all_cores"] = {"value": units_per_gen / t_all, "unit": unit, "cores": cores,
                            "sample": sample_all + f"; rollouts on {cores} threads"}
    return cpu


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    metric, unit, units_per_gen = unit_of(w)
    # per-step sample sized so that warm-up + timed steps take about two minutes in all
    n = members_for_budget(w, min(1.0, 120.0 / max(1, args.warmup + args.steps)))
    full, spent, sample = [], [], ""
    for i in range(args.warmup + args.steps):
        t, s, sample = oracle_generation_sample(w, max(n, 1), generation=i)
        if i >= args.warmup:
            full.append(t)
            spent.append(s)
    t_full = sum(full) / len(full)          # one whole generation, scaled from the sample
    t_step = sum(spent) / len(spent)        # what one timed step really took
    value = units_per_gen / t_full
    line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3,
            "ms_per_generation_scaled": t_full * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(w, args, stored=True),
            "generations_per_sec": 1.0 / t_full,
            "cpu_baseline": {"value": value, "unit": unit, "cores": 1, "kind": "oracle",
                             "sample": sample + "; a timed step is this sample, the value is the sample's rate"},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def config_of(w, args, stored):
    from paper_2202_05008_b200 import workloads as W
    task = {W.TASK_NONE: "none", W.TASK_CARTPOLE: "cartpole_swingup", W.TASK_TANH_LINEAR: "tanh_linear",
            W.TASK_SUPERVISED: "supervised_28x28", W.TASK_SEQ2SEQ_ADD: "seq2seq_addition",
            W.TASK_PAINT: f"triangle_painting_{int(w.task_param[0]) if w.task_param else 0}x{int(w.task_param[1]) if len(w.task_param) > 1 else 0}"}[w.task_kind]
    sharded_run = (args.gpus > 1 and not args.replicas) or getattr(args, "sharded", False)
    return {"workload": w.name, "pop_size": w.pop_size, "param_dim": w.param_dim, "task": task,
            "policy": "mlp " + "-".join(map(str, w.layer_sizes)) if w.policy_kind == W.POLICY_MLP else
                      {W.POLICY_CNN_28: "cnn_28",
                       W.POLICY_LSTM_SEQ2SEQ: f"lstm_encoder_decoder h={w.layer_sizes[0] if w.layer_sizes else 0}"
                       }.get(w.policy_kind, "none"),
            "episodes": w.episodes, "horizon": w.horizon, "batch": w.batch,
            "noise": "stored" if stored else "regenerated",
            "parallelism": f"{'one population, pair shards' if sharded_run else 'replicas'} x{args.gpus}",
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
def roofline_of(w, workload_key, noise, stages, work, peaks, sm_count, max_mhz, fma_measured, overridden):
    """Roofline record of the dominant kernel of one workload (CUDA-event stage times)."""
    from paper_2202_05008_b200 import workloads as W
    alu_peak = sm_count * FP32_LANES_PER_SM * 2 * max_mhz * 1e6 / 1e12      # TFLOP/s fp32 FMA
    if w.task_kind == W.TASK_NONE:
        dom = "ask" if stages["ask"]["ms"] >= stages["tell"]["ms"] else "tell"
        achieved = stages[dom]["GB/s"]
        r = {"kernel": "k_ask" if dom == "ask" else "k_grad_partial", "bound": "hbm",
             "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
             "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": None}
        if noise == "regenerated":
            r["note"] = ("regenerated noise: ask writes theta only and tell recomputes the normals, so both are "
                         "bound by integer/fp32 issue, not by HBM; the figure is the GB/s equivalent")
    elif w.task_kind in (W.TASK_SUPERVISED, W.TASK_SEQ2SEQ_ADD):
        achieved = stages["rollout"]["TFLOP/s"]
        r = {"kernel": "k_cnn_conv1_tc + k_cnn_conv2_tc" if w.task_kind == W.TASK_SUPERVISED else "k_s2s_tc",
             "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
             "frac": achieved / peaks["bf16_tflops"], "peak_source": peaks["source"], "traffic": None}
    else:
        achieved = stages["rollout"]["TFLOP/s"]
        # cart-pole: more than 8 episodes on a 32/64/128-wide shape run the warp-specialised two-group kernel
        cart = "k_rollout_cartpole_ws" if (w.episodes > 8 and len(w.layer_sizes) == 4 and
                                           16 < max(w.layer_sizes[1:3]) <= 128) else "k_rollout_mlp_tiled"
        kernel = {W.TASK_PAINT: "k_paint", W.TASK_TANH_LINEAR: "k_rollout_tl_tc", W.TASK_CARTPOLE: cart}[w.task_kind]
        r = {"kernel": kernel,
             "bound": "alu", "achieved": achieved, "peak": alu_peak, "unit": "TFLOP/s",
             "frac": achieved / alu_peak,
             "peak_source": f"{sm_count} SMs x 128 fp32 lanes x 2 x {max_mhz} MHz", "traffic": None}
        if fma_measured:
            r.update({"peak_measured": fma_measured, "frac_of_measured": achieved / fma_measured,
                      "peak_measured_source": "bench_fma_probe (16 FMA chains per thread, best of 5 launches)"})
        if w.task_kind == W.TASK_TANH_LINEAR and tuple(w.layer_sizes) == (28, 128, 128, 8):
            # the two wide layers run on the tensor cores as split-fp16 MMAs (hi/lo parts of weights and
            # activations: 4 tensor flops per algorithmic flop, in 128 x 8 x 16 tiles)
            wide = 2.0 * (28 * 128 + 128 * 128) * w.env_steps_per_generation
            t_s = stages["rollout"]["ms"] * 1e-3
            r["tensor"] = {"algorithmic_TFLOP/s_of_the_wide_layers": wide / t_s / 1e12,
                           "mma_TFLOP/s_issued": 4.0 * wide * (32.0 / 28.0 * 28 * 128 + 128 * 128) / (28 * 128 + 128 * 128) / t_s / 1e12,
                           "peak": peaks["bf16_tflops"], "peak_source": peaks["source"] + " (bf16 dense; fp16 runs at the same rate)"}
            r["tensor"]["frac"] = r["tensor"]["mma_TFLOP/s_issued"] / peaks["bf16_tflops"]
            r["note"] = ("fp32-accurate arithmetic reported against the fp32 pipe (the ceiling of any formulation on the "
                         "CUDA cores); the wide layers run on the tensor cores, whose own figures are under 'tensor'; the "
                         "kernel is bound by the latency of a step's serial chain, not by either pipe")
        if w.task_kind == W.TASK_PAINT:
            r["note"] = ("algorithmic flop = every pixel against every triangle; the kernel skips the pairs "
                         "outside a triangle's bounding box, so this is an equivalent rate, not pipe utilisation")
    entry = None if overridden else ncu_traffic(workload_key, noise)
    if entry is not None and (w.task_kind != W.TASK_NONE or r["kernel"] == entry["kernel"]):
        r["traffic"] = entry["bytes"]
        r["traffic_kernel"] = entry["kernel"]
        r["traffic_capture"] = entry["capture"]
    return r


def measure(w, workload_key, noise, steps, warmup, dev, rank, world, sharded_run, flush, sampler=None,
            graph=False, overridden=False):
    """Times `steps` generations of one workload (after `warmup` untimed ones) with CUDA events on
    the solver's stream, then the same generation end to end from pinned host buffers.  Returns
    the numbers of this rank with the cross-rank maxima already taken."""
    import torch
    import torch.distributed as dist
    from paper_2202_05008_b200 import Solver, sharded, workloads as W

    stored = noise == "stored"
    mode = W.NOISE_STORED if stored else W.NOISE_REGENERATED
    if sharded_run:                                     # one population, rank r owns a range of pairs
        first_pair, n_pairs = sharded.shard_of(w.pop_size // 2, rank, world)
        w_rank = w
        s = Solver(w_rank, device=dev, noise_mode=mode, shard_first_pair=first_pair, shard_pairs=n_pairs)
    else:
        first_pair, n_pairs = 0, w.pop_size // 2
        w_rank = w.with_(seed=rank_seed(w.seed, rank))  # independent replicas
        s = Solver(w_rank, device=dev, noise_mode=mode)
    P, D = s.P, w.param_dim                             # P = members this rank evaluates
    supervised = w.task_kind == W.TASK_SUPERVISED
    no_task = w.task_kind == W.TASK_NONE
    fitness = torch.empty(P, dtype=torch.float32, device=dev)
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
        if sharded_run:
            fits = [f[2 * first_pair:2 * (first_pair + n_pairs)].contiguous() for f in fits]

    def tell(f):
        if not sharded_run:
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

    for i in range(warmup):
        flush.fill_(i & 255)
        generation(i)
    torch.cuda.synchronize()
    if s.sync_status() != 0:
        raise SystemExit("bench.py: device status not ok after warm-up")

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    launches0 = s.launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    for i in range(steps):
        flush.fill_(i & 255)                            # evict L2 (untimed)
        generation(warmup + i, events[i])
    if sampler:
        sampler.sample()
    torch.cuda.synchronize()
    if sampler:
        sampler.stop()
    if world > 1:
        dist.barrier()
    launches = s.launch_count() - launches0
    status = s.sync_status()
    if status != 0:
        raise SystemExit(f"bench.py: device status {status} after the timed region")

    t_ask = sum(e[0].elapsed_time(e[1]) for e in events) / steps
    t_roll = sum(e[1].elapsed_time(e[2]) for e in events) / steps
    t_tell = sum(e[2].elapsed_time(e[3]) for e in events) / steps
    per_step = sorted(e[0].elapsed_time(e[3]) for e in events)
    t_step_ms = max_over_ranks(sum(per_step), dev, world) / steps

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
    e2e_steps = max(3, min(steps, 50))
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
    if graph and not sharded_run and not no_task:
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            sg = Solver(w_rank, device=dev, stream=side, noise_mode=mode)
            if supervised:
                sg.set_batch(*batches[0])
            if w.task_kind == W.TASK_PAINT:
                sg.set_target(d_target)
            gfit = torch.empty(P, dtype=torch.float32, device=dev)
            for _ in range(max(warmup, 3)):
                sg.ask(); sg.rollout(fitness=gfit); sg.tell(gfit)
            cg = sg.capture_generation(gfit)
            gev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            cg.replay()
            side.synchronize()
            for i in range(steps):
                flush.fill_(i & 255)
                gev[i][0].record(side)
                cg.replay()
                gev[i][1].record(side)
            side.synchronize()
            if sg.sync_status() != 0:
                raise SystemExit("bench.py: device status not ok after the graph replays")
            graph_ms = max_over_ranks(sum(a.elapsed_time(b) for a, b in gev), dev, world) / steps
            sg.close()

    work = stage_work(w.with_(pop_size=P) if sharded_run else w, stored)   # this rank's share
    stages = {
        "ask": {"ms": t_ask, "GB/s": work["ask_bytes"] / (t_ask * 1e-3) / 1e9},
        "rollout": {"ms": t_roll, "TFLOP/s": work["rollout_flops"] / (t_roll * 1e-3) / 1e12 if t_roll > 0 else 0.0},
        "tell": {"ms": t_tell, "GB/s": work["tell_bytes"] / (t_tell * 1e-3) / 1e9},
    }
    s.close()
    del s
    return {"ms_per_step": t_step_ms, "ms_per_step_median": per_step[len(per_step) // 2],
            "ms_per_step_best": per_step[0], "stages": stages, "work": work, "launches": int(launches),
            "e2e_ms": e2e_ms, "h2d": h2d, "d2h": d2h, "graph_ms": graph_ms, "overridden": overridden}


def per_config_record(key, noise, args, dev, flush, peaks, sm_count, max_mhz, fma_measured):
    """Compact record of one of the other configurations (N = 1 only)."""
    import torch
    from paper_2202_05008_b200 import workloads as W
    from paper_2202_05008_b200.binding import EvoConfig, make_config, load_library
    w = W.CONFIGS[key]
    name = key if key != "cfg5" else f"cfg5_{noise}"
    nbytes = ctypes.c_size_t(0)
    cfg = make_config(w, noise_mode=W.NOISE_STORED if noise == "stored" else W.NOISE_REGENERATED)
    load_library().evo_workspace_bytes(ctypes.byref(cfg), ctypes.byref(nbytes))
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info(dev)
    need = nbytes.value + (64 << 20)
    if need > free:
        return name, {"workload": w.name, "noise": noise,
                      "skipped": f"needs {need / 2**30:.1f} GiB free, {free / 2**30:.1f} GiB available"}
    steps = min(args.steps, 20) if key == "cfg5" else args.steps
    m = measure(w, key, noise, steps, max(3, min(args.warmup, 5)), dev, 0, 1, False, flush)
    torch.cuda.empty_cache()
    metric, unit, units = unit_of(w)
    rec = {"workload": w.name, "noise": noise, "metric": metric, "unit": unit, "steps": steps,
           "ms_per_step": m["ms_per_step"], "value": units / (m["ms_per_step"] * 1e-3),
           "generations_per_sec": 1.0 / (m["ms_per_step"] * 1e-3), "stages": m["stages"],
           "roofline": roofline_of(w, key, noise, m["stages"], m["work"], peaks, sm_count, max_mhz,
                                   fma_measured, False),
           "e2e": {"value": units / (m["e2e_ms"] * 1e-3), "unit": unit, "ms_per_step": m["e2e_ms"],
                   "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"]},
           "gpu_launches": m["launches"]}
    if not args.skip_cpu_baseline:
        rec["cpu_baseline"] = cpu_baseline_of(w, 2.0)
    return name, rec


def run_ours(args, w):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the GPU arm has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    sharded_run = (world > 1 and not args.replicas) or args.sharded
    overridden = bool(args.pop or args.dim)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    sampler = ClockSampler(local)
    m = measure(w, args.workload, args.noise, args.steps, args.warmup, dev, rank, world, sharded_run, flush,
                sampler=sampler, graph=args.graph, overridden=overridden)

    if rank == 0:
        metric, unit, units_per_gen = unit_of(w)
        value = whole_job_value(units_per_gen, world, m["ms_per_step"], sharded_run)
        peaks = measured_peaks()
        clocks = sampler.summary()
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        max_mhz = clocks["sm_max_mhz"] or 1965
        fma_measured = fma_probe(dev)                     # register-only FMA chains, timed alone
        roofline = roofline_of(w, args.workload, args.noise, m["stages"], m["work"], peaks, sm_count, max_mhz,
                               fma_measured, overridden)
        cpu = None if args.skip_cpu_baseline else cpu_baseline_of(w, 12.0, all_cores=True)
        line = {"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": m["ms_per_step"], "higher_is_better": True,
                "scaling": "strong" if sharded_run else "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": config_of(w, args, args.noise == "stored"),
                "generations_per_sec": (1 if sharded_run else world) / (m["ms_per_step"] * 1e-3),
                "ms_per_step_median": m["ms_per_step_median"], "ms_per_step_best": m["ms_per_step_best"],
                "sm_count": sm_count,
                "e2e": {"value": whole_job_value(units_per_gen, world, m["e2e_ms"], sharded_run), "unit": unit,
                        "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"], "ms_per_step": m["e2e_ms"]},
                "gpu_launches": m["launches"], "clocks": clocks, "roofline": roofline,
                "stages": m["stages"], "cpu_baseline": cpu}
        if m["graph_ms"] is not None:
            line["graph_replay"] = {"ms_per_step": m["graph_ms"],
                                    "value": whole_job_value(units_per_gen, world, m["graph_ms"]),
                                    "unit": unit, "note": "ask -> rollout -> tell captured once, replayed per step"}
        if world == 1 and args.workload == HEADLINE and not overridden and not args.no_per_config:
            per = {}
            for key, noise in PER_CONFIG:
                name, rec = per_config_record(key, noise, args, dev, flush, peaks, sm_count, max_mhz, fma_measured)
                per[name] = rec
            line["per_config"] = per
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE,
                    choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "seq2seq", "paint"])
    ap.add_argument("--noise", default="stored", choices=["stored", "regenerated"])
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="omit the oracle timing legs")
    ap.add_argument("--no-per-config", action="store_true",
                    help="headline workload only: leave out the records of the other configurations")
    ap.add_argument("--replicas", action="store_true",
                    help="N > 1: independent solvers (weak scaling) instead of one population in pair shards")
    ap.add_argument("--sharded", action="store_true",
                    help="take the pair-sharded code path even at N = 1 (one shard owning every pair; checks the path)")
    ap.add_argument("--graph", action="store_true",
                    help="also time the generation replayed from a CUDA graph (extra key graph_replay)")
    ap.add_argument("--traffic-digests", action="store_true",
                    help="print the source digest each NCU_TRAFFIC entry would need now (after a new capture) and exit")
    ap.add_argument("--pop", type=int, default=0, help="override the population size (experiments)")
    ap.add_argument("--dim", type=int, default=0, help="override the parameter count (cfg5 only)")
    args = ap.parse_args()
    if args.traffic_digests:
        for key, entry in NCU_TRAFFIC.items():
            now = source_digest(entry["files"])
            print(key, entry["kernel"], "stored", entry["digest"], "current", now, "OK" if now == entry["digest"] else "STALE")
        return
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
