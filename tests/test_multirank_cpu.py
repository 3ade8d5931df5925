"""The N > 1 plumbing of bench.py on CPU: two gloo ranks (no GPU involved)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    slowest = bench.max_over_ranks(local_ms, torch.device("cpu"), world)
    seeds = [None] * world
    dist.all_gather_object(seeds, bench.rank_seed(7, rank))
    dist.barrier()
    if rank == 0:
        json.dump({"slowest": slowest, "seeds": seeds,
                   "value": bench.whole_job_value(1000.0, world, slowest)}, open(out, "w"))
    dist.destroy_process_group()


def test_two_gloo_ranks_max_timing_distinct_seeds_and_aggregate(tmp_path):
    out = str(tmp_path / "r.json")
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["slowest"] == 15.0
    assert len(set(r["seeds"])) == 2
    assert abs(r["value"] - 2 * 1000.0 / 0.015) < 1e-6


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "cfg1"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


def _exchange_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2202_05008_b200 import sharded
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    H, D = 8, 5
    first, n = sharded.shard_of(H, rank, world)
    # member m has fitness 10 m; the shard holds members [2 first, 2 (first + n))
    fit_local = torch.arange(2 * first, 2 * (first + n), dtype=torch.float32) * 10.0
    fit_all = sharded.gather_fitness(fit_local, world)
    grad = torch.full((D,), float(rank + 1), dtype=torch.float64)
    sig = torch.full((D,), 0.5 * (rank + 1), dtype=torch.float32)
    sharded.reduce_sums(grad, sig, world)
    got = [None] * world
    dist.all_gather_object(got, (first, n, fit_all.tolist(), grad.tolist(), sig.tolist()))
    if rank == 0:
        json.dump(got, open(out, "w"))
    dist.destroy_process_group()


def test_pair_shards_gather_fitness_in_member_order_and_sum_gradients(tmp_path):
    out = str(tmp_path / "x.json")
    port = 33500 + os.getpid() % 2000
    mp.spawn(_exchange_worker, args=(2, port, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert [(a[0], a[1]) for a in r] == [(0, 4), (4, 4)]
    for a in r:                                            # every rank ends with the same values
        assert a[2] == [10.0 * m for m in range(16)]
        assert a[3] == [3.0] * 5 and a[4] == [1.5] * 5


def test_shard_of_rejects_uneven_split():
    sys.path.insert(0, ROOT)
    from paper_2202_05008_b200 import sharded
    import pytest
    with pytest.raises(ValueError):
        sharded.shard_of(10, 0, 4)
    assert sharded.shard_of(12, 2, 4) == (6, 3)


class _StubShard:
    """Host-only stand-in for a sharded solver: same five calls as the binding, CPU tensors, and an
    'update' that is a plain function of the reduced sums, so that the orchestration in
    sharded.generation (order of calls, what is exchanged) can be checked without a GPU."""

    def __init__(self, first_pair, n_pairs, n_pairs_total, D):
        self.first, self.n, self.H, self.D = first_pair, n_pairs, n_pairs_total, D
        self.center = torch.zeros(D, dtype=torch.float64)
        self.grad = torch.zeros(D, dtype=torch.float64)
        self.sig = torch.zeros(D, dtype=torch.float32)
        self.log = []

    def _eps(self, pair):                       # any pair's noise can be rebuilt anywhere
        g = torch.Generator().manual_seed(1000 + pair)
        return torch.randn(self.D, generator=g, dtype=torch.float64)

    def ask(self):
        self.log.append("ask")

    def rollout(self):
        self.log.append("rollout")              # fitness of member m = -(its first parameter)^2, 0.1 sigma
        f = []
        for j in range(self.first, self.first + self.n):
            e = self._eps(j)[0].item()
            f += [-(self.center[0].item() + 0.1 * e) ** 2, -(self.center[0].item() - 0.1 * e) ** 2]
        return torch.tensor(f, dtype=torch.float32)

    def tell_begin(self, fit_all):
        self.log.append("begin")
        assert fit_all.numel() == 2 * self.H
        u = torch.argsort(torch.argsort(fit_all)).double() / (2 * self.H - 1) - 0.5
        self.grad.zero_()
        for j in range(self.first, self.first + self.n):
            self.grad += (u[2 * j] - u[2 * j + 1]) * self._eps(j)
        self.sig.fill_(float(self.n))

    def reduce_buffers(self):
        self.log.append("buffers")
        return self.grad, self.sig

    def tell_end(self):
        self.log.append("end")
        self.center += 0.1 * self.grad / (2 * self.H)


def _generation_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2202_05008_b200 import sharded
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    H, D = 8, 3
    first, n = sharded.shard_of(H, rank, world)
    shard = _StubShard(first, n, H, D)
    for _ in range(3):
        fit_all = sharded.generation(shard, world)
    got = [None] * world
    dist.all_gather_object(got, (shard.center.tolist(), shard.log, fit_all.tolist(), shard.sig.tolist()))
    if rank == 0:
        json.dump(got, open(out, "w"))
    dist.destroy_process_group()


def test_sharded_generation_over_two_ranks_equals_one_rank(tmp_path):
    out = str(tmp_path / "g.json")
    port = 35500 + os.getpid() % 2000
    mp.spawn(_generation_worker, args=(2, port, out), nprocs=2, join=True)
    two = json.load(open(out))
    sys.path.insert(0, ROOT)
    from paper_2202_05008_b200 import sharded
    single = _StubShard(0, 8, 8, 3)
    for _ in range(3):
        fit = sharded.generation(single, 1)
    for center, log, fit_all, sig in two:
        assert log == ["ask", "rollout", "begin", "buffers", "end"] * 3
        assert max(abs(a - b) for a, b in zip(center, single.center.tolist())) < 1e-12
        assert fit_all == fit.tolist()                 # gathered in member order
        assert sig == [8.0] * 3                        # the second buffer was summed too
    assert two[0][0] == two[1][0]                      # both ranks hold the same centre, bit for bit
