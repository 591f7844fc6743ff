"""The N > 1 path on CPU: two `gloo` ranks split the (batch, head) pairs of one problem.

Eq. 5-6 and Eq. 9-12 sum over the positions of one sequence of one head only, so a shard of
the pairs is a complete problem and the reassembled shards must equal the undivided result bit
for bit (the oracle plays the per-rank worker here; on GPUs the library does).  Also covered: the
partition itself, the max-over-ranks timing reduction, the weak-scaling seeds, and the rank
filter of the benchmark's CPU arm.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2006_16236_b200 import shard  # noqa: E402
from paper_2006_16236_b200.inputs import WORKLOADS, draw_qkvg  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


# ------------------------------------------------------------------ partition (single process)
@pytest.mark.parametrize("pairs,world", [(0, 2), (1, 2), (5, 2), (64, 8), (7, 3), (3, 8)])
def test_pair_range_is_a_partition(pairs, world):
    ranges = [shard.pair_range(pairs, world, r) for r in range(world)]
    assert ranges[0][0] == 0 and ranges[-1][1] == pairs
    for (lo, hi), (lo2, _) in zip(ranges, ranges[1:]):
        assert hi == lo2 and lo <= hi
    sizes = [hi - lo for lo, hi in ranges]
    assert max(sizes) - min(sizes) <= 1


def test_pair_range_rejects_bad_ranks():
    with pytest.raises(ValueError):
        shard.pair_range(8, 2, 2)
    with pytest.raises(ValueError):
        shard.pair_range(8, 0, 0)
    with pytest.raises(ValueError):
        shard.pair_range(-1, 2, 0)


def test_shard_pairs_are_views_in_pair_order():
    x = torch.arange(2 * 3 * 4 * 5, dtype=torch.float32).reshape(2, 3, 4, 5)
    a, = shard.shard_pairs([x], 2, 0)
    b, = shard.shard_pairs([x], 2, 1)
    assert a.shape == (1, 3, 4, 5) and b.shape == (1, 3, 4, 5)
    assert torch.equal(torch.cat([a, b], 1).reshape(2, 3, 4, 5), x)
    assert a.data_ptr() == x.data_ptr()                    # nothing copied


def test_rank_workload_changes_only_the_seed():
    w = WORKLOADS["causal_fp32_small"]
    w1 = shard.rank_workload(w, 4, 3)
    assert (w1.B, w1.H, w1.N, w1.D, w1.M, w1.dtype) == (w.B, w.H, w.N, w.D, w.M, w.dtype)
    assert w1.seed == w.seed + 3 and shard.rank_workload(w, 4, 0) == w
    with pytest.raises(ValueError):
        shard.rank_workload(w, 2, 2)


# ------------------------------------------------------------------ two gloo ranks
def _worker(rank, world, port, causal, out_dir):
    os.environ.update(WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import oracle
    w_, r_, _ = shard.init_process_group("gloo")
    assert (w_, r_) == (world, rank)
    B, H, N, D, M = 1, 5, 96, 8, 8                         # 5 pairs over 2 ranks: 3 + 2
    tensors = draw_qkvg(B, H, N, D, M, 77, torch.float32, 1.0)
    Q, K, V, G = [t.double() for t in shard.shard_pairs(tensors, world, rank)]
    lo, hi = shard.pair_range(B * H, world, rank)
    assert Q.shape[1] == hi - lo
    O, den = oracle.linear_attention(Q.numpy(), K.numpy(), V.numpy(), causal)
    grads = oracle.linear_attention_backward(Q.numpy(), K.numpy(), V.numpy(), G.numpy(), causal)
    full = [shard.gather_pairs(torch.from_numpy(np.ascontiguousarray(g)), B * H, world, rank) for g in (O, den, *grads)]
    # timing reductions: the job's time is the slowest rank's, its size the sum of the shards
    slowest = shard.max_over_ranks(10.0 + rank, world)
    total_pairs = shard.sum_over_ranks(hi - lo, world)
    shard.barrier(world, cuda=False)
    if rank == 0:
        torch.save({"full": full, "slowest": slowest, "total_pairs": total_pairs}, os.path.join(out_dir, "out.pt"))
    import torch.distributed as dist
    dist.destroy_process_group()


@pytest.mark.parametrize("causal", [True, False])
def test_two_ranks_reproduce_the_undivided_problem(tmp_path, causal):
    import oracle
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), causal, str(tmp_path)), nprocs=world, join=True)
    got = torch.load(os.path.join(tmp_path, "out.pt"))
    assert got["slowest"] == 11.0 and got["total_pairs"] == 5.0
    Q, K, V, G = [t.double().numpy() for t in draw_qkvg(1, 5, 96, 8, 8, 77, torch.float32, 1.0)]
    O, den = oracle.linear_attention(Q, K, V, causal)
    grads = oracle.linear_attention_backward(Q, K, V, G, causal)
    for x, ref in zip(got["full"], (O, den, *grads)):
        assert x.shape == ref.shape
        assert np.array_equal(x.numpy(), ref)              # same arithmetic per pair: bit-identical


# ------------------------------------------------------------------ the benchmark's CPU arm under a launcher
def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", LOCAL_RANK="1", RANK="1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "causal_fp32_small"]
    other = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert other.returncode == 0 and other.stdout.strip() == ""
    env.update(RANK="0", LOCAL_RANK="0")
    first = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert first.returncode == 0, first.stderr
    line = json.loads(first.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
