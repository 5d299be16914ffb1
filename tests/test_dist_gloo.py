"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent replicas, max-over-ranks timing."""
import json
import os
import subprocess
import sys

import pytest
import torch.multiprocessing as mp

from paper_2506_04708_b200 import dist as sd, inputs, sharded

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert sd.env_ranks() == (rank, world, rank)
    d = sd.init("gloo")
    assert d is not None and d.get_world_size() == world
    sd.barrier(d)
    # every rank "measured" a different time: all of them learn the slowest one
    mine = 10.0 + 5.0 * rank
    slowest = sd.max_over_ranks(d, mine)
    # replicas are independent: different seeds give different streams
    w = inputs.scaled(inputs.WORKLOADS["cfg1"], B=2)
    s = inputs.token_streams(w, sd.replica_seed(0, rank), 64)
    res = {"rank": rank, "slowest": slowest, "stream_head": s[0, :8].tolist(),
           "rate": sd.whole_job_rate(w.B * w.N, world, 100, slowest)}
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump(res, f)
    sd.barrier(d)
    d.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"r{k}.json")) for k in range(world)]
    assert r[0]["slowest"] == r[1]["slowest"] == 15.0
    assert r[0]["stream_head"] != r[1]["stream_head"]
    # 2 ranks x (2 sequences x 8 nodes) x 100 steps over 15 ms
    assert r[0]["rate"] == pytest.approx(2 * 16 * 100 / 15e-3)


def test_single_process_needs_no_group():
    os.environ.pop("WORLD_SIZE", None)
    os.environ.pop("RANK", None)
    assert sd.env_ranks()[1] == 1
    assert sd.init("gloo") is None
    assert sd.max_over_ranks(None, 3.5) == 3.5
    assert sd.replica_seed(5, 0) == 5 and sd.replica_seed(5, 3) != sd.replica_seed(5, 2)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


def _exchange_worker(rank, world, port, out_dir):
    import numpy as np
    import torch
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    d = sd.init("gloo")
    B, W, n_max, K = 3, 4, 3, 5  # sequences per rank, path slots per sequence
    seq = rank * B + torch.arange(B).repeat_interleave(W)          # global sequence of every row
    pos = torch.arange(W).repeat(B)
    ctx = torch.stack([seq, pos, seq * 100 + pos], dim=1).to(torch.int32)
    ids = (seq * 1000 + pos * 10).to(torch.int32)[:, None] + torch.arange(K, dtype=torch.int32)[None, :]
    probs = (seq.double() + pos.double() / 10)[:, None].float().repeat(1, K)
    rows = torch.cat([ctx, ids, probs.view(torch.int32)], dim=1)   # the packed layout: context, ids, probability bits
    got = sharded.gather_rows(d, rows)
    np.save(os.path.join(out_dir, f"x{rank}.npy"), got.numpy())
    sd.barrier(d)
    d.destroy_process_group()


def test_record_exchange_keeps_global_sequence_order(tmp_path):
    """The update rows of all ranks arrive on every rank in (sequence, path position) order of the whole batch: the
    order in which one context holding the whole batch applies them.  One collective moves everything."""
    import numpy as np
    world, port = 2, 31000 + os.getpid() % 2000
    mp.spawn(_exchange_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [np.load(tmp_path / f"x{k}.npy") for k in range(world)]
    assert np.array_equal(r[0], r[1])
    rows = r[0]
    assert rows.shape == (2 * 3 * 4, 3 + 2 * 5)
    ctx, ids, probs = rows[:, :3], rows[:, 3:8], rows[:, 8:].copy().view(np.float32)
    order = ctx[:, 0] * 4 + ctx[:, 1]
    assert np.array_equal(order, np.arange(24))
    assert np.array_equal(ids[:, 0], ctx[:, 0] * 1000 + ctx[:, 1] * 10)
    assert np.allclose(probs[:, 0], ctx[:, 0] + ctx[:, 1] / 10)
    # no group: the rows pass through untouched
    import torch
    one = torch.zeros(2, 13, dtype=torch.int32)
    assert sharded.gather_rows(None, one) is one


def test_bench_starts_its_own_ranks_when_run_without_a_launcher():
    """`python bench.py --gpus 2` with no launcher environment starts two ranks itself (torch.distributed.run on
    127.0.0.1) and reports n_gpus = 2.  The reference arm needs no GPU, so this runs here: rank 0 times the
    oracle and prints the line, rank 1 exits without work."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0", "--workload", "cfg1"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["value"] > 0
