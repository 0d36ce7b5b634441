"""The N > 1 path of bench.py: independent replicas, no collective on the data path; the only
exchange is the max-over-ranks of the timing.  Exercised with world_size 2 on CPU (gloo)."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist

    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow replica
        ms = bench.max_over_ranks(local_ms, dist, "cpu")
        dist.barrier()
        out.put((rank, ms, bench.replica_throughput(40, world, ms)))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_sum_over_slowest():
    torch = pytest.importorskip("torch")
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 15.0                                   # every rank sees the slowest replica's time
        assert value == pytest.approx(2 * 40 / 0.015)       # all replicas' tokens over that time


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.replica_throughput(40, 1, 8.0) == pytest.approx(5000.0)


def test_reference_arm_runs_on_rank_zero_only():
    sys.path.insert(0, ROOT)
    import argparse

    import bench

    args = argparse.Namespace(workload="qwen3_8b_b64", steps=1, warmup=1, gpus=2)
    assert bench.run_reference(args, rank=1, world=2) is None     # returns at once, no weights built


def test_workload_recipe_matches_the_named_configuration():
    sys.path.insert(0, ROOT)
    import bench

    sh, B, slots, ctx, T, P, kv_std = bench.workload_inputs("qwen3_8b_b64")
    assert (sh.n_layers, sh.hidden, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.ffn, sh.vocab) == \
        (36, 4096, 32, 8, 128, 12288, 151936)
    assert B == 64 and len(slots) == 40 and len(set(slots.tolist())) == 40
    assert ctx.min() >= 512 and ctx.max() <= 4096 and (T, P) == (0.7, 0.95)
    assert sh.weight_bytes_per_step() == 2 * (36 * (6144 * 4096 + 4096 * 4096 + 24576 * 4096 + 4096 * 12288)
                                              + 151936 * 4096)
    assert sh.kv_bytes_per_token(2) == 147456
