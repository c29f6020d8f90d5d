"""The N > 1 path of bench.py on CPU: two gloo ranks on 127.0.0.1.

What the multi-GPU run adds to the single-GPU one is host logic only (the path shards by replicas:
every rank processes its own microbatch, no data-path collective): the max-over-ranks timing, the
whole-job aggregate, per-rank input seeds, and the reference arm running on rank 0 alone.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import hydra_workloads as hw  # noqa: E402


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        slowest = bench.max_over_ranks(mine, dist, "cpu")
        value = bench.whole_job_value(world, 2.0e12, 4, slowest)
        # every rank draws its own microbatch: same shapes, different seed
        bits = hw.tensor_bits("q", 16, [0], seed=hw.SEED + rank)
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump({"slowest": slowest, "value": value, "checksum": int(bits.astype(np.int64).sum())}, f)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"rank{i}.json")) for i in range(world)]
    assert r[0]["slowest"] == r[1]["slowest"] == 15.0
    # 2 ranks x 2 TFLOP x 4 steps in 15 ms
    assert r[0]["value"] == pytest.approx(2 * 2.0 * 4 / 15e-3)
    assert r[0]["value"] == r[1]["value"]
    assert r[0]["checksum"] != r[1]["checksum"]        # different microbatches


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_weak_scaling_aggregate_is_linear_in_ranks():
    one = bench.whole_job_value(1, 1.0e12, 10, 5.0)
    eight = bench.whole_job_value(8, 1.0e12, 10, 5.0)
    assert eight == pytest.approx(8 * one)


def _ulysses_rank(rank: int, world: int, port: int, out_dir: str):
    """One rank of a Ulysses group over gloo: pack, a real all-to-all, check the head split; then the way
    back through a second all-to-all and unpack."""
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n, h, d = 5, 6, 4
        hg = h // world
        X = np.arange(world * n * h * d, dtype=np.int64).reshape(world * n, h, d).astype(np.uint16)   # same on all ranks
        mine = X[rank * n:(rank + 1) * n]
        # the transport carries the 16-bit elements widened to int32 (gloo has no 16-bit all-to-all)
        send = torch.from_numpy(oracle.ulysses_pack(mine, world).astype(np.int32))
        recv = torch.empty_like(send)
        dist.all_to_all_single(recv, send)                           # equal blocks along dim 0
        got = recv.numpy().astype(np.uint16).reshape(world * n, hg, d)
        ok_in = bool(np.array_equal(got, X[:, rank * hg:(rank + 1) * hg, :]))
        back = torch.from_numpy(got.reshape(world, n, hg, d).astype(np.int32))
        recv2 = torch.empty_like(back)
        dist.all_to_all_single(recv2, back)
        ok_out = bool(np.array_equal(oracle.ulysses_unpack(recv2.numpy().astype(np.uint16)), mine))
        with open(os.path.join(out_dir, f"uly{rank}.json"), "w") as f:
            json.dump({"in": ok_in, "out": ok_out}, f)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_ulysses_pack_unpack_around_a_real_all_to_all(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_ulysses_rank, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for i in range(world):
        r = json.load(open(tmp_path / f"uly{i}.json"))
        assert r["in"] and r["out"]
