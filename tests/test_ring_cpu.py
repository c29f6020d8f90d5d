"""The outer ring on the CPU: the step schedule (integers only) and the exchange over two and three real gloo
ranks with a stand-in for the compute, so that what is checked is which chunks are where at which step and
that the gradient accumulators come home with every rank's share. The attention arithmetic of a ring is
checked on the GPU (tests/test_gpu_ring_local.py)."""
import json
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import hydra_workloads as hw  # noqa: E402
import oracle  # noqa: E402


def test_schedule_partitions_tokens_and_pairs():
    from paper_2609_34318_b200.ring import RingSchedule
    for lengths, cp_r in (([300, 77, 1001], 2), ([64], 4), ([5, 2, 130], 4), ([262144], 4)):
        cu = hw.cu_seqlens(lengths)
        sched = RingSchedule(cu, cp_r)
        # every token of the batch is owned by exactly one rank, and the local row order is the chunk order
        seen = np.concatenate([sched.global_rows(r) for r in range(cp_r)])
        assert sorted(seen.tolist()) == list(range(int(cu[-1])))
        # the steps of the ranks partition the causal chunk pairs, and each pair's kv chunk is the visitor's
        n = 0
        for r in range(cp_r):
            for t in range(cp_r):
                sel, rows = sched.step_pairs(r, t)
                n += len(sel)
                assert rows == int(sel["q_len"].sum())
                src = sched.source(r, t)
                for p in sel:
                    own_q = [(c["seq"], c["start"], c["len"]) for c in sched.tables[r]]
                    own_k = [(c["seq"], c["start"], c["len"]) for c in sched.tables[src]]
                    assert (p["seq"], p["q_start"], p["q_len"]) in own_q
                    assert (p["seq"], p["k_start"], p["k_len"]) in own_k
        assert n == len(sched.pairs) == len(oracle.causal_pairs(cu, cp_r))
        # the oracle's own zigzag ownership agrees with the tables
        for r in range(cp_r):
            for c in sched.tables[r]:
                chunks = oracle.zigzag_chunks(int(cu[c["seq"] + 1] - cu[c["seq"]]), cp_r)
                idx = chunks.index((int(c["start"]), int(c["len"])))
                assert oracle.zigzag_rank(idx, cp_r) == r


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class StubCompute:
    """Stands in for the library: remembers what visited, and adds this rank's mark to the visiting gradients."""
    def __init__(self, rank):
        self.h = self.h_kv = 1
        self.d_qk, self.d_v = 4, 2
        self.rank = rank
        self.seen = []

    def forward_step(self, sched, rank, step, q, k, v, out, lse, o_part, lse_part, workspace):
        rows = sched.rows[sched.source(rank, step)]
        self.seen.append(("fwd", step, float(k[0, 0, 0]), float(v[rows - 1, 0, 0])))

    def backward_step(self, sched, rank, step, q, k, v, out, lse, dout, dq_acc, dk_acc, dv_acc, workspace):
        self.seen.append(("bwd", step, float(k[0, 0, 0]), float(dk_acc[0, 0, 0])))
        dk_acc += 1.0                       # every rank adds one share
        dv_acc += float(10 ** rank)         # and a mark of its own


def _ring_rank(rank: int, world: int, port: int, out_dir: str):
    from paper_2609_34318_b200.ring import DistTransport, RingRank, RingSchedule
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cu = hw.cu_seqlens([90, 33, 7])
        sched = RingSchedule(cu, world)
        comp = StubCompute(rank)
        rr = RingRank(sched, rank, comp, DistTransport(), device="cpu")
        rows = sched.rows[rank]
        q = torch.zeros((rows, 1, 4), dtype=torch.bfloat16)
        k = torch.full((rows, 1, 4), float(rank + 1), dtype=torch.bfloat16)       # the owner's mark
        v = torch.full((rows, 1, 2), float(-(rank + 1)), dtype=torch.bfloat16)
        rr.forward(q, k, v)
        dq, dk, dv = rr.backward(k, v, torch.zeros((rows, 1, 2), dtype=torch.bfloat16))
        with open(os.path.join(out_dir, f"ring{rank}.json"), "w") as f:
            json.dump({"seen": comp.seen, "log": rr.log, "dk": float(dk.mean()), "dk_min": float(dk.min()),
                       "dv": float(dv[0, 0, 0]), "rows": rows}, f)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_ring_exchange_over_gloo(tmp_path, world):
    port = _free_port()
    mp.spawn(_ring_rank, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        d = json.load(open(tmp_path / f"ring{r}.json"))
        fwd = [s for s in d["seen"] if s[0] == "fwd"]
        bwd = [s for s in d["seen"] if s[0] == "bwd"]
        for t in range(world):
            src = (r - t) % world
            # at step t the visiting chunks carry their owner's mark, in k and in v
            assert fwd[t][1] == t and fwd[t][2] == src + 1 and fwd[t][3] == -(src + 1)
            assert bwd[t][1] == t and bwd[t][2] == src + 1
            # and the gradient accumulator that travels with them has gathered t shares so far
            assert bwd[t][3] == float(t)
        assert [tuple(x) for x in d["log"]] == [("fwd", t, (r - t) % world) for t in range(world)] + \
                                               [("bwd", t, (r - t) % world) for t in range(world)]
        # home again: every rank's share, and every rank's mark
        assert d["dk"] == float(world) and d["dk_min"] == float(world)
        assert d["dv"] == float(sum(10 ** s for s in range(world)))
