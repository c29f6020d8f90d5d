"""One rank of an outer ring of context parallelism (Section 5.2 of the paper: a shallow outer ring circulates
the K/V chunks while the inner Ulysses group has already given every rank all tokens of its heads; Section
3.5, Eq. (ring): every step a rank attends its own q chunks to the visiting kv chunks).

Every sequence of the micro-batch is cut into 2 * cp_r zigzag chunks; rank r owns chunks r and 2 * cp_r - 1 - r
of every sequence (its LOCAL q, k, v hold just those rows). At step t the rank holds the kv chunks of rank
(r - t) mod cp_r, computes the chunk pairs of that step with the library's local-layout entry points, folds
their partials into its running (out, lse), and passes the kv chunks on to rank r + 1. In the backward the fp32
accumulators of dk / dv travel with their chunks and arrive home after cp_r hops.

No arithmetic happens here: this module owns buffers, the step schedule (from hydra_zigzag_pairs) and the
exchange. The exchange is behind a small transport interface: `DistTransport` (torch.distributed point-to-point,
NCCL between GPUs; the received chunk lands in this GPU's own memory before any kernel reads it) and whatever a
test supplies. The compute is behind `compute` (the library by default), so that the schedule and the transport
can be exercised without a GPU.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import binding as B


# ------------------------------------------------------------------------------------------------
# schedule (host, integers only)
# ------------------------------------------------------------------------------------------------
class RingSchedule:
    """What every rank owns and which chunk pairs it computes at which step."""

    def __init__(self, cu_seqlens, cp_r: int):
        self.cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
        self.cp_r = int(cp_r)
        assert self.cp_r >= 1
        pairs, _rows, pair_rank, pair_step = B.hydra_zigzag_pairs(self.cu, self.cp_r)
        self.pairs, self.pair_rank, self.pair_step = pairs, pair_rank, pair_step
        n_c = 2 * self.cp_r
        # chunk tables: rank s holds, sequence after sequence, [chunk s | chunk n_c - 1 - s] (empty chunks dropped)
        self.tables: List[np.ndarray] = []
        self.rows: List[int] = []
        for s in range(self.cp_r):
            table, row = [], 0
            for b in range(len(self.cu) - 1):
                length = int(self.cu[b + 1] - self.cu[b])
                for c in (s, n_c - 1 - s):
                    lo, hi = c * length // n_c, (c + 1) * length // n_c
                    if hi > lo:
                        table.append((b, lo, hi - lo, row))
                        row += hi - lo
            self.tables.append(B.as_chunks(table))
            self.rows.append(row)
        self.max_rows = max(max(self.rows), 1)

    def source(self, rank: int, step: int) -> int:
        """The rank whose kv chunks visit `rank` at `step`."""
        return (rank - step) % self.cp_r

    def step_pairs(self, rank: int, step: int) -> Tuple[np.ndarray, int]:
        """The pairs `rank` computes at `step`, each writing its own rows of a step-local partial buffer."""
        sel = self.pairs[(self.pair_rank == rank) & (self.pair_step == step)].copy()
        row = 0
        for i in range(len(sel)):
            sel["part_row"][i] = row
            row += int(sel["q_len"][i])
        return sel, row

    def global_rows(self, rank: int) -> np.ndarray:
        """Row of the packed batch for every local row of `rank` (to scatter / gather in tests and loaders)."""
        out = np.empty(self.rows[rank], dtype=np.int64)
        for c in self.tables[rank]:
            out[c["row"]:c["row"] + c["len"]] = int(self.cu[c["seq"]]) + c["start"] + np.arange(c["len"])
        return out


# ------------------------------------------------------------------------------------------------
# transports
# ------------------------------------------------------------------------------------------------
class DistTransport:
    """Point-to-point exchange over torch.distributed (NCCL between GPUs, gloo on CPU). `shift` sends the
    listed tensors to the next rank of the ring and receives the same shapes from the previous one into
    `recv`; the returned handle's wait() completes both."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def shift(self, send: Sequence, recv: Sequence):
        dist = self.dist
        nxt = dist.get_global_rank(self.group, (self.rank + 1) % self.world) if self.group is not None \
            else (self.rank + 1) % self.world
        prv = dist.get_global_rank(self.group, (self.rank - 1) % self.world) if self.group is not None \
            else (self.rank - 1) % self.world
        import torch
        ops = []
        # raw bytes: every backend moves them, whatever the element type
        for t in send:
            ops.append(dist.P2POp(dist.isend, t.view(torch.uint8), nxt, self.group))
        for t in recv:
            ops.append(dist.P2POp(dist.irecv, t.view(torch.uint8), prv, self.group))
        reqs = dist.batch_isend_irecv(ops) if ops else []

        class _Handle:
            def wait(self_inner):
                for r in reqs:
                    r.wait()
        return _Handle()


# ------------------------------------------------------------------------------------------------
# compute (the library)
# ------------------------------------------------------------------------------------------------
class HydraCompute:
    """The per-step calls of a rank, on local tensors, through the C ABI."""

    def __init__(self, n_heads: int, n_kv_heads: Optional[int] = None, d_qk: int = B.D_QK, d_v: int = B.D_V,
                 softmax_scale: Optional[float] = None):
        self.h, self.h_kv = int(n_heads), int(n_kv_heads or n_heads)
        self.d_qk, self.d_v = int(d_qk), int(d_v)
        self.scale = float(np.float32(1.0 / np.sqrt(np.float32(d_qk)))) if softmax_scale is None else float(softmax_scale)

    def workspace_bytes(self, sched: RingSchedule, rank: int) -> int:
        need = 4096
        for t in range(sched.cp_r):
            pairs, _ = sched.step_pairs(rank, t)
            if len(pairs) == 0:
                continue
            src = sched.source(rank, t)
            need = max(need, B.hydra_workspace_bytes_local(B.HYDRA_WS_BWD, sched.cu, self.h, self.h_kv, self.d_qk, self.d_v,
                                                           sched.tables[rank], sched.rows[rank], sched.tables[src],
                                                           sched.max_rows, pairs))
        return need

    def forward_step(self, sched, rank, step, q, k, v, out, lse, o_part, lse_part, workspace):
        pairs, part_rows = sched.step_pairs(rank, step)
        if len(pairs) == 0:
            return
        src = sched.source(rank, step)
        B.hydra_attn_fwd_local(q, k, v, sched.cu, self.h, self.h_kv, self.d_qk, self.d_v, sched.tables[rank],
                               sched.rows[rank], sched.tables[src], sched.max_rows, pairs, True, self.scale, out, lse,
                               o_part, lse_part, part_rows, workspace)
        B.hydra_lse_merge_local(o_part, lse_part, part_rows, sched.cu, self.h, sched.tables[rank], sched.rows[rank],
                                pairs, step > 0, out, lse, workspace)

    def backward_step(self, sched, rank, step, q, k, v, out, lse, dout, dq_acc, dk_acc, dv_acc, workspace):
        pairs, _ = sched.step_pairs(rank, step)
        if len(pairs) == 0:
            return
        src = sched.source(rank, step)
        B.hydra_attn_bwd_accumulate_local(q, k, v, out, lse, dout, sched.cu, self.h, self.h_kv, self.d_qk, self.d_v,
                                          sched.tables[rank], sched.rows[rank], sched.tables[src], sched.max_rows,
                                          pairs, True, self.scale, dq_acc, dk_acc, dv_acc, workspace)


# ------------------------------------------------------------------------------------------------
# one rank
# ------------------------------------------------------------------------------------------------
class RingRank:
    """Buffers and step loop of one rank. `transport.shift(send, recv)` moves tensors one rank onward."""

    def __init__(self, sched: RingSchedule, rank: int, compute, transport, device="cuda"):
        import torch
        self.torch, self.sched, self.rank, self.compute, self.transport = torch, sched, int(rank), compute, transport
        self.device = torch.device(device)
        h, h_kv, dqk, dv = compute.h, compute.h_kv, compute.d_qk, compute.d_v
        rows, cap = max(sched.rows[rank], 1), sched.max_rows
        bf, f32 = torch.bfloat16, torch.float32
        new = lambda shape, dt: torch.zeros(shape, dtype=dt, device=self.device)
        # two sets of visiting kv buffers: the next step's chunks arrive while this step computes
        self.kv = [(new((cap, h_kv, dqk), bf), new((cap, h_kv, dv), bf)) for _ in range(2)]
        self.out, self.lse = new((rows, h, dv), bf), new((h, rows), f32)
        part_cap = max(max(sched.step_pairs(rank, t)[1] for t in range(sched.cp_r)), 1)
        self.o_part, self.lse_part = new((part_cap, h, dv), bf), new((h, part_cap), f32)
        self.dq_acc = new((rows, h, dqk), f32)
        self.dkv_acc = [(new((cap, h_kv, dqk), f32), new((cap, h_kv, dv), f32)) for _ in range(2)]
        ws = compute.workspace_bytes(sched, rank) if hasattr(compute, "workspace_bytes") else 4096
        # zeroed: a rank whose steps hold no pair (sequences shorter than the number of chunks) launches nothing,
        # and its status block must still read as OK
        self.workspace = torch.zeros(ws, dtype=torch.uint8, device=self.device)
        self.log: List[Tuple[str, int, int]] = []          # (phase, step, source): what ran, for the schedule tests

    def forward(self, q, k, v):
        """q [rows, h, d_qk], k [rows, h_kv, d_qk], v [rows, h_kv, d_v] of this rank's own chunks -> (out, lse)."""
        rows, R = self.sched.rows[self.rank], self.sched.cp_r
        self.q = q
        cur = 0
        self.kv[cur][0][:rows].copy_(k)
        self.kv[cur][1][:rows].copy_(v)
        for t in range(R):
            handle = None
            if t + 1 < R:                                   # pass this step's kv chunks on while they are used
                handle = self.transport.shift(list(self.kv[cur]), list(self.kv[cur ^ 1]))
            self.log.append(("fwd", t, self.sched.source(self.rank, t)))
            self.compute.forward_step(self.sched, self.rank, t, q, self.kv[cur][0], self.kv[cur][1], self.out, self.lse,
                                      self.o_part, self.lse_part, self.workspace)
            if handle is not None:
                handle.wait()
                cur ^= 1
        return self.out, self.lse

    def backward(self, k, v, dout):
        """Needs forward() first. Returns fp32 (dq, dk, dv) of this rank's own rows (round with hydra_grad_cast)."""
        rows, R = self.sched.rows[self.rank], self.sched.cp_r
        cur = 0
        self.kv[cur][0][:rows].copy_(k)
        self.kv[cur][1][:rows].copy_(v)
        self.dq_acc.zero_()
        for a in self.dkv_acc[cur]:
            a.zero_()
        for t in range(R):
            # the kv chunks move on while this step computes (they are only read); the gradients they have
            # gathered follow once this rank has added its share. After the last step that hop brings every
            # accumulator home.
            kv_handle = None
            if t + 1 < R:
                kv_handle = self.transport.shift(list(self.kv[cur]), list(self.kv[cur ^ 1]))
            self.log.append(("bwd", t, self.sched.source(self.rank, t)))
            self.compute.backward_step(self.sched, self.rank, t, self.q, self.kv[cur][0], self.kv[cur][1], self.out,
                                       self.lse, dout, self.dq_acc, self.dkv_acc[cur][0], self.dkv_acc[cur][1],
                                       self.workspace)
            acc_handle = self.transport.shift(list(self.dkv_acc[cur]), list(self.dkv_acc[cur ^ 1]))
            if kv_handle is not None:
                kv_handle.wait()
            acc_handle.wait()
            cur ^= 1
        dk, dv = self.dkv_acc[cur]
        return self.dq_acc[:rows], dk[:rows], dv[:rows]
