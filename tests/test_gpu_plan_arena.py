"""A new problem shape must cost no device allocation: the work tables live in an arena that the library
allocates once per device, and its halves are recycled when full.

Three hundred distinct problems (new cu_seqlens every time, as in a training loop where every micro-batch is
packed differently) run forward, merge and backward through an arena made small on purpose, so that its
halves are recycled a dozen times and the host-side cache evicts plans; the calls alternate between two
streams, so the waits between a recycling stream and the readers of another stream are exercised too. The
device's free memory must not move after the first call, and every twentieth problem is compared with the
oracle (results computed from recycled tables must still be right)."""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
from gpu_util import check, run_oracle

pytestmark = pytest.mark.gpu
DQK, DV = hw.D_QK, hw.D_V


def test_three_hundred_distinct_shapes_allocate_nothing_and_stay_correct():
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import bits_to_tensor
    h, t_max = 2, 1600
    rng = np.random.default_rng(41)
    bits = {n: hw.f32_to_bf16_bits(rng.standard_normal((t_max, h, DV if n in ("v", "do") else DQK)).astype(np.float32))
            for n in ("q", "k", "v", "do")}
    dev = {n: bits_to_tensor(b) for n, b in bits.items()}
    bf, f32 = torch.bfloat16, torch.float32
    out = torch.empty((t_max, h, DV), dtype=bf, device="cuda")
    dq = torch.empty((t_max, h, DQK), dtype=bf, device="cuda")
    dk = torch.empty((t_max, h, DQK), dtype=bf, device="cuda")
    dv = torch.empty((t_max, h, DV), dtype=bf, device="cuda")
    lse_buf = torch.empty(h * t_max, dtype=f32, device="cuda")
    part_cap = 8 * t_max
    o_part = torch.empty((part_cap, h, DV), dtype=bf, device="cuda")
    lse_part_buf = torch.empty(h * part_cap, dtype=f32, device="cuda")
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]

    def shape(i):
        n_seq = int(rng.integers(1, 6))
        lengths = [int(v) for v in rng.integers(1, 320, n_seq)]
        lengths[0] += i                       # no two problems share their cu_seqlens
        while sum(lengths) > t_max:
            lengths[int(np.argmax(lengths))] //= 2
        cp_r = int(rng.integers(0, 3))
        return lengths, cp_r

    def run(lengths, cp_r, stream):
        cu = hw.cu_seqlens(lengths)
        T = int(cu[-1])
        pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
        assert part_rows <= part_cap
        lse = lse_buf[:h * T].view(h, T)
        lse_part = lse_part_buf[:h * max(part_rows, 1)].view(h, max(part_rows, 1))
        scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
        q, k, v, do = (dev[n][:T] for n in ("q", "k", "v", "do"))
        need = max(P.hydra_workspace_bytes(wk, cu, h, pairs) for wk in (P.HYDRA_WS_FWD, P.HYDRA_WS_MERGE, P.HYDRA_WS_BWD))
        assert need <= ws.numel()
        has_part = bool((pairs["part_row"] >= 0).any())
        P.hydra_attn_fwd(q, k, v, cu, h, pairs, True, scale, out[:T], lse, o_part if has_part else None,
                         lse_part if has_part else None, part_rows, ws, stream=stream)
        if has_part:
            P.hydra_lse_merge(o_part, lse_part, part_rows, cu, h, pairs, out[:T], lse, ws, stream=stream)
        P.hydra_attn_bwd(q, k, v, out[:T], lse, do, cu, h, pairs, True, scale, dq[:T], dk[:T], dv[:T], ws,
                         stream=stream)
        return cu, T, lse

    P.hydra_shutdown()
    P.hydra_set_plan_arena_bytes(64 << 10)          # 32 KB halves: recycled many times below
    try:
        run([37, 200], 1, streams[0])                # first call on the device: the arena is allocated here
        P.hydra_set_bwd_scratch_limit(0)             # and every kernel has been launched once (lazy module
        run([37, 200], 1, streams[0])                # loading takes device memory at a kernel's first launch)
        P.hydra_set_bwd_scratch_limit(4 << 30)
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        checked = 0
        for i in range(300):
            lengths, cp_r = shape(i)
            stream = streams[i % 2]
            # the two streams share the output buffers: order them as a caller with shared buffers would
            stream.wait_stream(streams[(i + 1) % 2])
            cu, T, lse = run(lengths, cp_r, stream)
            assert torch.cuda.mem_get_info()[0] == free0, f"device memory moved at problem {i}"
            if i % 20 == 0:
                stream.synchronize()
                st, detail = P.hydra_poll_status(ws, stream)
                assert st == 0, (i, st, detail)
                x = {n: b[:T] for n, b in bits.items()}
                from oracle import causal_pairs
                ref = run_oracle(x, cu, pairs=causal_pairs(cu, cp_r) if cp_r else None)
                got = {"out": out[:T].cpu().float().numpy().astype(np.float64),
                       "lse": lse.cpu().numpy().astype(np.float64),
                       "dq": dq[:T].cpu().float().numpy().astype(np.float64),
                       "dk": dk[:T].cpu().float().numpy().astype(np.float64),
                       "dv": dv[:T].cpu().float().numpy().astype(np.float64)}
                check(got, ref, label=f"problem {i} {lengths} ring {cp_r}: ")
                checked += 1
        torch.cuda.synchronize()
        assert checked == 15
        assert torch.cuda.mem_get_info()[0] == free0
    finally:
        torch.cuda.synchronize()
        P.hydra_shutdown()
        P.hydra_set_plan_arena_bytes(32 << 20)


def test_results_do_not_depend_on_the_table_prefetch():
    """hydra_attn_fwd builds the tables of the merge and the backward ahead of their calls (host work only); with
    that switched off the same problems must give the same bits."""
    import paper_2609_34318_b200 as P
    from gpu_util import pairs_for, run_gpu
    rng = np.random.default_rng(43)
    cases = [([300, 77, 1001], 1), ([513, 64], 0), ([640, 200, 65], 2)]
    results = {}
    for prefetch in (True, False):
        P.hydra_shutdown()                              # forget every cached table: both passes build their own
        P.hydra_set_plan_prefetch(prefetch)
        try:
            for i, (lengths, cp_r) in enumerate(cases):
                cu = hw.cu_seqlens(lengths)
                T = int(cu[-1])
                r = np.random.default_rng(100 + i)
                x = {n: hw.f32_to_bf16_bits(r.standard_normal((T, 2, DV if n in ("v", "do") else DQK)).astype(np.float32))
                     for n in ("q", "k", "v", "do")}
                lib_pairs, rows, _ = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
                got = run_gpu(x, cu, 2, lib_pairs, rows)
                results[(prefetch, i)] = {n: got[n] for n in ("out", "lse", "dq", "dk", "dv")}
        finally:
            P.hydra_set_plan_prefetch(True)
    for i in range(len(cases)):
        for n in ("out", "lse", "dq", "dk", "dv"):
            assert np.array_equal(results[(True, i)][n], results[(False, i)][n], equal_nan=True), (i, n)
    del rng
