"""Calls from several host threads at once, each on its own stream with its own workspace.

The interface allows them (calls that may run at the same time need workspaces of their own): the work tables
live in one arena per device and a cache of plans shared by all callers, with more distinct problems here than
the cache holds, so plans are built, leased and evicted while other threads launch from them. Every result must
be bit-identical to the same problem run alone afterwards.
"""
import threading

import numpy as np
import pytest
import torch

import hydra_workloads as hw
from gpu_util import pairs_for

pytestmark = pytest.mark.gpu
THREADS, PROBLEMS = 4, 90            # 360 distinct problems, two or three plans each: the cache holds 256 plans


def problem(seed):
    from paper_2609_34318_b200.runner import bits_to_tensor
    rng = np.random.default_rng(seed)
    lengths = [int(v) for v in rng.integers(1, int(rng.choice([60, 400, 1500])), size=int(rng.integers(1, 8)))]
    h = int(rng.integers(1, 5))
    cp_r = [int(v) for v in rng.choice([0, 0, 1, 2], size=len(lengths))]
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    f = lambda d: hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32))
    x = {n: bits_to_tensor(f(d)) for n, d in (("q", hw.D_QK), ("k", hw.D_QK), ("v", hw.D_V), ("do", hw.D_V))}
    lib_pairs, rows, _ = pairs_for(cu, cp_r) if any(cp_r) else (None, 0, None)
    return cu, h, lib_pairs, rows, x


def run(cu, h, lib_pairs, rows, x, stream):
    from paper_2609_34318_b200.runner import AttnStep
    step = AttnStep(cu, h, lib_pairs, rows)
    s = stream.cuda_stream if stream is not None else None
    step.forward(x["q"], x["k"], x["v"], stream=s)
    step.backward(x["q"], x["k"], x["v"], x["do"], stream=s)
    assert step.poll(s)[0] == 0
    return [t.clone() for t in (step.out, step.lse, step.dq, step.dk, step.dv)]


def test_threads_with_their_own_streams_and_workspaces_get_the_results_of_serial_calls():
    problems = {(t, i): problem(424200 + 1000 * t + i) for t in range(THREADS) for i in range(PROBLEMS)}
    torch.cuda.synchronize()
    results, errors = {}, []

    def worker(t):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                for i in range(PROBLEMS):
                    results[(t, i)] = run(*problems[(t, i)], stream)
            stream.synchronize()
        except Exception as e:  # noqa: BLE001
            errors.append((t, repr(e)))

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(THREADS)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    torch.cuda.synchronize()
    assert not errors, errors[:3]
    for key, p in problems.items():
        alone = run(*p, None)
        torch.cuda.synchronize()
        for name, a, b in zip(("out", "lse", "dq", "dk", "dv"), alone, results[key]):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), (key, name)
