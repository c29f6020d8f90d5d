"""The failure path of the tensor-core kernels, exercised without faulting, trapping or hanging the GPU.

Every device-side wait in the kernels is bounded: a wait that runs out raises a flag the other roles of the
thread block notice, the block frees its tensor memory, writes HYDRA_ERR_DEVICE_TIMEOUT (with its index) to
the status word and returns. Here the wait is made to run out on purpose with the library's test hook
(hydra_debug_stall): the thread that hands out work idles for 3 ms and then hands out nothing, the limit of
a wait is set to 0.5 ms, so every other role waits for a signal that is never given. Nothing is in flight
when the kernel gives up, the context stays usable, and the same problem run again (hook off, limit
restored) must agree with the oracle.
"""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
from conftest import FWD_SHORT_LEN_DEFAULT
from gpu_util import check, pairs_for, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

CASES = {                       # name -> (kernel to stall, dS hand-off limit in bytes, forward's short-pair limit)
    "forward_cta_pairs": ("HYDRA_STALL_FWD", 4 << 30, 0),
    "forward_short_sequences": ("HYDRA_STALL_FWD", 4 << 30, 1 << 20),
    "backward_key_side": ("HYDRA_STALL_BWD_DKV", 4 << 30, None),
    "backward_query_side_from_ds": ("HYDRA_STALL_BWD_DQ", 4 << 30, None),
    "backward_query_side_recomputing": ("HYDRA_STALL_BWD_DQ", 0, None),
}


@pytest.mark.parametrize("case", list(CASES))
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct(case):
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor
    kernel = getattr(P, CASES[case][0])
    w = hw.workload("tiny")
    x = w.tensors()
    cu = w.cu()
    lib_pairs, rows, ora_pairs = pairs_for(cu, [0, 0, 0, 1])      # the 300-token sequence is cut and merged
    P.hydra_set_bwd_scratch_limit(CASES[case][1])
    if CASES[case][2] is not None:
        P.hydra_set_fwd_short_len(CASES[case][2])
    try:
        step = AttnStep(cu, w.n_heads, lib_pairs, rows)
        q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
        if kernel != P.HYDRA_STALL_FWD:
            step.forward(q, k, v)                                  # a good forward for the backward to follow
            assert step.poll()[0] == 0
        P.hydra_set_wait_limit_ns(500_000)
        P.hydra_debug_stall(kernel, 3_000_000)
        try:
            if kernel == P.HYDRA_STALL_FWD:
                P.hydra_attn_fwd(q, k, v, cu, w.n_heads, lib_pairs, True, step.scale, step.out, step.lse,
                                 step.o_part, step.lse_part, rows, step.workspace)
            else:
                step.backward(q, k, v, do)
            status, detail = step.poll()                           # synchronises the stream: the kernel returned
        finally:
            P.hydra_debug_stall(kernel, 0)
            P.hydra_set_wait_limit_ns(2_000_000_000)
        assert status == P.HYDRA_ERR_DEVICE_TIMEOUT, (case, status)
        assert P.hydra_status_string(status) == "HYDRA_ERR_DEVICE_TIMEOUT"
        assert 0 <= detail < 2 * torch.cuda.get_device_properties(0).multi_processor_count, (case, detail)
        # the context is intact: same problem again, hook off
        got = run_gpu(x, cu, w.n_heads, lib_pairs, rows)
        ref = run_oracle(x, cu, pairs=ora_pairs)
        check(got, ref, label=f"after a timed-out {case}: ")
    finally:
        P.hydra_set_bwd_scratch_limit(4 << 30)
        P.hydra_set_fwd_short_len(FWD_SHORT_LEN_DEFAULT)
