"""fp64 CPU oracle (test infrastructure only).

Only the test-suite, the smoke check and the benchmark's cpu_baseline / reference legs may import
this package.  It shares nothing with the CUDA library: its arithmetic lives in ``hydra_oracle.c``
(plain C, double precision) and in the few integer helpers of ``attention.py``.
"""
from .attention import (  # noqa: F401
    attn_bwd,
    attn_bwd_pairs,
    attn_fwd,
    attn_partial,
    build,
    bwd_prep,
    causal_pairs,
    f64_inputs,
    lse_merge,
    n_threads,
    p_row,
    sample_keys,
    sample_rows,
    spike_bwd,
    usp_factor,
    zigzag_chunks,
    zigzag_rank,
)
from .ulysses import all_to_all, ulysses_pack, ulysses_unpack  # noqa: F401,E402
from .gqa import attn_bwd_gqa, attn_bwd_pairs_gqa, attn_fwd_gqa, expand_kv, reduce_kv  # noqa: F401,E402
