"""Seeded synthetic inputs for the MiniCache hot path.

This package only draws random inputs and moves them between the logical
``[batch][token][kv_head][128]`` view and the paged pool layout.  It holds none
of the method's arithmetic (no norms, angles, interpolation, retention,
softmax): the CPU oracle and the CUDA path each receive the bits produced here
and never import one another.
"""
from .workload import (  # noqa: F401
    CONFIGS,
    WorkloadConfig,
    make_pair_tensors,
    make_projection_case,
    make_queries,
    make_new_tokens,
    make_lengths,
    make_block_table,
    to_paged,
    from_paged,
    torch_dtype,
    as_bits,
    quantise_q4,
)
