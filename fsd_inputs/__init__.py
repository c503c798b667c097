"""Seeded synthetic inputs for the FSD / SD verification step.

This package only manufactures inputs (logits, draft tokens, uniforms, draft
trees).  It contains none of the verification arithmetic: no softmax, no
divergence, no acceptance rule.  Both the CPU oracle's tests and the CUDA
path's tests and benchmark draw their inputs from here so that the two sides
see identical bits.
"""

from .generate import (  # noqa: F401
    CONFIGS,
    ChainInputs,
    TreeInputs,
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    make_chain,
    make_config,
    make_tree,
    tree_unique_rows,
)
