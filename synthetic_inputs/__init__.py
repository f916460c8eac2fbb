"""Seeded synthetic inputs for the KNN-SSD decode hot path.

This module only manufactures *data* (weights, prompts, skip masks, anchors,
request streams).  It holds none of the method's arithmetic: no decoder step,
no cosine search, no acceptance rule.  Both the CPU oracle's tests and the CUDA
path's tests/bench draw their inputs from here, so that the two sides see the
same bits without sharing any code of the method itself.

Everything is a pure function of (seed, tensor id, element index) through a
counter-based integer hash, so any slice of any tensor can be produced on any
device (CPU or CUDA) without generating the rest, and the bits are identical.
"""
from .generators import (  # noqa: F401
    ModelShape,
    SHAPES,
    TensorId,
    hash_u64,
    normal_f32,
    normal_weight,
    uniform_tokens,
    uniforms,
    skip_mask,
    skip_mask_split,
    nested_skip_masks,
    domain_centroids,
    anchors,
    prompt_lengths,
    hash_u64_int,
    request_stream,
    make_model_weights,
    f32_to_bf16_bits,
    bf16_bits_to_f32,
)
