"""Seeded synthetic inputs for the verification round.

This package only *draws inputs* (lengths, block tables, KV bytes, probability
rows, draft tokens, uniforms).  It holds none of the method's arithmetic: no
block copy, no attention, no acceptance rule.  Both the CPU oracle's tests and
the CUDA path's tests/bench read their inputs from here, so the two sides see
the same bytes without sharing any code of their own.
"""
from .gen import (  # noqa: F401
    CONFIGS,
    BatchMeta,
    RoundConfig,
    accept_inputs,
    bf16_to_f32,
    draw_ctx_len,
    draw_gamma_r,
    ragged_index,
    export_tables,
    f32_to_bf16,
    make_batch_meta,
    new_kv,
    pool_layer,
    pool_layer_chunks,
    queries,
    BF16_NAN,
)
