"""Test infrastructure only: a slow fp64 CPU statement of PyramidInfer's
layer-wise pivotal-context selection, written from the paper.

Nothing in the product path may import this package. It shares no code with the
CUDA library; tests, the smoke check and the benchmark's CPU-baseline leg are
its only callers.
"""
from .pyramid import (  # noqa: F401
    softmax_scale_default,
    recent_weights,
    recent_len_from_ratio,
    layer_budgets,
    attention_weights,
    causal_attention,
    ensemble_score,
    pooled_scores,
    select_topk,
    gather_rows,
    prefill_layer,
    decode_attention,
    generation_reselect,
    cache_capacities,
    cache_bytes,
    overlap_ratio,
)
