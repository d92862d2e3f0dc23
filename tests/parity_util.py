"""Helpers of the GPU parity tests: the tie-tolerant comparison of kept sets and
a one-layer cache with an exact budget."""
import numpy as np
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth

TIE_RTOL = 1e-6


def check_kept(kept_gpu, score_oracle, k, n, L):
    """The GPU's kept list against the oracle's scores for one (sequence, group).

    Returns "exact" or "tie". The list must be strictly ascending, of length
    k + window, end with the whole window, and may differ from the oracle's set
    only in keys whose oracle score lies within 1e-6 (relative) of the k-th
    largest score."""
    kept_gpu = np.asarray(kept_gpu, dtype=np.int64)
    c = max(n - L, 0)
    window = n - c
    assert kept_gpu.shape == (k + window,)
    assert np.all(np.diff(kept_gpu) > 0), "kept indices must ascend strictly"
    assert list(kept_gpu[k:]) == list(range(c, n)), "window must be kept"
    if k == 0 or k == c:
        assert list(kept_gpu[:k]) == list(range(k))
        return "exact"
    want = oracle.select_topk(score_oracle, k, n)[:k]
    G, O = set(kept_gpu[:k].tolist()), set(want.tolist())
    if G == O:
        return "exact"
    tau = np.sort(score_oracle)[::-1][k - 1]
    for j in G - O:
        assert score_oracle[j] >= tau * (1 - TIE_RTOL), (j, score_oracle[j], tau)
    for j in O - G:
        assert score_oracle[j] <= tau * (1 + TIE_RTOL), (j, score_oracle[j], tau)
    return "tie"


def one_layer_cache(w: dict, n: int, k: int, device="cuda", **over):
    """A cache whose single layer receives n tokens and keeps exactly k context
    keys (the budget is forced through the minimum-length bound)."""
    L = w["recent_len"]
    kw = pb.config_from_workload(w, [0.0], n_layers=1, prompt_len=n, min_len=[k + min(L, n)])
    kw.update(over)
    return pb.PyrCache(device=device, **kw)


def tol_for(dtype_name: str) -> float:
    """max-abs tolerance on attention outputs: 2e-2 for bf16, 1e-4 for fp32."""
    return 2e-2 if dtype_name == "bf16" else 1e-4
