"""fp64 CPU oracle of the decoder glue around the pyramid path for the tiny
Llama-style workload (not from the paper: the workload states "2 layers, hidden
256, 4 heads, head_dim 64, MHA, RoPE"; the rest of the block is the public Llama
layout). TEST INFRASTRUCTURE, plain numpy in float64.

Per layer: RMSNorm -> Q, K, V projections -> rotary embedding at each token's
ORIGINAL position (Appendix A.2, "gather": a kept key keeps its position) ->
one layer of Algorithm 1 (oracle.pyramid.prefill_layer) -> output projection and
residual on the kept rows -> RMSNorm -> SwiGLU MLP -> residual. Only the kept
rows go on to the next layer (Figure 2c: deeper layers compute only the PvC's
keys and values). After the last layer: RMSNorm, the output head on the last
token, argmax with the lowest id winning ties. Decode token t sits at position
N + t and attends over each layer's compressed cache.

Readings (the workload leaves them open): RMSNorm eps 1e-5 with gain 1;
rotate-half pairs (i, i + D/2) with theta_i = 10000^(-2i/D); SwiGLU with
intermediate size 768; vocabulary 1000, output head not tied to the embedding;
one kept set per sequence (mean over all heads), the only reading under which
hidden rows can be dropped.

Pins (tests/test_oracle_tiny_llama.py): rotated q.k depends only on the position
difference and the rotation preserves norms; RMSNorm and SwiGLU against their
formulas on hand values; with every ratio 1 the pyramid model's logits and greedy
tokens equal those of `plain_generate`, a full-cache forward written separately
below that calls none of the pyramid functions.
"""
from __future__ import annotations

import numpy as np

from . import pyramid

F64 = np.float64


def rmsnorm(x, gain, eps: float = 1e-5):
    x = np.asarray(x, dtype=F64)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * np.asarray(gain, dtype=F64)


def rope(x, pos, base: float = 10000.0):
    """x [..., n, H, D], pos [..., n]: rotate the pairs (i, i + D/2) of every head by pos * theta_i."""
    x = np.asarray(x, dtype=F64)
    D = x.shape[-1]
    half = D // 2
    theta = base ** (-2.0 * np.arange(half, dtype=F64) / D)
    ang = np.asarray(pos, dtype=F64)[..., None, None] * theta          # [..., n, 1, half]
    cos, sin = np.cos(ang), np.sin(ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * cos - b * sin, b * cos + a * sin], axis=-1)


def swiglu_mlp(x, Wg, Wu, Wd):
    g = x @ Wg
    return ((g / (1.0 + np.exp(-g))) * (x @ Wu)) @ Wd


def _argmax_lowest(logits):
    return int(np.flatnonzero(logits == logits.max())[0])


def pyramid_generate(W, ids, n_heads: int, recent_len: int, ratio, steps: int, kept_override=None, tokens_override=None):
    """Prefill with pyramid compression (one kept set per sequence), then `steps` greedy decode steps.

    W: dict of float arrays (emb [V, d], per layer l: wq{l}, wk{l}, wv{l}, wo{l} [d, d], wg{l}, wu{l} [d, f],
    wd{l} [f, d], n1{l}, n2{l} [d]; nf [d], head [d, V]). ids [B, N] ints.
    kept_override[l] ([B, n_out] ints), when given, replaces layer l's own top-k (per-call comparison
    with another implementation on identical inputs); tokens_override [B, steps] likewise replaces
    the greedy choice fed to the next step. Returns a dict: logits [B, steps + 1, V], tokens
    [B, steps + 1] (argmax of every logits row), kept (per layer [B, n_out]), scores (per layer [B, c]),
    cache_len (per layer)."""
    W = {k: np.asarray(v, dtype=F64) for k, v in W.items()}
    ids = np.asarray(ids)
    B, N = ids.shape
    nL = sum(1 for k in W if k.startswith("wq"))
    d = W["emb"].shape[1]
    H = n_heads
    D = d // H
    budgets = pyramid.layer_budgets(N, recent_len, ratio)
    x = W["emb"][ids]                                        # [B, N, d]
    pos = np.broadcast_to(np.arange(N), (B, N)).copy()
    caches, kepts, scores = [], [], []
    for l, bud in enumerate(budgets):
        n = x.shape[1]
        assert n == bud["n_in"]
        h = rmsnorm(x, W[f"n1{l}"])
        q = rope((h @ W[f"wq{l}"]).reshape(B, n, H, D), pos)
        k = rope((h @ W[f"wk{l}"]).reshape(B, n, H, D), pos)
        v = (h @ W[f"wv{l}"]).reshape(B, n, H, D)
        out = pyramid.prefill_layer(q, k, v, recent_len, bud["k"], 1, pos=pos[:, None, :])
        kept = out["kept"][:, 0]
        if kept_override is not None and kept_override[l] is not None:
            kept = np.asarray(kept_override[l])
        Kc = np.stack([k[b, kept[b]].transpose(1, 0, 2) for b in range(B)])       # [B, H, n_out, D]
        Vc = np.stack([v[b, kept[b]].transpose(1, 0, 2) for b in range(B)])
        caches.append([Kc, Vc])
        kepts.append(kept)
        scores.append(out["score"][:, 0])
        xk = np.stack([x[b, kept[b]] for b in range(B)])
        ok = np.stack([out["O"][b, kept[b]].reshape(-1, d) for b in range(B)])
        y = xk + ok @ W[f"wo{l}"]
        x = y + swiglu_mlp(rmsnorm(y, W[f"n2{l}"]), W[f"wg{l}"], W[f"wu{l}"], W[f"wd{l}"])
        pos = np.stack([pos[b, kept[b]] for b in range(B)])
    logits = [rmsnorm(x[:, -1], W["nf"]) @ W["head"]]
    for t in range(steps):
        prev = np.array([_argmax_lowest(logits[-1][b]) for b in range(B)])
        if tokens_override is not None:
            prev = np.asarray(tokens_override)[:, t]
        xt = W["emb"][prev]                                  # [B, d]
        p = N + t
        for l in range(nL):
            h = rmsnorm(xt, W[f"n1{l}"])
            q = rope((h @ W[f"wq{l}"]).reshape(B, 1, H, D), np.full((B, 1), p))[:, 0]
            k = rope((h @ W[f"wk{l}"]).reshape(B, 1, H, D), np.full((B, 1), p))[:, 0]
            v = (h @ W[f"wv{l}"]).reshape(B, H, D)
            o = np.zeros((B, H, D), dtype=F64)
            for b in range(B):
                o[b], Kn, Vn = pyramid.decode_attention(q[b], caches[l][0][b], caches[l][1][b], k[b], v[b])
                if b == 0:
                    Ks, Vs = [Kn], [Vn]
                else:
                    Ks.append(Kn); Vs.append(Vn)
            caches[l] = [np.stack(Ks), np.stack(Vs)]
            y = xt + o.reshape(B, d) @ W[f"wo{l}"]
            xt = y + swiglu_mlp(rmsnorm(y, W[f"n2{l}"]), W[f"wg{l}"], W[f"wu{l}"], W[f"wd{l}"])
        logits.append(rmsnorm(xt, W["nf"]) @ W["head"])
    logits = np.stack(logits, axis=1)
    tokens = np.array([[_argmax_lowest(logits[b, t]) for t in range(steps + 1)] for b in range(B)])
    return {"logits": logits, "tokens": tokens, "kept": kepts, "scores": scores,
            "cache_len": [c[0].shape[2] for c in caches]}


def plain_generate(W, ids, n_heads: int, steps: int):
    """Full-cache greedy generation, written on its own (explicit masked softmax, no pyramid
    function): what the pyramid model must reproduce when every ratio is 1."""
    W = {k: np.asarray(v, dtype=F64) for k, v in W.items()}
    ids = np.asarray(ids)
    B = ids.shape[0]
    nL = sum(1 for k in W if k.startswith("wq"))
    d = W["emb"].shape[1]
    H = n_heads
    D = d // H
    toks = ids.copy()
    all_logits = []
    for t in range(steps + 1):
        n = toks.shape[1]
        x = W["emb"][toks]
        pos = np.arange(n)
        for l in range(nL):
            h = rmsnorm(x, W[f"n1{l}"])
            q = rope((h @ W[f"wq{l}"]).reshape(B, n, H, D), pos)
            k = rope((h @ W[f"wk{l}"]).reshape(B, n, H, D), pos)
            v = (h @ W[f"wv{l}"]).reshape(B, n, H, D)
            s = np.einsum("bihd,bjhd->bhij", q, k) / np.sqrt(D)
            s = np.where(np.triu(np.ones((n, n), dtype=bool), 1), -np.inf, s)
            s = s - s.max(-1, keepdims=True)
            a = np.exp(s)
            a = a / a.sum(-1, keepdims=True)
            o = np.einsum("bhij,bjhd->bihd", a, v).reshape(B, n, d)
            y = x + o @ W[f"wo{l}"]
            x = y + swiglu_mlp(rmsnorm(y, W[f"n2{l}"]), W[f"wg{l}"], W[f"wu{l}"], W[f"wd{l}"])
        lg = rmsnorm(x[:, -1], W["nf"]) @ W["head"]
        all_logits.append(lg)
        nxt = np.array([_argmax_lowest(lg[b]) for b in range(B)])
        toks = np.concatenate([toks, nxt[:, None]], axis=1)
    logits = np.stack(all_logits, axis=1)
    return {"logits": logits, "tokens": toks[:, ids.shape[1]:]}
