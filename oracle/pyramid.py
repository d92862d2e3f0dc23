"""fp64 CPU oracle for PyramidInfer's prefill selection path and the decode
attention that follows it.

TEST INFRASTRUCTURE. Plain numpy in float64, one definition per function, no
blocking, no fusion, no reuse of anything from the CUDA library. Every function
names the passage of the paper (arXiv 2405.12532) it follows. The method is a
heuristic (an importance score, a top-k cut, a gather), so the functions take
the steps of Algorithm 1 in the paper's order; the attention itself is the
textbook definition.

Pins (tests/test_oracle_*.py): causal attention against a library routine,
the ensemble score against explicit loops, a closed form and a row-sum
invariant, the top-k against subset enumeration, budgets against the integer
identities of the schedule, decode against one row of causal attention, the
generation-phase re-selection against the prefill step it must agree with and
against explicit loops, cache bytes against the paper's Section 1 figure.

parity unpinned: the absolute values of the ensemble score and the kept sets
on real text. The paper prints no worked example of either.

Readings of points the paper leaves open (each is a parameter or a stated
choice, repeated where it is used):
  * "top-p" keeps a fraction of the *count* of context keys (Section 3.1.1,
    Figure 3 caption speak of a retention ratio of keys and values).
  * the ratio of layer l is taken against the ORIGINAL context length c_0,
    so the per-layer ratios are absolute, not compounding.
  * the recent window S_r is never evicted (Algorithm 1 slices [:-L];
    Section 5.2 "Recent Sequence Ratio").
  * kept keys stay in ascending original order.
  * layer l attends over everything it received; the cut applies to its
    cache and to what layer l+1 receives.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def softmax_scale_default(head_dim: int) -> float:
    """1/sqrt(D); the paper does not state a scale, this is the usual one."""
    return 1.0 / float(np.sqrt(F64(head_dim)))


def recent_weights(L: int) -> np.ndarray:
    """Weights of the weighted average over the recent window.

    Section 4.1 (Prefill Phase) only says more recent tokens get larger
    weights. Default taken here: a linear ramp w_i = 2(i+1)/(L(L+1)),
    i = 0 the oldest recent query, i = L-1 the newest; the weights sum to 1.
    """
    i = np.arange(L, dtype=F64)
    return 2.0 * (i + 1.0) / (F64(L) * F64(L + 1))


def recent_len_from_ratio(prompt_len: int, ratio: float) -> int:
    """Section 5.2, "Recent Sequence Ratio": the window as a fraction of the input.
    L = floor(ratio * N) clamped to [1, N]; 0 for a negative ratio or an empty prompt."""
    N = int(prompt_len)
    if N < 1 or not ratio >= 0:
        return 0
    return int(min(N, max(1, np.floor(F64(ratio) * F64(N)))))


def layer_budgets(prompt_len: int, recent_len: int, ratio, min_len=None):
    """Per-layer sizes of the pyramid (Algorithm 1: ratio p, its decay, the
    minimum PvC lengths N_l; Section 4.1).

    Returns a list of dicts with n_in (tokens the layer receives), c (its
    context length n_in - L), k (context keys kept) and n_out = k + window.

    k = min(c, max(floor(ratio[l] * c_0), N_l - L, 0)), c_0 = prompt_len - L.
    A layer that receives no more than L tokens has no context and keeps all.
    """
    N, L = int(prompt_len), int(recent_len)
    c0 = max(N - L, 0)
    out = []
    n_in = N
    for l, r in enumerate(ratio):
        c = max(n_in - L, 0)
        window = n_in - c
        want = int(np.floor(F64(r) * F64(c0)))
        floor_l = 0 if min_len is None else int(min_len[l]) - L
        k = min(c, max(want, floor_l, 0))
        out.append({"layer": l, "n_in": n_in, "c": c, "k": k, "n_out": k + window})
        n_in = k + window
    return out


def attention_weights(q: np.ndarray, k: np.ndarray, scale: float, rows=None):
    """Causal softmax weights of one head (Algorithm 1, "compute attention
    weights of KV").

    q [n, D], k [n, D]. Query i sees keys 0..i of the layer's current
    (compacted, order-preserving) sequence. Returns (A, lse): A [len(rows), n]
    with exact zeros at masked entries, lse[i] = log sum_j exp(scale q_i.k_j).
    `rows` restricts the computation to those query rows (same definition).
    """
    q = np.asarray(q, dtype=F64)
    k = np.asarray(k, dtype=F64)
    n = k.shape[0]
    rows = np.arange(n) if rows is None else np.asarray(rows, dtype=np.int64)
    S = F64(scale) * (q[rows] @ k.T)
    hidden = np.arange(n)[None, :] > rows[:, None]
    S = np.where(hidden, -np.inf, S)
    m = S.max(axis=1, keepdims=True)
    P = np.exp(S - m)
    Z = P.sum(axis=1, keepdims=True)
    return P / Z, (m + np.log(Z))[:, 0]


def causal_attention(Q, K, V, scale: float, rows=None):
    """Attention output of every query head of one sequence.

    Q [n, Hq, D], K and V [n, Hkv, D]; query head h reads KV head h // r,
    r = Hq / Hkv. Returns (O [len(rows), Hq, D], lse [Hq, len(rows)]).
    """
    Q = np.asarray(Q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    n, Hq, D = Q.shape
    Hkv = K.shape[1]
    r = Hq // Hkv
    nr = n if rows is None else len(rows)
    O = np.zeros((nr, Hq, D), dtype=F64)
    lse = np.zeros((Hq, nr), dtype=F64)
    for h in range(Hq):
        g = h // r
        A, lse[h] = attention_weights(Q[:, h], K[:, g], scale, rows)
        O[:, h] = A @ V[:, g]
    return O, lse


def ensemble_score(A_recent: np.ndarray, L: int, w: np.ndarray) -> np.ndarray:
    """Ensemble attention weights A_e of one head (Algorithm 1:
    weighted_avg(A[-L:, :-L], dim=-2); Section 4.1).

    A_recent [L, n] holds the softmax rows of the L most recent queries.
    Returns E [n - L]: for each context key the w-weighted sum of the weights
    those queries give it. Keys inside the window are not scored.
    """
    A_recent = np.asarray(A_recent, dtype=F64)
    n = A_recent.shape[1]
    assert A_recent.shape[0] == L and len(w) == L and n >= L
    return np.asarray(w, dtype=F64) @ A_recent[:, : n - L]


def pooled_scores(E_heads: np.ndarray, sel_groups: int) -> np.ndarray:
    """Pool per-head ensemble scores into one score per selection group.

    The paper's algorithm has no head axis. Reading taken: the arithmetic mean
    over the query heads of the group, the groups being consecutive equal
    slices of the head axis (all heads when sel_groups == 1; the heads sharing
    a KV head when sel_groups == Hkv). E_heads [Hq, c] -> [sel_groups, c].
    """
    E_heads = np.asarray(E_heads, dtype=F64)
    Hq, c = E_heads.shape
    per = Hq // sel_groups
    return E_heads.reshape(sel_groups, per, c).mean(axis=1)


def select_topk(score: np.ndarray, k: int, n: int) -> np.ndarray:
    """TopP index followed by the recent window (Algorithm 1: TopP, then the
    window rows that the [:-L] slice never offers for eviction).

    score [c] scores the context keys 0..c-1 of a layer holding n tokens. The k
    largest are kept, an exact tie going to the lower index; the result lists
    them in ascending order followed by c, c+1, ..., n-1.
    """
    score = np.asarray(score)
    c = score.shape[0]
    assert 0 <= k <= c <= n
    order = sorted(range(c), key=lambda j: (-score[j], j))
    top = np.sort(np.asarray(order[:k], dtype=np.int64))
    return np.concatenate([top, np.arange(c, n, dtype=np.int64)])


def gather_rows(x: np.ndarray, kept: np.ndarray, axis: int = 0) -> np.ndarray:
    """Gather(KV, index) of Algorithm 1: rows of x at the kept indices."""
    return np.take(x, np.asarray(kept, dtype=np.int64), axis=axis)


def prefill_layer(Q, K, V, recent_len: int, k_keep: int, sel_groups: int,
                  scale: float | None = None, w=None, pos=None, out_rows=None, reencode: bool = False):
    """One layer of Algorithm 1's prefill branch on a batch.

    Q [B, n, Hq, D], K/V [B, n, Hkv, D] are the layer's inputs for the n tokens
    it received. Steps, in the paper's order: attention weights over all n
    tokens; ensemble score from the last L queries on the context columns;
    pooling per selection group; top-k of k_keep context keys plus the window;
    gather of K, V and positions.

    Returns a dict: O [B, n or len(out_rows), Hq, D], lse [B, Hq, rows],
    score [B, G, c], kept [B, G, k_keep + window], K_kept/V_kept
    [B, Hkv, n_out, D] (KV head g gathered with the kept set of the group that
    contains it), pos_kept [B, G, n_out].
    """
    Q = np.asarray(Q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    B, n, Hq, D = Q.shape
    Hkv = K.shape[2]
    L = int(recent_len)
    G = int(sel_groups)
    assert G in (1, Hkv)
    scale = softmax_scale_default(D) if scale is None else float(scale)
    c = max(n - L, 0)
    Lw = n - c
    w = recent_weights(L) if w is None else np.asarray(w, dtype=F64)
    r = Hq // Hkv
    pos = np.broadcast_to(np.arange(n, dtype=np.int64), (B, G, n)) if pos is None else np.asarray(pos)

    Os, lses, scores, kepts = [], [], [], []
    for b in range(B):
        O, lse = causal_attention(Q[b], K[b], V[b], scale, out_rows)
        Os.append(O)
        lses.append(lse)
        if c > 0:
            E = np.zeros((Hq, c), dtype=F64)
            recent = np.arange(c, n)
            for h in range(Hq):
                A_rec, _ = attention_weights(Q[b, :, h], K[b, :, h // r], scale, recent)
                E[h] = ensemble_score(A_rec, L, w)
            sc = pooled_scores(E, G)
        else:
            sc = np.zeros((G, 0), dtype=F64)
        scores.append(sc)
        kepts.append(np.stack([select_topk(sc[g], k_keep, n) for g in range(G)]))
    kept = np.stack(kepts)
    n_out = k_keep + Lw
    Kk = np.zeros((B, Hkv, n_out, D), dtype=F64)
    Vk = np.zeros((B, Hkv, n_out, D), dtype=F64)
    pk = np.zeros((B, G, n_out), dtype=np.int64)
    for b in range(B):
        for g in range(Hkv):
            idx = kept[b, g if G == Hkv else 0]
            Kk[b, g] = gather_rows(K[b, :, g], idx)
            Vk[b, g] = gather_rows(V[b, :, g], idx)
        for gg in range(G):
            # Appendix A.2: gather the original positions (default), or re-encode from 0 in order
            pk[b, gg] = np.arange(n_out) if reencode else gather_rows(pos[b, gg], kept[b, gg])
    return {"O": np.stack(Os), "lse": np.stack(lses), "score": np.stack(scores),
            "kept": kept, "K_kept": Kk, "V_kept": Vk, "pos_kept": pk}


def decode_attention(q, K_cache, V_cache, k_new, v_new, scale: float | None = None):
    """Generation step over a compressed cache (Section 4.1: the generation
    phase reuses the smaller initial KV cache).

    q [Hq, D]; K_cache/V_cache [Hkv, len, D]; k_new/v_new [Hkv, D] are appended
    first. Every cached key precedes the new token, so there is no mask.
    Returns (out [Hq, D], K_cache', V_cache').
    """
    q = np.asarray(q, dtype=F64)
    Kc = np.concatenate([np.asarray(K_cache, dtype=F64), np.asarray(k_new, dtype=F64)[:, None, :]], axis=1)
    Vc = np.concatenate([np.asarray(V_cache, dtype=F64), np.asarray(v_new, dtype=F64)[:, None, :]], axis=1)
    Hq, D = q.shape
    Hkv = Kc.shape[0]
    r = Hq // Hkv
    scale = softmax_scale_default(D) if scale is None else float(scale)
    out = np.zeros((Hq, D), dtype=F64)
    for h in range(Hq):
        g = h // r
        s = F64(scale) * (Kc[g] @ q[h])
        p = np.exp(s - s.max())
        p = p / p.sum()
        out[h] = p @ Vc[g]
    return out, Kc, Vc


def generation_reselect(Q_recent, K_cache, V_cache, k_keep: int, sel_groups: int,
                        scale: float | None = None, w=None, pos=None):
    """Generation-phase update of one sequence's PvC of one layer (Algorithm 1
    with KV = cat([PvC_past, KV]); Section 4.1, Generation Phase: the recent
    window slides over the generated tokens and the PvCs are re-selected "the
    same as the prefill phase").

    K_cache/V_cache [Hkv, len, D] hold the layer's cache in order: the context
    rows, then the rows of the Lw most recent tokens. Q_recent [Lw, Hq, D]
    holds those tokens' queries, oldest first. Reading taken: the attention
    weights of the window queries are computed over the cache as it is now;
    window query i sees the context and the window rows up to its own (row
    c + i). The ensemble score, its pooling and the top-k are those of the
    prefill step. Algorithm 1 selects only while len(KV) exceeds the layer's
    bound: here, while the context is longer than k_keep.

    Returns a dict: score [G, c], kept [G, n_out] (indices into the cache's
    rows, ascending, the window last), K_kept/V_kept [Hkv, n_out, D],
    pos_kept [G, n_out]; n_out = min(c, k_keep) + Lw.
    """
    Q_recent = np.asarray(Q_recent, dtype=F64)
    K_cache = np.asarray(K_cache, dtype=F64)
    V_cache = np.asarray(V_cache, dtype=F64)
    Lw, Hq, D = Q_recent.shape
    Hkv, n, _ = K_cache.shape
    G = int(sel_groups)
    assert G in (1, Hkv) and n >= Lw
    c = n - Lw
    r = Hq // Hkv
    scale = softmax_scale_default(D) if scale is None else float(scale)
    w = recent_weights(Lw) if w is None else np.asarray(w, dtype=F64)
    pos = np.broadcast_to(np.arange(n, dtype=np.int64), (G, n)) if pos is None else np.asarray(pos)
    k = min(c, int(k_keep))
    E = np.zeros((Hq, c), dtype=F64)
    window = np.arange(c, n)
    for h in range(Hq):
        q_rows = np.zeros((n, D), dtype=F64)
        q_rows[c:] = Q_recent[:, h]                 # only the window's rows are read
        A, _ = attention_weights(q_rows, K_cache[h // r], scale, window)
        E[h] = ensemble_score(A, Lw, w)
    score = pooled_scores(E, G) if c > 0 else np.zeros((G, 0), dtype=F64)
    kept = np.stack([select_topk(score[g], k, n) for g in range(G)])
    n_out = k + Lw
    Kk = np.zeros((Hkv, n_out, D), dtype=F64)
    Vk = np.zeros((Hkv, n_out, D), dtype=F64)
    for g in range(Hkv):
        idx = kept[g if G == Hkv else 0]
        Kk[g] = gather_rows(K_cache[g], idx)
        Vk[g] = gather_rows(V_cache[g], idx)
    pk = np.stack([gather_rows(pos[g], kept[g]) for g in range(G)])
    return {"score": score, "kept": kept, "K_kept": Kk, "V_kept": Vk, "pos_kept": pk}


def cache_capacities(prompt_len, recent_len, ratio, max_new_tokens, min_len=None):
    """Rows each layer's cache must hold: what the layer keeps plus one row
    per generated token."""
    return [b["n_out"] + int(max_new_tokens)
            for b in layer_budgets(prompt_len, recent_len, ratio, min_len)]


def cache_bytes(batch, n_kv_heads, head_dim, elem_bytes, prompt_len, recent_len,
                ratio, max_new_tokens, min_len=None) -> int:
    """Bytes of K plus V over all layers. With every ratio 1 this is the full
    cache 2 * layers * Hkv * D * bytes * B * (N + T) that Section 1 quotes for
    a 7B model at 64 x 2k."""
    caps = cache_capacities(prompt_len, recent_len, ratio, max_new_tokens, min_len)
    return int(sum(2 * batch * n_kv_heads * cap * head_dim * elem_bytes for cap in caps))


def overlap_ratio(pvc_i, pvc_last) -> float:
    """Eq. 1: |PvC_i ∩ PvC_last| / |PvC_last|."""
    a, b = set(int(x) for x in pvc_i), set(int(x) for x in pvc_last)
    return len(a & b) / len(b)
