"""Pins of the fp64 oracle against things other than itself: a library
attention routine, explicit loops, closed forms, invariants, enumeration."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(7)


def _rand(*shape):
    return rng.standard_normal(shape)


# ---- attention: the textbook definition, checked against torch's CPU routine ----
@pytest.mark.parametrize("n,Hq,Hkv,D", [(37, 4, 4, 16), (64, 8, 2, 32)])
def test_causal_attention_matches_library(n, Hq, Hkv, D):
    Q, K, V = _rand(n, Hq, D), _rand(n, Hkv, D), _rand(n, Hkv, D)
    O, lse = oracle.causal_attention(Q, K, V, 1.0 / np.sqrt(D))
    tq = torch.from_numpy(Q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)[None]
    tv = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0]
    np.testing.assert_allclose(O, ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    # lse against a masked logsumexp from the library
    s = (tq[0] @ tk[0].transpose(1, 2)) / np.sqrt(D)
    s = s.masked_fill(torch.triu(torch.ones(n, n, dtype=torch.bool), 1), float("-inf"))
    np.testing.assert_allclose(lse, torch.logsumexp(s, -1).numpy(), rtol=1e-12)


def test_attention_rows_subset_is_same_definition():
    n, D = 50, 8
    q, k = _rand(n, D), _rand(n, D)
    A, lse = oracle.attention_weights(q, k, 0.3)
    rows = [0, 7, 49]
    A2, lse2 = oracle.attention_weights(q, k, 0.3, rows)
    np.testing.assert_allclose(A[rows], A2, rtol=1e-13)
    np.testing.assert_allclose(lse[rows], lse2, rtol=1e-13)
    assert np.all(np.triu(A, 1) == 0.0)
    np.testing.assert_allclose(A.sum(1), 1.0, rtol=1e-13)


def test_transposed_operand_would_fail():
    # q.k^T with distinct q and k is not symmetric: a swapped operand changes A
    n, D = 12, 4
    q, k = _rand(n, D), _rand(n, D)
    A, _ = oracle.attention_weights(q, k, 1.0)
    B, _ = oracle.attention_weights(k, q, 1.0)
    assert np.abs(A - B).max() > 1e-3


# ---- ensemble score ----
def _score_by_loops(q, k, L, w, scale):
    """Full n x n matrix by explicit loops, slice [-L:, :-L], dot with w."""
    n, D = q.shape
    A = [[0.0] * n for _ in range(n)]
    for i in range(n):
        s = [scale * sum(q[i][d] * k[j][d] for d in range(D)) for j in range(i + 1)]
        m = max(s)
        e = [np.exp(x - m) for x in s]
        z = sum(e)
        for j in range(i + 1):
            A[i][j] = e[j] / z
    c = n - L
    return np.array([sum(w[i] * A[c + i][j] for i in range(L)) for j in range(c)])


def test_score_brute_force_loops():
    n, D, L = 19, 5, 6
    q, k = _rand(n, D), _rand(n, D)
    w = oracle.recent_weights(L)
    A, _ = oracle.attention_weights(q, k, 0.7, np.arange(n - L, n))
    E = oracle.ensemble_score(A, L, w)
    np.testing.assert_allclose(E, _score_by_loops(q, k, L, w, 0.7), rtol=1e-12)


def test_score_closed_form_identical_keys():
    # all keys equal => A[i, j] = 1/(i+1) => E[j] = sum_i w_i / (c + i + 1) for every j
    n, D, L = 40, 8, 10
    c = n - L
    q = _rand(n, D)
    k = np.tile(_rand(1, D), (n, 1))
    w = oracle.recent_weights(L)
    A, _ = oracle.attention_weights(q, k, 0.5, np.arange(c, n))
    E = oracle.ensemble_score(A, L, w)
    want = sum(w[i] / (c + i + 1) for i in range(L))
    np.testing.assert_allclose(E, np.full(c, want), rtol=1e-12)


def test_score_row_sum_invariant():
    # context mass + window mass of the weighted rows = sum(w) = 1
    n, D, L = 33, 6, 9
    c = n - L
    q, k = _rand(n, D), _rand(n, D)
    w = oracle.recent_weights(L)
    A, _ = oracle.attention_weights(q, k, 1.0, np.arange(c, n))
    E = oracle.ensemble_score(A, L, w)
    window_mass = float(w @ A[:, c:].sum(1))
    assert abs(E.sum() + window_mass - 1.0) < 1e-13


def test_score_single_query_window():
    # L = 1, w = [1]: the score is the last query's softmax row on the context
    n, D = 17, 4
    q, k = _rand(n, D), _rand(n, D)
    A_full, _ = oracle.attention_weights(q, k, 1.0)
    A, _ = oracle.attention_weights(q, k, 1.0, [n - 1])
    E = oracle.ensemble_score(A, 1, np.array([1.0]))
    np.testing.assert_allclose(E, A_full[-1, : n - 1], rtol=1e-13)


def test_recent_weights_ramp():
    w = oracle.recent_weights(5)
    np.testing.assert_allclose(w, np.array([1, 2, 3, 4, 5]) / 15.0, rtol=1e-15)
    assert abs(oracle.recent_weights(256).sum() - 1.0) < 1e-14
    assert np.all(np.diff(oracle.recent_weights(32)) > 0)   # newest query weighs most


def test_pooling_is_mean_and_head_order_free():
    E = np.abs(_rand(8, 11))
    p1 = oracle.pooled_scores(E, 1)
    np.testing.assert_allclose(p1[0], E.mean(0), rtol=1e-15)
    p2 = oracle.pooled_scores(E, 2)
    np.testing.assert_allclose(p2[1], E[4:].mean(0), rtol=1e-15)
    perm = np.array([3, 1, 0, 2, 6, 7, 5, 4])      # permutes heads inside each group of 4
    np.testing.assert_allclose(oracle.pooled_scores(E[perm], 2), p2, rtol=1e-14)


# ---- budgets ----
def test_budget_identity_small():
    b = oracle.layer_budgets(256, 32, [1.0, 0.5])
    assert [x["n_out"] for x in b] == [256, 144]
    assert [x["k"] for x in b] == [224, 112]
    assert [x["n_in"] for x in b] == [256, 256]


def _golden_schedules():
    rows = []
    with open(os.path.join(GOLDEN, "schedule_budgets.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            head, tail = line.split(":")
            name, layers, N, L, r0, r1 = head.split()
            first, last = tail.split("...")
            rows.append((name, int(layers), int(N), int(L), float(r0), float(r1),
                         [int(x) for x in first.split()], [int(x) for x in last.split()]))
    return rows


@pytest.mark.parametrize("row", _golden_schedules(), ids=lambda r: r[0])
def test_budget_matches_workload_tables(row):
    _, layers, N, L, r0, r1, first, last = row
    ratio = synth.geometric_ratio(layers, r0, r1)
    b = oracle.layer_budgets(N, L, ratio)
    ks = [x["k"] for x in b]
    assert ks[: len(first)] == first
    assert ks[-len(last):] == last
    for l, x in enumerate(b):
        assert x["n_out"] == x["k"] + L
        assert x["k"] <= x["c"] == x["n_in"] - L
        if l:
            assert x["n_in"] == b[l - 1]["n_out"]
            assert x["k"] <= b[l - 1]["k"]                   # the pyramid never widens


def test_budget_edges():
    # window longer than the prompt: nothing to evict, ever
    b = oracle.layer_budgets(20, 32, [0.5, 0.1])
    assert all(x["k"] == 0 and x["n_out"] == 20 for x in b)
    # ratio 0: only the window survives (the "local" strategy of Section 5.1)
    b = oracle.layer_budgets(100, 10, [0.0])
    assert b[0]["n_out"] == 10
    # min PvC length N_l clamps from below and a layer no longer than N_l keeps all
    b = oracle.layer_budgets(100, 10, [0.1, 0.1], min_len=[50, 60])
    assert b[0]["n_out"] == 50 and b[1]["n_out"] == 50
    # k never exceeds what is left
    b = oracle.layer_budgets(100, 10, [0.5, 0.9])
    assert b[1]["k"] == 45


# ---- top-k ----
@pytest.mark.parametrize("c,k", [(6, 0), (6, 3), (9, 4), (12, 5), (7, 7)])
def test_topk_against_subset_enumeration(c, k):
    s = np.abs(_rand(c)) + 0.01
    n = c + 3
    kept = oracle.select_topk(s, k, n)
    assert list(kept[k:]) == list(range(c, n))            # window always kept
    assert np.all(np.diff(kept) > 0)                       # strictly ascending
    best = max(itertools.combinations(range(c), k), key=lambda S: sum(s[j] for j in S))
    assert list(kept[:k]) == sorted(best)


def test_topk_ties_go_to_lower_index():
    kept = oracle.select_topk(np.ones(10), 4, 12)
    assert list(kept) == [0, 1, 2, 3, 10, 11]
    s = np.array([0.5, 0.9, 0.5, 0.5, 0.1])
    assert list(oracle.select_topk(s, 3, 5)) == [0, 1, 2]


def test_topk_scale_invariant_and_planted_key():
    D, n, L = 16, 60, 8
    c = n - L
    q, k = _rand(n, D), _rand(n, D)
    k[17] = 4.0 * q[c:].mean(0) / np.linalg.norm(q[c:].mean(0)) * np.sqrt(D)
    A, _ = oracle.attention_weights(q, k, 1 / np.sqrt(D), np.arange(c, n))
    w = oracle.recent_weights(L)
    E = oracle.ensemble_score(A, L, w)
    kept = oracle.select_topk(E, 5, n)
    assert 17 in kept
    E3 = oracle.ensemble_score(A, L, 3.0 * w)
    np.testing.assert_array_equal(kept, oracle.select_topk(E3, 5, n))


# ---- one full layer: structure ----
def test_prefill_layer_structure_and_ratio_one():
    B, n, Hq, Hkv, D, L = 2, 48, 4, 2, 8, 8
    Q, K, V = _rand(B, n, Hq, D), _rand(B, n, Hkv, D), _rand(B, n, Hkv, D)
    c = n - L
    full = oracle.prefill_layer(Q, K, V, L, c, Hkv)
    # ratio 1 => kept = everything, gather = identity, O = plain causal attention
    assert np.all(full["kept"] == np.arange(n))
    np.testing.assert_array_equal(full["K_kept"], K.transpose(0, 2, 1, 3))
    half = oracle.prefill_layer(Q, K, V, L, 13, Hkv)
    np.testing.assert_array_equal(half["O"], full["O"])      # the cut does not touch this layer's output
    assert half["kept"].shape == (B, Hkv, 13 + L)
    for b in range(B):
        for g in range(Hkv):
            kept = half["kept"][b, g]
            assert list(kept[-L:]) == list(range(c, n))
            assert np.all(np.diff(kept) > 0)
            np.testing.assert_array_equal(half["K_kept"][b, g], K[b, kept, g])
            np.testing.assert_array_equal(half["V_kept"][b, g], V[b, kept, g])
            np.testing.assert_array_equal(half["pos_kept"][b, g], kept)
            # every kept context key scores at least as much as every dropped one
            sc = half["score"][b, g]
            dropped = np.setdiff1d(np.arange(c), kept)
            assert sc[kept[:13]].min() >= sc[dropped].max()
    one = oracle.prefill_layer(Q, K, V, L, 13, 1)
    assert one["kept"].shape == (B, 1, 13 + L)
    np.testing.assert_allclose(one["score"][:, 0], half["score"].mean(1), rtol=1e-13)


def _heads_by_loops(Q, K, L, w, scale, b):
    """Per-head scores of sequence b by explicit loops; query head h reads KV
    head h // (Hq / Hkv), written out here independently of the oracle."""
    Hq, Hkv = Q.shape[2], K.shape[2]
    per_kv = Hq // Hkv
    return np.stack([_score_by_loops(Q[b, :, h], K[b, :, h // per_kv], L, w, scale) for h in range(Hq)])


@pytest.mark.parametrize("G", [2, 1])
def test_prefill_layer_score_grouped_heads_by_loops(G):
    # Hq = 8 query heads over Hkv = 2 KV heads: a wrong head-to-KV-head mapping (h % Hkv in place
    # of h // r), a wrong pooling axis or a missing mean changes the pooled score
    B, n, Hq, Hkv, D, L = 2, 21, 8, 2, 4, 5
    Q, K, V = _rand(B, n, Hq, D), _rand(B, n, Hkv, D), _rand(B, n, Hkv, D)
    w = oracle.recent_weights(L)
    scale = 0.6
    got = oracle.prefill_layer(Q, K, V, L, 7, G, scale=scale)["score"]
    assert got.shape == (B, G, n - L)
    for b in range(B):
        E = _heads_by_loops(Q, K, L, w, scale, b)                      # [Hq, c]
        per = Hq // G
        for g in range(G):
            want = sum(E[g * per + i] for i in range(per)) / per
            np.testing.assert_allclose(got[b, g], want, rtol=1e-12)


def test_default_softmax_scale_is_inverse_sqrt_head_dim():
    assert oracle.softmax_scale_default(64) == 0.125
    assert abs(oracle.softmax_scale_default(128) - 0.08838834764831845) < 1e-16     # 2^-3.5
    assert oracle.softmax_scale_default(16) == 0.25
    # the defaults of the layer and of the decode step against the library's own default scale
    B, n, H, D, L = 1, 24, 2, 16, 4
    Q, K, V = _rand(B, n, H, D), _rand(B, n, H, D), _rand(B, n, H, D)
    out = oracle.prefill_layer(Q, K, V, L, 5, H)
    t = lambda x: torch.from_numpy(x[0]).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(t(Q), t(K), t(V), is_causal=True)[0]
    np.testing.assert_allclose(out["O"][0], ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    w = oracle.recent_weights(L)
    for h in range(H):
        np.testing.assert_allclose(out["score"][0, h], _score_by_loops(Q[0, :, h], K[0, :, h], L, w, 0.25), rtol=1e-12)
    dec, _, _ = oracle.decode_attention(Q[0, n - 1], K[0, : n - 1].transpose(1, 0, 2), V[0, : n - 1].transpose(1, 0, 2),
                                        K[0, n - 1], V[0, n - 1])
    np.testing.assert_allclose(dec, ref[:, n - 1].numpy(), rtol=1e-10, atol=1e-12)


def test_nesting_of_positions_across_layers():
    B, N, H, D, L = 1, 40, 2, 8, 6
    budgets = oracle.layer_budgets(N, L, [1.0, 0.6, 0.3])
    pos = None
    prev = None
    for bud in budgets:
        n = bud["n_in"]
        Q, K, V = _rand(B, n, H, D), _rand(B, n, H, D), _rand(B, n, H, D)
        out = oracle.prefill_layer(Q, K, V, L, bud["k"], H, pos=pos)
        pos = out["pos_kept"]
        assert pos.shape[-1] == bud["n_out"]
        if prev is not None:
            for g in range(H):
                assert set(pos[0, g]) <= set(prev[0, g])
        prev = pos


# ---- decode ----
def test_decode_equals_last_row_of_causal_attention():
    n, Hq, Hkv, D = 21, 4, 2, 8
    Q, K, V = _rand(n + 1, Hq, D), _rand(n + 1, Hkv, D), _rand(n + 1, Hkv, D)
    O, _ = oracle.causal_attention(Q, K, V, 0.4)
    out, Kc, Vc = oracle.decode_attention(Q[n], K[:n].transpose(1, 0, 2), V[:n].transpose(1, 0, 2),
                                          K[n], V[n], 0.4)
    np.testing.assert_allclose(out, O[n], rtol=1e-12, atol=1e-14)
    assert Kc.shape == (Hkv, n + 1, D)
    np.testing.assert_array_equal(Kc[:, n], K[n])
    np.testing.assert_array_equal(Vc[:, n], V[n])


# ---- generation-phase re-selection ----
def _window_scores_by_loops(Qw, K, w, scale):
    """Rectangular causal block by explicit loops: window query i (of Lw) sees cache rows 0..c+i."""
    Lw, D = Qw.shape
    n = K.shape[0]
    c = n - Lw
    E = np.zeros(c)
    for i in range(Lw):
        s = [scale * sum(Qw[i][d] * K[j][d] for d in range(D)) for j in range(c + i + 1)]
        m = max(s)
        e = [np.exp(x - m) for x in s]
        z = sum(e)
        for j in range(c):
            E[j] += w[i] * e[j] / z
    return E


@pytest.mark.parametrize("G", [2, 1])
def test_generation_reselect_by_loops_and_structure(G):
    Hq, Hkv, D, n, Lw, k = 4, 2, 4, 17, 5, 6
    Qw, K, V = _rand(Lw, Hq, D), _rand(Hkv, n, D), _rand(Hkv, n, D)
    w = oracle.recent_weights(Lw)
    out = oracle.generation_reselect(Qw, K, V, k, G, scale=0.8)
    c = n - Lw
    E = np.stack([_window_scores_by_loops(Qw[:, h], K[h // 2], w, 0.8) for h in range(Hq)])
    per = Hq // G
    for g in range(G):
        np.testing.assert_allclose(out["score"][g], sum(E[g * per + i] for i in range(per)) / per, rtol=1e-12)
        kept = out["kept"][g]
        assert kept.shape == (k + Lw,) and np.all(np.diff(kept) > 0)
        assert list(kept[k:]) == list(range(c, n))                      # the window is never evicted
        dropped = np.setdiff1d(np.arange(c), kept)
        assert out["score"][g][kept[:k]].min() >= out["score"][g][dropped].max()
        np.testing.assert_array_equal(out["pos_kept"][g], kept)
    for hk in range(Hkv):
        idx = out["kept"][hk if G == Hkv else 0]
        np.testing.assert_array_equal(out["K_kept"][hk], K[hk, idx])
        np.testing.assert_array_equal(out["V_kept"][hk], V[hk, idx])


def test_generation_reselect_is_the_prefill_operation():
    # on an untouched prompt cache, with the last L prompt queries as the window, the generation-phase
    # update must give the prefill step's scores and kept set (Section 4.1: "the same as the prefill phase")
    B, n, Hq, Hkv, D, L, k = 1, 40, 4, 2, 8, 7, 11
    Q, K, V = _rand(B, n, Hq, D), _rand(B, n, Hkv, D), _rand(B, n, Hkv, D)
    pre = oracle.prefill_layer(Q, K, V, L, k, Hkv)
    gen = oracle.generation_reselect(Q[0, n - L:], K[0].transpose(1, 0, 2), V[0].transpose(1, 0, 2), k, Hkv)
    np.testing.assert_allclose(gen["score"], pre["score"][0], rtol=1e-12)
    np.testing.assert_array_equal(gen["kept"], pre["kept"][0])
    np.testing.assert_array_equal(gen["K_kept"], pre["K_kept"][0])


def test_generation_reselect_edges_and_closed_form():
    Hq, Hkv, D, n, Lw = 2, 2, 4, 30, 6
    c = n - Lw
    Qw, V = _rand(Lw, Hq, D), _rand(Hkv, n, D)
    # a budget that covers the context evicts nothing
    K = _rand(Hkv, n, D)
    out = oracle.generation_reselect(Qw, K, V, c + 3, Hkv)
    assert np.all(out["kept"] == np.arange(n))
    np.testing.assert_array_equal(out["K_kept"], K)
    # budget 0: only the window survives
    out = oracle.generation_reselect(Qw, K, V, 0, 1)
    assert list(out["kept"][0]) == list(range(c, n))
    # identical keys: A[i, j] = 1 / (c + i + 1), so every context key scores sum_i w_i / (c + i + 1)
    Kc = np.tile(_rand(1, 1, D), (Hkv, n, 1))
    w = oracle.recent_weights(Lw)
    out = oracle.generation_reselect(Qw, Kc, V, 4, Hkv)
    want = sum(w[i] / (c + i + 1) for i in range(Lw))
    np.testing.assert_allclose(out["score"], np.full((Hkv, c), want), rtol=1e-12)
    assert list(out["kept"][0][:4]) == [0, 1, 2, 3]                     # ties go to the lower index


def test_generation_reselect_then_decode_reads_the_gathered_cache():
    Hq, Hkv, D, n, Lw, k = 4, 2, 8, 25, 5, 9
    Qw, K, V = _rand(Lw, Hq, D), _rand(Hkv, n, D), _rand(Hkv, n, D)
    out = oracle.generation_reselect(Qw, K, V, k, Hkv)
    q, kn, vn = _rand(Hq, D), _rand(Hkv, D), _rand(Hkv, D)
    got, Kc, _ = oracle.decode_attention(q, out["K_kept"], out["V_kept"], kn, vn)
    assert Kc.shape[1] == k + Lw + 1
    # head 0 by hand over its kept rows
    idx = out["kept"][0]
    s = np.concatenate([K[0, idx] @ q[0], [kn[0] @ q[0]]]) / np.sqrt(D)
    p = np.exp(s - s.max()); p /= p.sum()
    np.testing.assert_allclose(got[0], p @ np.concatenate([V[0, idx], vn[0][None]]), rtol=1e-12)


# ---- cache bytes ----
def test_cache_bytes_full_cache_closed_form_and_paper_figure():
    with open(os.path.join(GOLDEN, "kv_cache_7b_64x2k.txt")) as f:
        row = [ln for ln in f if not ln.startswith("#")][0].split()
    layers, hkv, D, eb, B, N, paper_gb, _ = (int(x) for x in row)
    got = oracle.cache_bytes(B, hkv, D, eb, N, 256, [1.0] * layers, 0)
    assert got == 2 * layers * hkv * D * eb * B * N
    assert abs(got / 1e9 - paper_gb) / paper_gb < 0.06      # "around 72 GB"
    pyr = oracle.cache_bytes(B, hkv, D, eb, N, 256, synth.geometric_ratio(layers, 1.0, 0.3), 128)
    full = oracle.cache_bytes(B, hkv, D, eb, N, 256, [1.0] * layers, 128)
    assert 0.6 < pyr / full < 0.7


def test_overlap_ratio_eq1():
    assert oracle.overlap_ratio([1, 2, 3, 9], [2, 3, 4, 5]) == 0.5
