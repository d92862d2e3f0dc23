"""GPU parity at the full sizes of the workloads, in the launch configuration the
benchmark times: one layer of the schedule at the full batch, checked against the
oracle on sampled (sequence, group) pairs and sampled rows. Every (layer,
sequence, group) call of an attention stack is independent of the others (its
inputs are drawn at the surviving length), so a sample is a complete check of
the calls it covers."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import check_kept, one_layer_cache, tol_for

pytestmark = pytest.mark.gpu
DEV = "cuda"

CASES = [
    # workload, layers of its schedule to run (first, spread middle ones whose lengths are not
    # multiples of 128, the short memory-bound ones at the end), (sequence, group) samples per layer
    ("7b_stack_8x2k", [0, 1, 8, 16, 24, 28, 31], 6),
    ("7b_64x2k", [0, 6, 12, 19, 26, 31], 6),
    ("13b_stack_32x4k", [0, 7, 15, 23, 31, 39], 6),
    ("70b_gqa_16x8k", [0, 16, 32, 48, 64, 79], 4),
    # the shapes of the paper's efficiency tables (short prompts: every layer is memory-bound)
    ("13b_table_32x512", [0, 13, 26, 39], 6),
    ("70b_table_8x256", [0, 40, 79], 4),
]


def _sample_pairs(B, G, count, seed):
    rng = np.random.default_rng(seed)
    pairs = {(0, 0), (B - 1, G - 1)}
    while len(pairs) < count + 2:
        pairs.add((int(rng.integers(B)), int(rng.integers(G))))
    return sorted(pairs)


@pytest.mark.parametrize("name,layers,nsamp", CASES, ids=[c[0] for c in CASES])
def test_full_size_layer_against_oracle(name, layers, nsamp):
    w = dict(synth.CONFIGS[name])
    ratio = synth.ratio_schedule(w)
    budgets = oracle.layer_budgets(w["prompt_len"], w["recent_len"], ratio)
    B, Hq, Hkv, D, L, G = w["batch"], w["n_q_heads"], w["n_kv_heads"], w["head_dim"], w["recent_len"], w["sel_groups"]
    rep = Hq // Hkv
    heads_per_group = Hq // G
    tol = tol_for(w["dtype"])
    w1 = dict(w, max_new_tokens=2)
    ties = exact = 0
    for l in layers:
        bud = budgets[l]
        n, k, c = bud["n_in"], bud["k"], bud["c"]
        cache = one_layer_cache(w1, n, k)
        assert cache.layer_info(0)["k_ctx"] == k
        Q, K, V = synth.stack_layer_inputs(w, l, n, device=DEV)
        out = torch.empty_like(Q)
        cache.prefill_layer(0, Q, K, V, out)
        torch.cuda.synchronize()
        lse = cache.lse(0)
        score = cache.scores(0).clone()
        O0 = out.clone() if G != 1 else None
        if G == 1:
            hidden = w.get("hidden", Hq * D)
            gen = torch.Generator(device=DEV); gen.manual_seed(l)
            rows = torch.randn(B, n, hidden, generator=gen, device=DEV).to(torch.bfloat16)
            rows0 = rows.clone()
            n_out = cache.select_compact(0, K, V, rows, hidden, n * hidden, hidden, 0)
        else:
            n_out = cache.select_compact(0, K, V, out, rep * D, out.stride(0), out.stride(1), rep * D)
        torch.cuda.synchronize()
        assert cache.status() == 0
        assert n_out == bud["n_out"]
        kept_all, pos_all = cache.kept(0)
        Kc, Vc = cache.kv(0)
        rng = np.random.default_rng(100 + l)
        for (b, g) in _sample_pairs(B, G, nsamp, seed=l):
            heads = list(range(g * heads_per_group, (g + 1) * heads_per_group))
            # scores of the group from the recent rows of each of its heads
            E = np.zeros((len(heads), c))
            recent = np.arange(c, n)
            wts = oracle.recent_weights(L)
            for hi, h in enumerate(heads):
                A, lse_ref = oracle.attention_weights(synth.widen(Q[b, :, h]), synth.widen(K[b, :, h // rep]),
                                                      oracle.softmax_scale_default(D), recent)
                E[hi] = oracle.ensemble_score(A, L, wts)
                assert np.abs(synth.widen(lse[b, h, c:]) - lse_ref).max() <= 2e-3
            sc_ref = oracle.pooled_scores(E, 1)[0]
            np.testing.assert_allclose(synth.widen(score[b, g]), sc_ref, rtol=2e-3, atol=1e-30)
            kept = kept_all[b, g].cpu().numpy()
            res = check_kept(kept, sc_ref, k, n, L)
            ties += res == "tie"; exact += res == "exact"
            np.testing.assert_array_equal(pos_all[b, g].cpu().numpy(), kept)
            idx = torch.from_numpy(kept).to(DEV).long()
            # attention output on sampled rows of one head of the group
            h = heads[int(rng.integers(len(heads)))]
            rows_s = np.sort(rng.choice(n, size=48, replace=False))
            rows_s[0], rows_s[-1] = 0, n - 1
            A, _ = oracle.attention_weights(synth.widen(Q[b, :, h]), synth.widen(K[b, :, h // rep]),
                                            oracle.softmax_scale_default(D), rows_s)
            O_ref = A @ synth.widen(V[b, :, h // rep])
            O_src = out if G == 1 else O0
            assert np.abs(synth.widen(O_src[b, torch.from_numpy(rows_s).to(DEV), h]) - O_ref).max() <= tol
            # gathers are byte-exact
            for kvh in ([h // rep] if G != 1 else [int(rng.integers(Hkv))]):
                assert torch.equal(Kc[b, kvh, :n_out], K[b, idx, kvh])
                assert torch.equal(Vc[b, kvh, :n_out], V[b, idx, kvh])
            if G == 1:
                assert torch.equal(rows[b, :n_out], rows0[b, idx])
            else:
                assert torch.equal(out[b, :n_out, g * rep:(g + 1) * rep], O0[b, idx, g * rep:(g + 1) * rep])
        # two decode steps over this layer's cache, checked on sampled (sequence, head) pairs
        for t in range(2):
            q, kn, vn = synth.decode_step_inputs(w, l, t, device=DEV)
            o = torch.empty_like(q)
            ln = cache.layer_info(0)["len_now"]
            cache.decode_attn(0, q, kn, vn, o)
            torch.cuda.synchronize()
            for (b, g) in _sample_pairs(B, Hkv, 2, seed=7 + t):
                Kb, Vb = synth.widen(Kc[b, g:g + 1, :ln]), synth.widen(Vc[b, g:g + 1, :ln])
                qs = synth.widen(q[b, g * rep:(g + 1) * rep])
                want, _, _ = oracle.decode_attention(qs, Kb, Vb, synth.widen(kn[b, g:g + 1]), synth.widen(vn[b, g:g + 1]))
                assert np.abs(synth.widen(o[b, g * rep:(g + 1) * rep]) - want).max() <= tol
            assert torch.equal(Kc[:, :, ln], kn) and torch.equal(Vc[:, :, ln], vn)
        cache.close()
        del Q, K, V, out, cache
        torch.cuda.empty_cache()
    print(f"{name}: {exact} selections identical to the oracle's, {ties} differ only within the 1e-6 tie band")


def test_chained_stack_all_layers_batch2():
    """The 7B-shaped stack at batch 2 through all 32 layers of its schedule in ONE cache: the kept
    set the GPU produced at layer l fixes what layer l + 1 receives (its length and its position
    ids). Every call is compared with the oracle on the inputs the GPU call had (teacher forcing):
    the kept set of sampled heads at every layer, the position chain of every group at every layer."""
    w = dict(synth.CONFIGS["7b_stack_8x2k"], batch=2)
    ratio = synth.ratio_schedule(w)
    budgets = oracle.layer_budgets(w["prompt_len"], w["recent_len"], ratio)
    B, H, D, L, N = w["batch"], w["n_q_heads"], w["head_dim"], w["recent_len"], w["prompt_len"]
    cache = pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio))
    pos_prev = np.broadcast_to(np.arange(N), (B, H, N)).copy()
    wts = oracle.recent_weights(L)
    exact = ties = 0
    heads = [0, 5, 11, 17, 23, 31]
    for l, bud in enumerate(budgets):
        n, k, c = bud["n_in"], bud["k"], bud["c"]
        assert cache.layer_info(l)["n_in"] == n
        Q, K, V = synth.stack_layer_inputs(w, l, n, device=DEV)
        out = torch.empty_like(Q)
        cache.prefill_layer(l, Q, K, V, out)
        n_out = cache.select_compact(l, K, V, out, D, out.stride(0), out.stride(1), D)
        torch.cuda.synchronize()
        assert n_out == bud["n_out"]
        kept_all, pos_all = cache.kept(l)
        kept_np, pos_np = kept_all.cpu().numpy(), pos_all.cpu().numpy()
        for b in range(B):
            for h in heads:
                A, _ = oracle.attention_weights(synth.widen(Q[b, :, h]), synth.widen(K[b, :, h]),
                                                oracle.softmax_scale_default(D), np.arange(c, n))
                res = check_kept(kept_np[b, h], oracle.ensemble_score(A, L, wts), k, n, L)
                exact += res == "exact"; ties += res == "tie"
            # positions: every group, chained through the GPU's own kept sets
            for h in range(H):
                np.testing.assert_array_equal(pos_np[b, h], pos_prev[b, h][kept_np[b, h]])
        pos_prev = np.stack([[pos_prev[b, h][kept_np[b, h]] for h in range(H)] for b in range(B)])
        Kc, Vc = cache.kv(l)
        idx = torch.from_numpy(kept_np[1, 7]).to(DEV).long()
        assert torch.equal(Kc[1, 7, :n_out], K[1, idx, 7]) and torch.equal(Vc[1, 7, :n_out], V[1, idx, 7])
    assert cache.status() == 0
    cache.close()
    print(f"chained 7b stack, batch 2, 32 layers: {exact} sampled selections identical to the oracle's, "
          f"{ties} differ only within the 1e-6 tie band")


@pytest.mark.parametrize("name,layers", [("13b_stack_32x4k", [1, 20, 39]), ("70b_gqa_16x8k", [1, 40])],
                         ids=["13b_stack_32x4k", "70b_gqa_16x8k"])
def test_full_size_select_first_against_oracle(name, layers):
    """Select-first ordering at full size (the configuration bench.py times on the long per-head workloads):
    kept sets under the tie rule, kept output rows on sampled rows, caches byte for byte."""
    w = dict(synth.CONFIGS[name])
    ratio = synth.ratio_schedule(w)
    budgets = oracle.layer_budgets(w["prompt_len"], w["recent_len"], ratio)
    B, Hq, Hkv, D, L, G = w["batch"], w["n_q_heads"], w["n_kv_heads"], w["head_dim"], w["recent_len"], w["sel_groups"]
    rep = Hq // Hkv
    per = Hq // G
    for l in layers:
        bud = budgets[l]
        n, k, c = bud["n_in"], bud["k"], bud["c"]
        cache = one_layer_cache(dict(w, max_new_tokens=0), n, k, flags=pb.PYR_FLAG_SELECT_FIRST)
        Q, K, V = synth.stack_layer_inputs(w, l, n, device=DEV)
        out = torch.empty_like(Q)
        launches = pb.launch_count()
        cache.prefill_layer(0, Q, K, V, out)
        assert pb.launch_count() - launches == 5          # window tiles, score (2), selection, other tiles
        n_out = cache.select_compact(0, K, V, out, per * D, out.stride(0), out.stride(1), per * D)
        torch.cuda.synchronize()
        assert cache.status() == 0 and n_out == bud["n_out"]
        kept_all, _ = cache.kept(0)
        Kc, Vc = cache.kv(0)
        wts = oracle.recent_weights(L)
        rng = np.random.default_rng(300 + l)
        for (b, g) in _sample_pairs(B, G, 3, seed=50 + l):
            heads = list(range(g * per, (g + 1) * per))
            E = np.zeros((len(heads), c))
            for hi, h in enumerate(heads):
                A, _ = oracle.attention_weights(synth.widen(Q[b, :, h]), synth.widen(K[b, :, h // rep]),
                                                oracle.softmax_scale_default(D), np.arange(c, n))
                E[hi] = oracle.ensemble_score(A, L, wts)
            kept = kept_all[b, g].cpu().numpy()
            check_kept(kept, oracle.pooled_scores(E, 1)[0], k, n, L)
            idx = torch.from_numpy(kept).to(DEV).long()
            h = heads[int(rng.integers(len(heads)))]
            js = np.sort(rng.choice(n_out, size=40, replace=False))
            js[0], js[-1] = 0, n_out - 1                       # first kept row and the newest window row
            A, _ = oracle.attention_weights(synth.widen(Q[b, :, h]), synth.widen(K[b, :, h // rep]),
                                            oracle.softmax_scale_default(D), kept[js])
            O_ref = A @ synth.widen(V[b, :, h // rep])
            assert np.abs(synth.widen(out[b, torch.from_numpy(js).to(DEV), h]) - O_ref).max() <= 2e-2
            assert torch.equal(Kc[b, h // rep, :n_out], K[b, idx, h // rep])
            assert torch.equal(Vc[b, h // rep, :n_out], V[b, idx, h // rep])
        cache.close()
        del Q, K, V, out, cache
        torch.cuda.empty_cache()
