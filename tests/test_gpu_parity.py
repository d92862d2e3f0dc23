"""GPU parity: the CUDA library against the fp64 oracle, element by element,
on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import check_kept, one_layer_cache, tol_for

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _run_layer(cache, layer, Q, K, V, rows=None, row_args=None):
    out = torch.empty_like(Q)
    cache.prefill_layer(layer, Q, K, V, out)
    torch.cuda.synchronize()
    info = cache.layer_info(layer)
    res = {"O": out, "lse": cache.lse(layer).clone(), "score": cache.scores(layer).clone()}
    n_out = cache.select_compact(layer, K, V, rows, *(row_args or (0, 0, 0, 0)))
    torch.cuda.synchronize()
    idx, pos = cache.kept(layer)
    res.update(kept=idx.clone(), pos=pos.clone(), n_out=n_out, info=info)
    assert cache.status() == 0
    return res


def _check_layer(w, res, Q, K, V, cache, layer, pos_in=None, score_rtol=2e-3):
    """One pyr_prefill_layer + pyr_select_compact call against the oracle on the same inputs."""
    B, n = Q.shape[0], Q.shape[1]
    L, G, Hkv = w["recent_len"], cache.cfg.sel_groups, w["n_kv_heads"]
    k = res["info"]["k_ctx"]
    ref = oracle.prefill_layer(synth.widen(Q), synth.widen(K), synth.widen(V), L, k, G, pos=pos_in)
    tol = tol_for(w["dtype"])
    O = synth.widen(res["O"])
    assert np.abs(O - ref["O"]).max() <= tol
    assert np.abs(synth.widen(res["lse"]) - ref["lse"]).max() <= (1e-4 if w["dtype"] == "f32" else 2e-3)
    c = max(n - L, 0)
    ties = 0
    if c > 0:
        sc = synth.widen(res["score"])
        np.testing.assert_allclose(sc, ref["score"], rtol=score_rtol, atol=1e-30)
    kept = res["kept"].cpu().numpy()
    pos = res["pos"].cpu().numpy()
    Kc, Vc = cache.kv(layer)
    for b in range(B):
        for g in range(G):
            ties += check_kept(kept[b, g], ref["score"][b, g] if c > 0 else None, k, n, L) == "tie"
            src_pos = np.arange(n) if pos_in is None else np.asarray(pos_in)[b, g]
            np.testing.assert_array_equal(pos[b, g], src_pos[kept[b, g]])
        for h in range(Hkv):
            idx = torch.from_numpy(kept[b, h if G == Hkv else 0]).to(DEV).long()
            assert torch.equal(Kc[b, h, : res["n_out"]], K[b, idx, h])      # byte-exact gather
            assert torch.equal(Vc[b, h, : res["n_out"]], V[b, idx, h])
    assert res["n_out"] == k + (n - c)
    return ref, kept, pos, ties


# ---------------------------------------------------------------- tiny fp32 workload, chained
@pytest.mark.parametrize("sel_groups", [1, 4])
def test_tiny_fp32_chain_and_decode(sel_groups):
    w = synth.scaled_config(synth.CONFIGS["tiny_fp32"], sel_groups=sel_groups)
    ratio = synth.ratio_schedule(w)
    cache = pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio))
    budgets = oracle.layer_budgets(w["prompt_len"], w["recent_len"], ratio)
    assert [b["n_out"] for b in budgets] == [256, 144]
    B, Hq, D = w["batch"], w["n_q_heads"], w["head_dim"]
    pos_in = None
    for l, bud in enumerate(budgets):
        n = bud["n_in"]
        Q, K, V = synth.stack_layer_inputs(w, l, n, device=DEV)
        if sel_groups == 1:
            gen = torch.Generator(device=DEV); gen.manual_seed(77 + l)
            rows = torch.randn(B, n, 256, generator=gen, device=DEV)
            rows0 = rows.clone()
            res = _run_layer(cache, l, Q, K, V, rows, (256, n * 256, 256, 0))
        else:
            # the attention output of each group's heads is what gets compacted
            out_rows = None
            res = _run_layer(cache, l, Q, K, V)
        ref, kept, pos, _ = _check_layer(w, res, Q, K, V, cache, l, pos_in)
        if sel_groups == 1:
            for b in range(B):
                idx = torch.from_numpy(kept[b, 0]).to(DEV).long()
                assert torch.equal(rows[b, : res["n_out"]], rows0[b, idx])
                if res["n_out"] < n:   # rows beyond the kept length are left alone
                    assert torch.equal(rows[b, res["n_out"]:], rows0[b, res["n_out"]:])
        pos_in = pos
    # 16 decode steps per layer over the ragged caches
    for l, bud in enumerate(budgets):
        Kc, Vc = cache.kv(l)
        for t in range(w["max_new_tokens"]):
            q, kn, vn = synth.decode_step_inputs(w, l, t, device=DEV)
            out = torch.empty_like(q)
            ln = cache.layer_info(l)["len_now"]
            assert ln == bud["n_out"] + t
            Kbefore, Vbefore = synth.widen(Kc[:, :, :ln]), synth.widen(Vc[:, :, :ln])
            cache.decode_attn(l, q, kn, vn, out)
            torch.cuda.synchronize()
            for b in range(B):
                want, _, _ = oracle.decode_attention(synth.widen(q[b]), Kbefore[b], Vbefore[b],
                                                     synth.widen(kn[b]), synth.widen(vn[b]))
                assert np.abs(synth.widen(out[b]) - want).max() <= 1e-4
            assert torch.equal(Kc[:, :, ln], kn) and torch.equal(Vc[:, :, ln], vn)
        with pytest.raises(pb.PyrError) as e:
            cache.decode_attn(l, q, kn, vn, out)
        assert e.value.status == pb.PYR_ERR_CAPACITY
    cache.close()


# ---------------------------------------------------------------- one layer, many shapes
SHAPES = [
    # dtype, Hq, Hkv, G, D, B, n, L, k
    ("bf16", 4, 4, 4, 128, 2, 300, 64, 100),       # ragged tail, per-head selection
    ("bf16", 8, 2, 2, 128, 1, 257, 33, 50),        # GQA pooled per KV head, odd sizes
    ("bf16", 8, 2, 1, 128, 2, 384, 128, 96),       # one kept set per sequence
    ("bf16", 4, 4, 4, 64, 1, 200, 16, 77),
    ("f32", 4, 2, 2, 128, 1, 150, 20, 60),
    ("f32", 2, 2, 1, 64, 3, 97, 5, 11),
    ("bf16", 2, 2, 2, 128, 1, 40, 64, 0),          # window longer than the layer: nothing to select
    ("bf16", 2, 2, 2, 128, 1, 130, 30, 0),         # k = 0: only the window survives
    ("bf16", 2, 2, 2, 128, 1, 130, 30, 100),       # k = c: keep everything
    ("bf16", 2, 1, 1, 128, 1, 1, 1, 0),            # a single token
    ("bf16", 2, 2, 2, 128, 1, 1100, 200, 333),     # several key tiles per query tile, ragged last pair
    ("bf16", 4, 1, 1, 128, 2, 1536, 256, 700),     # GQA, six full query-tile pairs
    ("bf16", 2, 2, 2, 128, 1, 900, 640, 100),      # window of five query tiles: two score chunks, the second short
]


@pytest.mark.parametrize("flags", [pb.PYR_FLAG_CUDA_CORE_PREFILL, 0], ids=["cuda_core", "default"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "-".join(str(x) for x in s))
def test_one_layer_shapes(shape, flags):
    dtype, Hq, Hkv, G, D, B, n, L, k = shape
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=G, dtype=dtype, batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=0, hitter_frac=0.05, hitter_mag=3.0)
    cache = one_layer_cache(w, n, k, flags=flags)
    assert cache.layer_info(0)["k_ctx"] == min(k, max(n - L, 0))
    Q, K, V = synth.stack_layer_inputs(w, 3, n, device=DEV, boost_queries=True)
    res = _run_layer(cache, 0, Q, K, V)
    _check_layer(w, res, Q, K, V, cache, 0)
    cache.close()


def test_strided_inputs_and_output_rows_per_group():
    # q/k/v as slices of one fused [B, n, (Hq + 2 Hkv), D] tensor; O rows compacted per KV group
    Hq, Hkv, D, B, n, L, k = 8, 4, 128, 2, 200, 40, 60
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=Hkv, dtype="bf16", batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=0, hitter_frac=0.05, hitter_mag=3.0)
    cache = one_layer_cache(w, n, k)
    gen = torch.Generator(device=DEV); gen.manual_seed(5)
    fused = torch.randn(B, n, Hq + 2 * Hkv, D, generator=gen, device=DEV).to(torch.bfloat16)
    Q, K, V = fused[:, :, :Hq], fused[:, :, Hq:Hq + Hkv], fused[:, :, Hq + Hkv:]
    out = torch.empty(B, n, Hq, D, device=DEV, dtype=torch.bfloat16)
    cache.prefill_layer(0, Q, K, V, out)
    torch.cuda.synchronize()
    O0 = out.clone()
    rep = Hq // Hkv
    n_out = cache.select_compact(0, K, V, out, rep * D, n * Hq * D, Hq * D, rep * D)
    torch.cuda.synchronize()
    kept = cache.kept(0)[0].cpu().numpy()
    ref = oracle.prefill_layer(synth.widen(Q), synth.widen(K), synth.widen(V), L, k, Hkv)
    assert np.abs(synth.widen(O0) - ref["O"]).max() <= 2e-2
    for b in range(B):
        for g in range(Hkv):
            check_kept(kept[b, g], ref["score"][b, g], k, n, L)
            idx = torch.from_numpy(kept[b, g]).to(DEV).long()
            assert torch.equal(out[b, :n_out, g * rep:(g + 1) * rep], O0[b, idx, g * rep:(g + 1) * rep])
    cache.close()


# ---------------------------------------------------------------- selection on planted scores
def _select_with_scores(scores: torch.Tensor, k: int, L: int = 8):
    """Runs a layer, overwrites the scores it left with `scores` [B, G, c], then selects."""
    B, G, c = scores.shape
    n = c + L
    w = dict(n_layers=1, n_q_heads=G, n_kv_heads=G, head_dim=64, sel_groups=G, dtype="f32", batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=0, hitter_frac=0.0, hitter_mag=0.0)
    cache = one_layer_cache(w, n, k)
    Q, K, V = synth.stack_layer_inputs(w, 0, n, device=DEV)
    out = torch.empty_like(Q)
    cache.prefill_layer(0, Q, K, V, out)
    cache.scores(0).copy_(scores)
    cache.select_compact(0, K, V)
    torch.cuda.synchronize()
    kept = cache.kept(0)[0].cpu().numpy()
    cache.close()
    return kept, n


@pytest.mark.parametrize("case", ["all_equal", "many_ties_at_cut", "distinct", "tiny_values", "two_levels",
                                  "long"])
def test_select_bit_exact_on_planted_scores(case):
    g = torch.Generator(device="cpu"); g.manual_seed(11)
    B, G, c, k = 2, 3, 1500, 400
    if case == "all_equal":
        s = torch.full((B, G, c), 0.125)
    elif case == "many_ties_at_cut":
        s = torch.randint(0, 6, (B, G, c), generator=g).float() / 8 + 0.01
    elif case == "distinct":
        s = torch.rand(B, G, c, generator=g)
    elif case == "tiny_values":
        s = torch.rand(B, G, c, generator=g) * 1e-38        # reaches into the subnormals
    elif case == "two_levels":
        s = torch.where(torch.rand(B, G, c, generator=g) < 0.02, torch.tensor(0.5), torch.tensor(1e-4))
    else:
        c, k = 7168, 1433
        s = torch.rand(B, G, c, generator=g).pow(4)
    kept, n = _select_with_scores(s.to(DEV), k)
    for b in range(B):
        for gg in range(G):
            want = oracle.select_topk(s[b, gg].numpy(), k, n)     # exact comparisons on the same fp32 values
            np.testing.assert_array_equal(kept[b, gg], want)


def test_select_is_reproducible():
    g = torch.Generator(device="cpu"); g.manual_seed(3)
    s = (torch.randint(0, 50, (4, 2, 3000), generator=g).float() + 1) / 64
    a, _ = _select_with_scores(s.to(DEV), 900)
    b, _ = _select_with_scores(s.to(DEV), 900)
    np.testing.assert_array_equal(a, b)


# ---------------------------------------------------------------- in-place compaction of wide rows
def test_hidden_rows_compaction_wide():
    Hq, D, B, n, L, k, hidden = 2, 64, 3, 700, 50, 333, 4096
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hq, head_dim=D, sel_groups=1, dtype="bf16", batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=0, hitter_frac=0.05, hitter_mag=3.0)
    cache = one_layer_cache(w, n, k)
    Q, K, V = synth.stack_layer_inputs(w, 1, n, device=DEV)
    gen = torch.Generator(device=DEV); gen.manual_seed(9)
    rows = torch.randn(B, n, hidden, generator=gen, device=DEV).to(torch.bfloat16)
    rows0 = rows.clone()
    out = torch.empty_like(Q)
    cache.prefill_layer(0, Q, K, V, out)
    n_out = cache.select_compact(0, K, V, rows, hidden, n * hidden, hidden, 0)
    torch.cuda.synchronize()
    kept = cache.kept(0)[0]
    for b in range(B):
        assert torch.equal(rows[b, :n_out], rows0[b, kept[b, 0].long()])
        assert torch.equal(rows[b, n_out:], rows0[b, n_out:])
    cache.close()


# ---------------------------------------------------------------- decode over longer caches (split-K)
@pytest.mark.parametrize("dtype,Hq,Hkv,D,B,n", [("bf16", 8, 1, 128, 2, 3000), ("bf16", 4, 4, 128, 3, 1111),
                                                 ("f32", 4, 2, 128, 1, 900), ("bf16", 6, 3, 64, 2, 517),
                                                 ("f32", 3, 3, 64, 2, 140), ("bf16", 16, 2, 128, 1, 2500),
                                                 # 8 heads per KV head, splits long enough to wrap the stage ring
                                                 ("bf16", 64, 8, 128, 4, 6000), ("bf16", 8, 2, 128, 24, 3333)])
def test_decode_split_k(dtype, Hq, Hkv, D, B, n):
    L, T = 32, 3
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=Hkv, dtype=dtype, batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=T, hitter_frac=0.02, hitter_mag=3.0)
    k = (n - L) * 2 // 3
    cache = one_layer_cache(w, n, k)
    Q, K, V = synth.stack_layer_inputs(w, 2, n, device=DEV)
    out = torch.empty_like(Q)
    cache.prefill_layer(0, Q, K, V, out)
    cache.select_compact(0, K, V)
    Kc, Vc = cache.kv(0)
    tol = tol_for(dtype)
    for t in range(T):
        q, kn, vn = synth.decode_step_inputs(w, 0, t, device=DEV)
        o = torch.empty_like(q)
        ln = cache.layer_info(0)["len_now"]
        Kb, Vb = synth.widen(Kc[:, :, :ln]), synth.widen(Vc[:, :, :ln])
        cache.decode_attn(0, q, kn, vn, o)
        torch.cuda.synchronize()
        for b in range(B):
            want, _, _ = oracle.decode_attention(synth.widen(q[b]), Kb[b], Vb[b], synth.widen(kn[b]), synth.widen(vn[b]))
            assert np.abs(synth.widen(o[b]) - want).max() <= tol
        assert torch.equal(Kc[:, :, ln], kn) and torch.equal(Vc[:, :, ln], vn)
    cache.close()


def test_reset_allows_a_new_batch():
    w = synth.CONFIGS["tiny_fp32"]
    ratio = synth.ratio_schedule(w)
    cache = pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio))
    kepts = []
    for rnd in range(2):
        for l, bud in enumerate(oracle.layer_budgets(w["prompt_len"], w["recent_len"], ratio)):
            Q, K, V = synth.stack_layer_inputs(w, l, bud["n_in"], device=DEV)
            res = _run_layer(cache, l, Q, K, V)
            kepts.append(res["kept"].cpu())
        cache.reset()
    assert torch.equal(kepts[0], kepts[2]) and torch.equal(kepts[1], kepts[3])
    cache.close()
