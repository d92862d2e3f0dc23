"""Select-first ordering (PYR_FLAG_SELECT_FIRST): the query tiles that hold the window, the scores and the
selection run first, the remaining tiles write their kept rows straight to their places. Checked against
the oracle like the default ordering (outputs of kept rows, kept sets under the tie rule, cache rows,
positions) and against the default ordering's result on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import check_kept, one_layer_cache

pytestmark = pytest.mark.gpu
DEV = "cuda"

#        Hq Hkv G  B  n     L    k
SHAPES = [(4, 4, 4, 2, 700, 128, 300),      # window = one tile exactly; ragged last tile
          (8, 2, 2, 1, 1000, 256, 500),     # grouped-query heads: rows of a group's four heads move together
          (4, 4, 1, 2, 900, 130, 400),      # one kept set per sequence; the window straddles a tile
          (2, 2, 2, 1, 2048, 256, 1723),    # the first dropping layer of the 7B schedule
          (2, 2, 2, 2, 300, 256, 10),       # almost everything dropped, context shorter than a tile
          (2, 2, 2, 1, 640, 128, 512)]      # nothing dropped: the default ordering is taken


def _run(w, n, k, Q, K, V, flags):
    cache = one_layer_cache(w, n, k, flags=flags)
    B, Hq, Hkv, D, G = w["batch"], w["n_q_heads"], w["n_kv_heads"], w["head_dim"], w["sel_groups"]
    out = torch.full((B, n, Hq, D), 7.0, device=DEV, dtype=torch.bfloat16)
    cache.prefill_layer(0, Q, K, V, out)
    per = Hq // G
    n_out = cache.select_compact(0, K, V, out, per * D, n * Hq * D, Hq * D, per * D if G > 1 else 0)
    torch.cuda.synchronize()
    assert cache.status() == 0
    kept, pos = cache.kept(0)
    Kc, Vc = cache.kv(0)
    res = dict(out=out, n_out=n_out, kept=kept.cpu().numpy(), pos=pos.cpu().numpy(), Kc=Kc[:, :, :n_out].clone(),
               Vc=Vc[:, :, :n_out].clone())
    cache.close()
    return res


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "-".join(str(x) for x in s))
def test_select_first_matches_oracle_and_default_ordering(shape):
    Hq, Hkv, G, B, n, L, k = shape
    D = 128
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=G, dtype="bf16", batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=0, hitter_frac=0.05, hitter_mag=3.0)
    Q, K, V = synth.stack_layer_inputs(w, 11, n, device=DEV, boost_queries=True)
    first = _run(w, n, k, Q, K, V, pb.PYR_FLAG_SELECT_FIRST)
    plain = _run(w, n, k, Q, K, V, 0)
    ref = oracle.prefill_layer(synth.widen(Q), synth.widen(K), synth.widen(V), L, k, G)
    n_out = first["n_out"]
    assert n_out == plain["n_out"] == min(k, max(n - L, 0)) + min(L, n)
    per = Hq // G
    for b in range(B):
        for g in range(G):
            check_kept(first["kept"][b, g], ref["score"][b, g], min(k, max(n - L, 0)), n, L)
            idx = first["kept"][b, g]
            hs = slice(g * per, (g + 1) * per)
            got = synth.widen(first["out"][b, :n_out, hs])
            assert np.abs(got - ref["O"][b][idx][:, hs]).max() <= 2e-2
            np.testing.assert_array_equal(first["pos"][b, g], idx)
            # same kept set as the default ordering here (no ties at the cut in these inputs): rows agree to
            # bf16 rounding (a tile's key order may differ between the two orderings), caches bit for bit
            np.testing.assert_array_equal(idx, plain["kept"][b, g])
            assert np.abs(got - synth.widen(plain["out"][b, :n_out, hs])).max() <= 2e-2
    assert torch.equal(first["Kc"], plain["Kc"]) and torch.equal(first["Vc"], plain["Vc"])


def test_select_first_over_a_chain_of_layers_with_other_rows():
    """Three layers with shrinking budgets; beside the attention output a second tensor (standing for hidden
    states, one kept set per sequence) is compacted in full by the same call."""
    Hq, Hkv, B, N, L, D = 4, 4, 2, 1100, 128, 128
    w = dict(n_layers=3, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=1, dtype="bf16", batch=B,
             prompt_len=N, recent_len=L, max_new_tokens=4, hitter_frac=0.05, hitter_mag=3.0)
    ratio = [0.9, 0.7, 0.5]
    cache = pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio, flags=pb.PYR_FLAG_SELECT_FIRST))
    budgets = oracle.layer_budgets(N, L, ratio)
    hidden = torch.randn(B, N, 64, device=DEV).to(torch.bfloat16)
    pos = np.tile(np.arange(N), (B, 1))
    for l, bud in enumerate(budgets):
        n, k = bud["n_in"], bud["k"]
        Q, K, V = synth.stack_layer_inputs(w, 20 + l, n, device=DEV, boost_queries=True)
        out = torch.empty(B, n, Hq, D, device=DEV, dtype=torch.bfloat16)
        cache.prefill_layer(l, Q, K, V, out)
        rows = hidden[:, :n].contiguous()
        rows0 = rows.clone()
        n_out = cache.select_compact(l, K, V, rows, 64, n * 64, 64, 0)
        torch.cuda.synchronize()
        assert n_out == bud["n_out"]
        kept, posk = cache.kept(l)
        ref = oracle.prefill_layer(synth.widen(Q), synth.widen(K), synth.widen(V), L, k, 1)
        for b in range(B):
            check_kept(kept[b, 0].cpu().numpy(), ref["score"][b, 0], k, n, L)
            idx = kept[b, 0].long()
            assert torch.equal(rows[b, :n_out], rows0[b, idx])                     # compacted in full
            got = synth.widen(out[b, :int((idx < (n - L) // 128 * 128).sum())])     # rows written in kept order
            want = ref["O"][b][idx.cpu().numpy()][:got.shape[0]]
            assert np.abs(got - want).max() <= 2e-2
            np.testing.assert_array_equal(posk[b, 0].cpu().numpy(), pos[b][idx.cpu().numpy()])
        pos = np.stack([pos[b][kept[b, 0].cpu().numpy()] for b in range(B)])
        hidden = rows
    q = torch.randn(B, Hq, D, device=DEV).to(torch.bfloat16)
    o = torch.empty_like(q)
    cache.decode_attn(0, q, q.clone(), q.clone(), o)
    torch.cuda.synchronize()
    assert cache.status() == 0
    cache.close()


def test_select_first_with_reencoded_positions_and_generation_update():
    """The flag combined with re-encoded positions and the generation-phase update: same kept lists, positions and
    caches as the default ordering, before and after a re-selection during decode."""
    Hq, Hkv, B, N, L, D, T = 4, 2, 2, 900, 128, 128, 6
    w = dict(n_layers=2, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=Hkv, dtype="bf16", batch=B,
             prompt_len=N, recent_len=L, max_new_tokens=T, hitter_frac=0.05, hitter_mag=3.0)
    ratio = [0.8, 0.5]
    base = pb.PYR_FLAG_POS_REENCODE | pb.PYR_FLAG_GEN_RESELECT
    got = []
    for flags in (base | pb.PYR_FLAG_SELECT_FIRST, base):
        cache = pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio, flags=flags))
        snap = []
        for l in range(2):
            n = cache.layer_info(l)["n_in"]
            Q, K, V = synth.stack_layer_inputs(w, 30 + l, n, device=DEV, boost_queries=True)
            out = torch.empty(B, n, Hq, D, device=DEV, dtype=torch.bfloat16)
            cache.prefill_layer(l, Q, K, V, out)
            per = Hq // Hkv
            n_out = cache.select_compact(l, K, V, out, per * D, n * Hq * D, Hq * D, per * D)
            kept, pos = cache.kept(l)
            snap.append((kept.clone(), pos.clone(), n_out))
        for t in range(4):
            q, kn, vn = synth.decode_step_inputs(w, 0, t, device=DEV)
            o = torch.empty_like(q)
            for l in range(2):
                cache.decode_attn(l, q, kn, vn, o)
        for l in range(2):
            cache.decode_reselect(l)
        torch.cuda.synchronize()
        assert cache.status() == 0
        caches = []
        for l in range(2):
            Kc, Vc = cache.kv(l)
            ln = cache.layer_info(l)["len_now"]
            caches.append((Kc[:, :, :ln].clone(), Vc[:, :, :ln].clone()))
        got.append((snap, caches))
        cache.close()
    (s1, c1), (s0, c0) = got
    for l in range(2):
        assert torch.equal(s1[l][0], s0[l][0]) and torch.equal(s1[l][1], s0[l][1]) and s1[l][2] == s0[l][2]
        assert torch.equal(c1[l][0], c0[l][0]) and torch.equal(c1[l][1], c0[l][1])


@pytest.mark.parametrize("dtype,D,flags", [("f32", 64, 0), ("bf16", 64, 0), ("bf16", 128, pb.PYR_FLAG_CUDA_CORE_PREFILL)],
                         ids=["fp32", "bf16-d64", "bf16-cuda-core"])
def test_select_first_falls_back_where_tensor_cores_do_not_apply(dtype, D, flags):
    """With the flag set, configurations outside the tensor-core kernels take the default ordering: same launches,
    same outputs, bit for bit."""
    Hq, Hkv, G, B, n, L, k = 4, 2, 2, 2, 300, 64, 100
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=G, dtype=dtype, batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=0, hitter_frac=0.05, hitter_mag=3.0)
    Q, K, V = synth.stack_layer_inputs(w, 5, n, device=DEV, boost_queries=True)
    res = []
    for f in (flags | pb.PYR_FLAG_SELECT_FIRST, flags):
        cache = one_layer_cache(w, n, k, flags=f)
        out = torch.zeros_like(Q)
        launches = pb.launch_count()
        cache.prefill_layer(0, Q, K, V, out)
        n_prefill = pb.launch_count() - launches
        per = Hq // G
        cache.select_compact(0, K, V, out, per * D, out.stride(0), out.stride(1), per * D)
        torch.cuda.synchronize()
        res.append((out.clone(), cache.kept(0)[0].clone(), n_prefill))
        cache.close()
    assert res[0][2] == res[1][2]
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])
