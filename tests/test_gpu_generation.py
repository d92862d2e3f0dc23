"""Generation-phase PvC update on the GPU against the oracle (Algorithm 1 with
past PvC; Section 4.1, Generation Phase): decode steps append to every layer's
cache, and every few steps each layer's cache is re-selected from the sliding
window of recent queries, so the caches stop growing. Every call is compared on
the inputs the GPU call had (the cache contents are read back before the call)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import check_kept, tol_for

pytestmark = pytest.mark.gpu
DEV = "cuda"

CASES = [
    # dtype, Hq, Hkv, D, G, B, N, L, ratios, T (decode rows reserved), steps, reselect every
    ("bf16", 4, 4, 128, 4, 2, 640, 128, [1.0, 0.6, 0.3], 24, 72, 8),     # 13B-stack shape, reduced: one kept set per head
    ("bf16", 8, 2, 128, 2, 2, 768, 256, [0.8, 0.4], 16, 64, 16),          # 70B-GQA shape, reduced: pooled per KV-head group
    ("bf16", 4, 2, 128, 1, 1, 520, 128, [1.0, 0.5], 8, 64, 5),            # one kept set per sequence
    ("f32", 4, 4, 64, 4, 2, 256, 32, [1.0, 0.5], 16, 66, 11),             # the tiny fp32 geometry
]


@pytest.mark.parametrize("dtype,Hq,Hkv,D,G,B,N,L,ratio,T,steps,every", CASES)
def test_generation_reselect_against_oracle(dtype, Hq, Hkv, D, G, B, N, L, ratio, T, steps, every):
    w = dict(n_layers=len(ratio), n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=G, dtype=dtype, batch=B,
             prompt_len=N, recent_len=L, max_new_tokens=T, hitter_frac=0.02, hitter_mag=3.0)
    cache = pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio, flags=pb.PYR_FLAG_GEN_RESELECT))
    budgets = oracle.layer_budgets(N, L, ratio)
    nL = len(ratio)
    tol = tol_for(dtype)
    window_q = []                     # per layer: list of the recent queries [B, Hq, D], oldest first
    for l, bud in enumerate(budgets):
        n = bud["n_in"]
        Q, K, V = synth.stack_layer_inputs(w, l, n, device=DEV, boost_queries=True)
        cache.prefill_layer(l, Q, K, V, torch.empty_like(Q))
        cache.select_compact(l, K, V)
        window_q.append([Q[:, i].clone() for i in range(n - min(L, n), n)])
    torch.cuda.synchronize()
    wts_full = oracle.recent_weights(L)
    exact = ties = selections = 0
    for t in range(steps):
        for l in range(nL):
            q, kn, vn = synth.decode_step_inputs(w, l, t, device=DEV)
            Kc, Vc = cache.kv(l)
            ln = cache.layer_info(l)["len_now"]
            Kb, Vb = synth.widen(Kc[:, :, :ln]), synth.widen(Vc[:, :, :ln])
            o = torch.empty_like(q)
            cache.decode_attn(l, q, kn, vn, o)
            torch.cuda.synchronize()
            for b in range(B):
                want, _, _ = oracle.decode_attention(synth.widen(q[b]), Kb[b], Vb[b], synth.widen(kn[b]), synth.widen(vn[b]))
                assert np.abs(synth.widen(o[b]) - want).max() <= tol
            window_q[l].append(q.clone())
            window_q[l] = window_q[l][-L:]
        if (t + 1) % every == 0:
            for l, bud in enumerate(budgets):
                Kc, Vc = cache.kv(l)
                ln = cache.layer_info(l)["len_now"]
                K0, V0 = Kc[:, :, :ln].clone(), Vc[:, :, :ln].clone()
                c_ctx, n_out = cache.decode_reselect(l)
                torch.cuda.synchronize()
                Lw = len(window_q[l])
                assert c_ctx == ln - Lw
                k = bud["k"]
                if c_ctx <= k:                       # nothing to evict: the cache is untouched
                    assert n_out == ln and torch.equal(Kc[:, :, :ln], K0)
                    continue
                assert n_out == k + Lw and cache.layer_info(l)["len_now"] == n_out
                kept, score = cache.reselect_views(l, c_ctx, n_out)
                Qw = torch.stack(window_q[l], dim=1)                       # [B, Lw, Hq, D]
                for b in range(B):
                    ref = oracle.generation_reselect(synth.widen(Qw[b]), synth.widen(K0[b]), synth.widen(V0[b]), k, G,
                                                     w=wts_full[L - Lw:])
                    np.testing.assert_allclose(synth.widen(score[b]), ref["score"], rtol=2e-3 if dtype == "bf16" else 2e-4,
                                               atol=1e-30)
                    for g in range(G):
                        res = check_kept(kept[b, g].cpu().numpy(), ref["score"][g], k, ln, Lw)
                        exact += res == "exact"; ties += res == "tie"; selections += 1
                    # the cache after the call: the GPU's own kept rows of the cache before it, byte for byte
                    for hk in range(Hkv):
                        idx = kept[b, hk if G == Hkv else 0].long()
                        assert torch.equal(Kc[b, hk, :n_out], K0[b, hk, idx])
                        assert torch.equal(Vc[b, hk, :n_out], V0[b, hk, idx])
    # the caches stopped growing: every layer is back within its budget plus the steps since the last update
    for l, bud in enumerate(budgets):
        assert cache.layer_info(l)["len_now"] <= bud["k"] + L + (steps % every if steps % every else 0) + every
    assert selections > 0 and cache.status() == 0
    cache.close()
    print(f"{dtype} Hq={Hq} Hkv={Hkv} G={G}: {selections} generation-phase selections, {exact} identical to the "
          f"oracle's, {ties} within the tie band")


def test_reselect_needs_the_flag_and_the_decode_phase():
    w = dict(n_layers=1, n_q_heads=2, n_kv_heads=2, head_dim=64, sel_groups=2, dtype="f32", batch=1,
             prompt_len=96, recent_len=16, max_new_tokens=4, hitter_frac=0.0, hitter_mag=0.0)
    plain = pb.PyrCache(device=DEV, **pb.config_from_workload(w, [0.5]))
    with pytest.raises(pb.PyrError) as e:
        plain.decode_reselect(0)
    assert e.value.status == pb.PYR_ERR_UNSUPPORTED
    plain.close()
    gen = pb.PyrCache(device=DEV, **pb.config_from_workload(w, [0.5], flags=pb.PYR_FLAG_GEN_RESELECT))
    with pytest.raises(pb.PyrError) as e:
        gen.decode_reselect(0)                     # before the prompt has been processed
    assert e.value.status == pb.PYR_ERR_ORDER
    gen.close()
