"""The variants of the method the paper describes besides its default: positions re-encoded from 0
after each selection (Appendix A.2), the recent window given as a fraction of the input (Section 5.2),
a fixed number of PvCs per layer under unbounded generation (Section 4.1, last sentence) and the
"local" strategy that keeps only the window (Section 5.1)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import check_kept, tol_for

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _stack(w, ratio, **over):
    return pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio, **over))


def test_positions_reencoded_or_gathered():
    w = dict(n_layers=3, n_q_heads=4, n_kv_heads=2, head_dim=128, sel_groups=2, dtype="bf16", batch=2,
             prompt_len=400, recent_len=64, max_new_tokens=0, hitter_frac=0.02, hitter_mag=3.0)
    ratio = [0.8, 0.5, 0.25]
    for flag, reencode in ((0, False), (pb.PYR_FLAG_POS_REENCODE, True)):
        cache = _stack(w, ratio, flags=flag)
        pos_ref = None
        for l, bud in enumerate(oracle.layer_budgets(400, 64, ratio)):
            n = bud["n_in"]
            Q, K, V = synth.stack_layer_inputs(w, l, n, device=DEV, boost_queries=True)
            cache.prefill_layer(l, Q, K, V, torch.empty_like(Q))
            cache.select_compact(l, K, V)
            torch.cuda.synchronize()
            ref = oracle.prefill_layer(synth.widen(Q), synth.widen(K), synth.widen(V), 64, bud["k"], 2, pos=pos_ref,
                                       reencode=reencode)
            kept, pos = cache.kept(l)
            np.testing.assert_array_equal(kept.cpu().numpy(), ref["kept"])
            np.testing.assert_array_equal(pos.cpu().numpy(), ref["pos_kept"])
            if reencode:
                assert np.all(ref["pos_kept"] == np.arange(bud["n_out"]))
            pos_ref = ref["pos_kept"]
        cache.close()


def test_window_as_a_fraction_of_the_input():
    N = 600
    L = pb.recent_len_from_ratio(N, 0.4)                      # the paper's trade-off: 40 % of the input
    assert L == 240 == oracle.recent_len_from_ratio(N, 0.4)
    w = dict(n_layers=1, n_q_heads=2, n_kv_heads=2, head_dim=128, sel_groups=2, dtype="bf16", batch=1,
             prompt_len=N, recent_len=L, max_new_tokens=0, hitter_frac=0.02, hitter_mag=3.0)
    cache = _stack(w, [0.5])
    Q, K, V = synth.stack_layer_inputs(w, 0, N, device=DEV, boost_queries=True)
    out = torch.empty_like(Q)
    cache.prefill_layer(0, Q, K, V, out)
    n_out = cache.select_compact(0, K, V)
    torch.cuda.synchronize()
    bud = oracle.layer_budgets(N, L, [0.5])[0]
    assert n_out == bud["n_out"] == 180 + 240
    ref = oracle.prefill_layer(synth.widen(Q), synth.widen(K), synth.widen(V), L, bud["k"], 2)
    kept = cache.kept(0)[0].cpu().numpy()
    for g in range(2):
        check_kept(kept[0, g], ref["score"][0, g], bud["k"], N, L)
    assert np.abs(synth.widen(out) - ref["O"]).max() <= tol_for("bf16")
    cache.close()


def test_fixed_pvc_count_and_local_strategy_under_long_generation():
    """ratio 0 with a minimum length keeps exactly `count` context keys per layer (count 0 is the
    "local" strategy: the window alone). With a re-selection every s <= T steps the caches stay
    within count + L + s rows over many more decode steps than T."""
    L, T, s, steps = 64, 8, 8, 48
    counts = [96, 0]
    w = dict(n_layers=2, n_q_heads=4, n_kv_heads=4, head_dim=128, sel_groups=4, dtype="bf16", batch=1,
             prompt_len=512, recent_len=L, max_new_tokens=T, hitter_frac=0.02, hitter_mag=3.0)
    cache = _stack(w, [0.0, 0.0], min_len=[c + L for c in counts], flags=pb.PYR_FLAG_GEN_RESELECT)
    budgets = oracle.layer_budgets(512, L, [0.0, 0.0], min_len=[c + L for c in counts])
    assert [b["k"] for b in budgets] == counts
    for l, bud in enumerate(budgets):
        Q, K, V = synth.stack_layer_inputs(w, l, bud["n_in"], device=DEV)
        cache.prefill_layer(l, Q, K, V, torch.empty_like(Q))
        assert cache.select_compact(l, K, V) == counts[l] + L
    for t in range(steps):
        for l in range(2):
            q, kn, vn = synth.decode_step_inputs(w, l, t, device=DEV)
            Kc, Vc = cache.kv(l)
            ln = cache.layer_info(l)["len_now"]
            assert ln <= counts[l] + L + s
            Kb, Vb = synth.widen(Kc[:, :, :ln]), synth.widen(Vc[:, :, :ln])
            o = torch.empty_like(q)
            cache.decode_attn(l, q, kn, vn, o)
            torch.cuda.synchronize()
            want, _, _ = oracle.decode_attention(synth.widen(q[0]), Kb[0], Vb[0], synth.widen(kn[0]), synth.widen(vn[0]))
            assert np.abs(synth.widen(o[0]) - want).max() <= tol_for("bf16")
        if (t + 1) % s == 0:
            for l in range(2):
                _, n_out = cache.decode_reselect(l)
                assert n_out == counts[l] + L
    assert cache.status() == 0
    cache.close()
