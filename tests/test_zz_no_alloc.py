"""pyr_decode_attn_noalloc: decode attention for hosts that cannot allocate.

A caller embedded in a serving engine that owns all device memory, or a plugin
that is handed tensors and nothing else, cannot give the library a cache buffer
with a split-K workspace. The entry point tested here keeps that workspace in
an array inside the library image instead. The test drives it through the C
ABI next to pyr_decode_attn on the same cache contents, twice in a row (the
second call finds the first call's partials still in the shared array), and
checks the size limit. It runs last so that a stop-at-first-failure run has
already covered every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import one_layer_cache, tol_for

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype,Hq,Hkv,D,B,n", [("bf16", 8, 2, 128, 2, 2600), ("f32", 4, 4, 64, 1, 1500)])
def test_noalloc_decode_matches_handle_decode_twice(dtype, Hq, Hkv, D, B, n):
    L, T = 32, 2
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=Hkv, dtype=dtype, batch=B,
             prompt_len=n, recent_len=L, max_new_tokens=T, hitter_frac=0.02, hitter_mag=3.0)
    k = (n - L) * 3 // 4
    cache = one_layer_cache(w, n, k)
    Q, K, V = synth.stack_layer_inputs(w, 4, n, device=DEV)
    cache.prefill_layer(0, Q, K, V, torch.empty_like(Q))
    cache.select_compact(0, K, V)
    torch.cuda.synchronize()
    Kc, Vc = cache.kv(0)
    # the no-alloc caller's own cache tensors: a copy of what the handle holds
    Kmine, Vmine = Kc.clone(), Vc.clone()
    length = cache.layer_info(0)["len_now"]
    assert (length + 1 + 127) // 128 > 1          # several splits, so the scratch array is in use
    for t in range(T):
        q, kn, vn = synth.decode_step_inputs(w, 0, t, device=DEV)
        want = torch.empty_like(q)
        cache.decode_attn(0, q, kn, vn, want)
        got = torch.full_like(q, float("nan"))
        st = pb.decode_attn_noalloc(q, kn, vn, got, Kmine, Vmine, length + t)
        assert st == pb.PYR_OK, pb.status_string(st)
        torch.cuda.synchronize()
        err = (got.double() - want.double()).abs().max().item()
        assert err <= tol_for(dtype), err
        # and against the CPU oracle on the same cache contents (rows 0..length+t-1 before the append)
        for b in range(B):
            ref, _, _ = oracle.decode_attention(synth.widen(q[b]), synth.widen(Kc[b, :, : length + t]),
                                                synth.widen(Vc[b, :, : length + t]), synth.widen(kn[b]), synth.widen(vn[b]))
            assert np.abs(synth.widen(got[b]) - ref).max() <= tol_for(dtype)
        assert torch.equal(Kmine[:, :, length + t], kn) and torch.equal(Vmine[:, :, length + t], vn)
        assert torch.equal(Kmine[:, :, : length + t + 1], Kc[:, :, : length + t + 1])
    assert pb.decode_attn_noalloc_status() == 0
    cache.close()


def test_noalloc_one_split_then_several():
    """A short cache takes one split (no scratch), a longer one several: both against the oracle,
    in that order, so the address lookup of the first call serves the second."""
    Hq, Hkv, D, B = 4, 2, 128, 1
    w = dict(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, dtype="bf16", batch=B)
    for length, cap in ((100, 128), (3000, 3072)):
        gen = torch.Generator(device=DEV)
        gen.manual_seed(length)
        Kc = torch.randn(B, Hkv, cap, D, generator=gen, device=DEV).to(torch.bfloat16)
        Vc = torch.randn(B, Hkv, cap, D, generator=gen, device=DEV).to(torch.bfloat16)
        Kc[:, :, length:] = 0
        Vc[:, :, length:] = 0
        q, kn, vn = synth.decode_step_inputs(w, 0, length, device=DEV)
        Kb, Vb = synth.widen(Kc[0, :, :length]), synth.widen(Vc[0, :, :length])
        got = torch.full_like(q, float("nan"))
        launches = pb.launch_count()
        assert pb.decode_attn_noalloc(q, kn, vn, got, Kc, Vc, length) == pb.PYR_OK
        torch.cuda.synchronize()
        assert pb.launch_count() - launches == (1 if length < 128 else 2)
        ref, _, _ = oracle.decode_attention(synth.widen(q[0]), Kb, Vb, synth.widen(kn[0]), synth.widen(vn[0]))
        assert np.abs(synth.widen(got[0]) - ref).max() <= tol_for("bf16")
    assert pb.decode_attn_noalloc_status() == 0


def test_noalloc_rejects_what_does_not_fit():
    B, Hq, Hkv, D, cap = 64, 64, 1, 128, 9000          # 64 * 64 * 4 splits * 130 floats > 4 MiB
    q = torch.zeros(B, Hq, D, device=DEV, dtype=torch.bfloat16)
    kn = torch.zeros(B, Hkv, D, device=DEV, dtype=torch.bfloat16)
    Kc = torch.zeros(B, Hkv, cap, D, device=DEV, dtype=torch.bfloat16)
    out = torch.empty_like(q)
    assert pb.decode_attn_noalloc(q, kn, kn, out, Kc, Kc.clone(), cap - 10) == pb.PYR_ERR_SCRATCH_LIMIT
    assert "scratch" in pb.status_string(pb.PYR_ERR_SCRATCH_LIMIT)
    assert pb.decode_attn_noalloc(q, kn, kn, out, Kc, Kc, cap) == pb.PYR_ERR_CAPACITY
