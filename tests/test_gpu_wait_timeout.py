"""The failure path of the bounded device-side waits, without faulting or hanging anything: a
decode launch whose loader leaves one chunk of cache rows out (a test aid of the library) and
whose waits spin a few thousand times at most. The waits run out, the kernel returns, the status
word says so, and the same cache works again afterwards."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import one_layer_cache, tol_for

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("f32", 64)])
def test_wait_runs_out_is_reported_and_the_cache_recovers(dtype, D):
    Hq = Hkv = 4
    n, L, T = 700, 32, 4
    w = dict(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sel_groups=Hkv, dtype=dtype, batch=2,
             prompt_len=n, recent_len=L, max_new_tokens=T, hitter_frac=0.02, hitter_mag=3.0)
    cache = one_layer_cache(w, n, 300)

    def fill():
        Q, K, V = synth.stack_layer_inputs(w, 0, n, device=DEV)
        cache.prefill_layer(0, Q, K, V, torch.empty_like(Q))
        cache.select_compact(0, K, V)

    fill()
    q, kn, vn = synth.decode_step_inputs(w, 0, 0, device=DEV)
    out = torch.empty_like(q)
    cache.arm_wait_test()
    cache.decode_attn(0, q, kn, vn, out)          # returns: nothing faults, nothing hangs
    torch.cuda.synchronize()
    assert cache.status() == pb.PYR_ERR_TIMEOUT
    # a new prompt batch on the same cache: the record is cleared and every call is right again
    cache.reset()
    fill()
    assert cache.status() == 0
    for t in range(2):
        q, kn, vn = synth.decode_step_inputs(w, 0, t, device=DEV)
        Kc, Vc = cache.kv(0)
        ln = cache.layer_info(0)["len_now"]
        Kb, Vb = synth.widen(Kc[:, :, :ln]), synth.widen(Vc[:, :, :ln])
        cache.decode_attn(0, q, kn, vn, out)
        torch.cuda.synchronize()
        for b in range(2):
            want, _, _ = oracle.decode_attention(synth.widen(q[b]), Kb[b], Vb[b], synth.widen(kn[b]), synth.widen(vn[b]))
            assert np.abs(synth.widen(out[b]) - want).max() <= tol_for(dtype)
    assert cache.status() == 0
    cache.close()
