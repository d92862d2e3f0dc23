"""The decoder glue kernels (pyr_glue_*), one by one, against the oracle's fp64 formulas."""
import numpy as np
import pytest
import torch

from oracle import tiny_llama as tl
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _r(*shape, seed=0, dtype=torch.float32):
    g = torch.Generator(device="cpu"); g.manual_seed(seed)
    return torch.randn(*shape, generator=g).to(dtype).to(DEV)


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 2e-6), (torch.bfloat16, 1e-2)])
def test_glue_kernels_against_fp64(dtype, tol):
    T, d, f, V, H = 37, 96, 200, 77, 3
    x = _r(T, d, seed=1, dtype=dtype)
    g = (1 + 0.1 * _r(d, seed=2)).to(dtype)
    xn = synth.widen(x)
    np.testing.assert_allclose(synth.widen(pb.glue_rmsnorm(x, g)), tl.rmsnorm(xn, synth.widen(g)), rtol=tol, atol=tol)
    w = _r(f, d, seed=3, dtype=dtype) * 0.1                      # [out, in]
    res = _r(T, f, seed=4, dtype=dtype)
    want = xn @ synth.widen(w).T
    scale = np.abs(want).max()
    assert np.abs(synth.widen(pb.glue_linear(x, w)) - want).max() <= tol * max(scale, 1)
    assert np.abs(synth.widen(pb.glue_linear(x, w, res)) - (want + synth.widen(res))).max() <= tol * max(scale, 1) * 2
    gate, up = _r(T, f, seed=5, dtype=dtype), _r(T, f, seed=6, dtype=dtype)
    gn = synth.widen(gate)
    np.testing.assert_allclose(synth.widen(pb.glue_swiglu(gate, up)), gn / (1 + np.exp(-gn)) * synth.widen(up), rtol=tol, atol=tol)
    q = _r(2, T, H, 32, seed=7, dtype=dtype)
    pos = torch.randint(0, 5000, (2, T), generator=torch.Generator().manual_seed(8)).to(torch.int32).to(DEV)
    got = pb.glue_rope_(q.clone(), pos)
    np.testing.assert_allclose(synth.widen(got), tl.rope(synth.widen(q), pos.cpu().numpy()), rtol=tol, atol=tol)
    table = _r(V, d, seed=9, dtype=dtype)
    ids = torch.randint(0, V, (5, 7), generator=torch.Generator().manual_seed(10)).to(torch.int32).to(DEV)
    assert torch.equal(pb.glue_embed(ids, table), table[ids.long()])
    lg = _r(6, 1000, seed=11, dtype=dtype)
    lg[2, 17] = lg[2, 900] = 50.0                                 # a tie: the lower index wins
    lg[4, :] = -3.0
    am = pb.glue_argmax(lg).cpu().numpy()
    assert am[2] == 17 and am[4] == 0
    np.testing.assert_array_equal(am[[0, 1, 3, 5]], synth.widen(lg).argmax(-1)[[0, 1, 3, 5]])
