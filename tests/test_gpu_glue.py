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


@pytest.mark.parametrize("M,N,K,res", [(300, 512, 256, False), (64, 4096, 4096, True), (2048, 11008, 4096, True),
                                       (129, 1000, 64, False), (5000, 4096, 11008, False), (1, 32000, 4096, False)])
def test_tensor_core_linear_against_fp64_samples(M, N, K, res):
    """bf16 pyr_glue_linear with K a multiple of 64 runs on the tcgen05 GEMM: sampled entries (first and
    last rows and columns among them) against fp64 dot products of the bf16 inputs, untouched padding."""
    x = _r(M, K, seed=21, dtype=torch.bfloat16)
    w = (_r(N, K, seed=22) * 0.05).to(torch.bfloat16)
    r = _r(M, N, seed=23, dtype=torch.bfloat16) if res else None
    launches = pb.launch_count()
    y = pb.glue_linear(x, w, r)
    torch.cuda.synchronize()
    assert pb.launch_count() - launches == 1
    rng = np.random.default_rng(M + N)
    rows = np.concatenate([[0, M - 1, min(127, M - 1), min(128, M - 1)], rng.integers(0, M, size=60)])
    cols = np.concatenate([[0, N - 1, min(255, N - 1), min(256, N - 1)], rng.integers(0, N, size=60)])
    rt, ct = torch.from_numpy(rows).to(DEV), torch.from_numpy(cols).to(DEV)
    want = (x[rt].double() * w[ct].double()).sum(-1)
    if res:
        want = want + r[rt, ct].double()
    got = y[rt, ct].double()
    scale = float(want.abs().max().clamp_min(1e-3))
    assert float((got - want).abs().max()) <= 2 ** -7 * scale
    # a whole row and a whole column
    np.testing.assert_allclose(synth.widen(y[M // 2]), synth.widen(x[M // 2]) @ synth.widen(w).T + (synth.widen(r[M // 2]) if res else 0),
                               atol=2 ** -7 * scale, rtol=2 ** -7)


@pytest.mark.parametrize("M,N,K,res", [(64, 4096, 11008, True), (37, 11008, 4096, False), (17, 128, 64, False),
                                       (64, 64, 512, True), (1, 4096, 4096, True), (65, 4096, 4096, True)])
def test_skinny_linear_whole_output(M, N, K, res):
    """At most 64 rows: the weight-streaming kernel (K slices summed across a cluster in slice order).
    The whole output against fp64, and bit-identical on a second run; 65 rows take the tcgen05 path."""
    x = _r(M, K, seed=31, dtype=torch.bfloat16)
    w = (_r(N, K, seed=32) * 0.05).to(torch.bfloat16)
    r = _r(M, N, seed=33, dtype=torch.bfloat16) if res else None
    y = pb.glue_linear(x, w, r)
    y2 = pb.glue_linear(x, w, r)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)
    want = x.double() @ w.double().T
    if res:
        want = want + r.double()
    scale = float(want.abs().max().clamp_min(1e-3))
    assert float((y.double() - want).abs().max()) <= 2 ** -7 * scale


@pytest.mark.parametrize("M,N,K", [(300, 512, 256), (4096, 11008, 4096), (129, 1000, 64), (65, 128, 128)])
def test_gated_linear_against_fp64(M, N, K):
    """pyr_glue_linear_swiglu: silu(x wg^T) * (x wu^T) from the fp32 accumulators, against fp64 on sampled
    entries and one whole row; fp32 and unaligned shapes are refused."""
    x = _r(M, K, seed=41, dtype=torch.bfloat16)
    wg = (_r(N, K, seed=42) * 0.05).to(torch.bfloat16)
    wu = (_r(N, K, seed=43) * 0.05).to(torch.bfloat16)
    launches = pb.launch_count()
    out = pb.glue_linear_swiglu(x, wg, wu)
    torch.cuda.synchronize()
    assert pb.launch_count() - launches == 1
    rng = np.random.default_rng(M + N)
    rows = np.concatenate([[0, M - 1, min(127, M - 1), min(128, M - 1)], rng.integers(0, M, size=60)])
    cols = np.concatenate([[0, N - 1, min(127, N - 1), min(128, N - 1)], rng.integers(0, N, size=60)])
    rt, ct = torch.from_numpy(rows).to(DEV), torch.from_numpy(cols).to(DEV)
    g = (x[rt].double() * wg[ct].double()).sum(-1)
    u = (x[rt].double() * wu[ct].double()).sum(-1)
    want = g / (1 + torch.exp(-g)) * u
    got = out[rt, ct].double()
    scale = float(want.abs().max().clamp_min(1e-3))
    assert float((got - want).abs().max()) <= 2 ** -7 * scale
    gr = synth.widen(x[M // 2]) @ synth.widen(wg).T
    ur = synth.widen(x[M // 2]) @ synth.widen(wu).T
    np.testing.assert_allclose(synth.widen(out[M // 2]), gr / (1 + np.exp(-gr)) * ur, atol=2 ** -7 * scale, rtol=2 ** -7)
    with pytest.raises(Exception):
        pb.glue_linear_swiglu(x.float(), wg.float(), wu.float())


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-5), (torch.bfloat16, 2 ** -7)])
def test_row_mapped_norm_and_residual(dtype, tol):
    """pyr_glue_rmsnorm_rows / pyr_glue_linear_rows read kept rows where they lie: equal to gathering first."""
    B, n_src, n_dst, d, N = 3, 300, 170, 256, 384
    g = torch.Generator().manual_seed(5)
    rows = torch.stack([torch.sort(torch.randperm(n_src, generator=g)[:n_dst]).values for _ in range(B)]).to(torch.int32)
    pad = torch.full((B, 7), -1, dtype=torch.int32)                       # a list stride wider than n_dst
    rows_dev = torch.cat([rows, pad], 1).to(DEV)[:, :n_dst]
    x = _r(B, n_src, d, seed=51, dtype=dtype)
    gain = _r(d, seed=52, dtype=dtype)
    gathered = torch.gather(x, 1, rows.to(DEV).long()[:, :, None].expand(B, n_dst, d)).contiguous()
    got = pb.glue_rmsnorm_rows(x, rows_dev, gain)
    assert torch.equal(got, pb.glue_rmsnorm(gathered, gain))
    h = _r(B, n_dst, d, seed=53, dtype=dtype)
    w = (_r(N, d, seed=54) * 0.05).to(dtype)
    res = _r(B, n_src, N, seed=55, dtype=dtype)
    res_g = torch.gather(res, 1, rows.to(DEV).long()[:, :, None].expand(B, n_dst, N)).contiguous()
    y = pb.glue_linear_rows(h, w, res, rows_dev)
    assert torch.equal(y, pb.glue_linear(h, w, res_g))
    want = synth.widen(h) @ synth.widen(w).T + synth.widen(res_g)
    np.testing.assert_allclose(synth.widen(y), want, atol=tol * float(np.abs(want).max()), rtol=tol)
    # a bigger bf16 case that takes the tensor-core kernel
    if dtype == torch.bfloat16:
        B2, s2, d2, k2 = 2, 900, 700, 512
        rows2 = torch.stack([torch.sort(torch.randperm(s2, generator=g)[:d2]).values for _ in range(B2)]).to(torch.int32).to(DEV)
        h2 = _r(B2, d2, k2, seed=56, dtype=dtype)
        w2 = (_r(1024, k2, seed=57) * 0.05).to(dtype)
        r2 = _r(B2, s2, 1024, seed=58, dtype=dtype)
        r2g = torch.gather(r2, 1, rows2.long()[:, :, None].expand(B2, d2, 1024)).contiguous()
        assert torch.equal(pb.glue_linear_rows(h2, w2, r2, rows2), pb.glue_linear(h2, w2, r2g))


@pytest.mark.parametrize("M,parts,part_n,K", [(64, 3, 4096, 4096), (9, 2, 11008, 4096), (64, 4, 128, 192), (200, 3, 256, 128),
                                              (7, 2, 100, 64)])
def test_split_linear_equals_separate_products(M, parts, part_n, K):
    """pyr_glue_linear_split: stacked projections through one weight-streaming launch (few rows, parts of whole
    128s) or one product per part otherwise; either way each part equals x . w_part^T to bf16 rounding."""
    x = _r(M, K, seed=61, dtype=torch.bfloat16)
    w = (_r(parts * part_n, K, seed=62) * 0.05).to(torch.bfloat16)
    launches = pb.launch_count()
    ys = pb.glue_linear_split(x, w, parts)
    torch.cuda.synchronize()
    one_launch = M <= 64 and part_n % 128 == 0 and K % 64 == 0
    assert pb.launch_count() - launches == (1 if one_launch else parts)
    for i, y in enumerate(ys):
        want = x.double() @ w[i * part_n:(i + 1) * part_n].double().T
        scale = float(want.abs().max().clamp_min(1e-3))
        assert y.shape == (M, part_n)
        assert float((y.double() - want).abs().max()) <= 2 ** -7 * scale


def test_glue_status_word_is_clean_after_the_linear_layers():
    """pyr_glue_status: no bounded wait of a tensor-core linear layer ran out in this process; reading twice is fine."""
    x = _r(300, 256, seed=71, dtype=torch.bfloat16)
    w = (_r(512, 256, seed=72) * 0.05).to(torch.bfloat16)
    pb.glue_linear(x, w)
    pb.glue_linear(x[:8].contiguous(), w)
    assert pb.glue_status() == 0
    assert pb.glue_status() == 0
