"""The tiny Llama-style workload as a whole model: 2 layers, hidden 256, 4 heads x 64, fp32, batch 2,
prompt 256, window 32, ratios [1.0, 0.5], 16 greedy decode steps. Attention + score, selection,
compaction of the hidden rows and decode over the compressed caches run in the CUDA library, and so
does the decoder glue around them (embedding, RMSNorm, projections, rotary embedding, MLP, output head,
greedy argmax: the pyr_glue_* kernels); torch only holds the tensors and slices them. Compared with the fp64 oracle chained through the
same kept sets and tokens (per-call comparison on identical inputs), and with the oracle's own
free-running generation."""
import numpy as np
import pytest
import torch

import oracle
from oracle import tiny_llama as tl
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth
from parity_util import check_kept

pytestmark = pytest.mark.gpu
DEV = "cuda"
H, D, HID, L, N, B, STEPS = 4, 64, 256, 32, 256, 2, 16


def _rms(x, g, eps=1e-5):
    return pb.glue_rmsnorm(x.contiguous(), g, eps)


def _rope(x, pos):
    """x [B, n, H, D], pos [B, n] ints -> rotated copy (pyr_glue_rope at the tokens' positions)."""
    return pb.glue_rope_(x.contiguous().clone(), pos.to(torch.int32).contiguous())


def _lin(x, W, res=None):
    return pb.glue_linear(x.contiguous(), W, None if res is None else res.contiguous())


def _mlp(x, Wg, Wu, Wd, res):
    return _lin(pb.glue_swiglu(_lin(x, Wg), _lin(x, Wu)), Wd, res)


def _gpu_generate(W, ids, ratio, steps):
    nL = len(ratio)
    W = {k: (v.t().contiguous() if v.dim() == 2 and k != "emb" else v) for k, v in W.items()}   # linear weights as [out, in]
    w = dict(n_layers=nL, n_q_heads=H, n_kv_heads=H, head_dim=D, sel_groups=1, dtype="f32", batch=B,
             prompt_len=N, recent_len=L, max_new_tokens=steps)
    cache = pb.PyrCache(device=DEV, **pb.config_from_workload(w, ratio))
    x = pb.glue_embed(ids.to(torch.int32).contiguous(), W["emb"])
    pos = torch.arange(N, device=DEV).expand(B, N).contiguous()
    kepts, scores = [], []
    for l in range(nL):
        n = x.shape[1]
        assert n == cache.layer_info(l)["n_in"]
        h = _rms(x, W[f"n1{l}"])
        q = _rope(_lin(h, W[f"wq{l}"]).view(B, n, H, D), pos)
        k = _rope(_lin(h, W[f"wk{l}"]).view(B, n, H, D), pos)
        v = _lin(h, W[f"wv{l}"]).view(B, n, H, D)
        o = torch.empty_like(q)
        cache.prefill_layer(l, q, k, v, o)
        scores.append(cache.scores(l).clone())
        # the residual stream and the attention output of a token travel together: one row of 2 * hidden
        rows = torch.cat([x, o.view(B, n, HID)], -1).contiguous()
        n_out = cache.select_compact(l, k, v, rows, 2 * HID, n * 2 * HID, 2 * HID, 0)
        kept, posk = cache.kept(l)
        kepts.append(kept[:, 0].clone())
        y = _lin(rows[:, :n_out, HID:], W[f"wo{l}"], rows[:, :n_out, :HID])
        x = _mlp(_rms(y, W[f"n2{l}"]), W[f"wg{l}"], W[f"wu{l}"], W[f"wd{l}"], y)
        pos = posk[:, 0].clone().long()
    logits = [_lin(_rms(x[:, -1], W["nf"]), W["head"])]
    tokens = []
    for t in range(steps):
        prev = pb.glue_argmax(logits[-1].contiguous())
        tokens.append(prev.long())
        xt = pb.glue_embed(prev, W["emb"])
        p = torch.full((B, 1), N + t, device=DEV)
        for l in range(nL):
            h = _rms(xt, W[f"n1{l}"])
            q = _rope(_lin(h, W[f"wq{l}"]).view(B, 1, H, D), p)[:, 0].contiguous()
            k = _rope(_lin(h, W[f"wk{l}"]).view(B, 1, H, D), p)[:, 0].contiguous()
            v = _lin(h, W[f"wv{l}"]).view(B, H, D)
            o = torch.empty_like(q)
            cache.decode_attn(l, q, k, v, o)
            y = _lin(o.view(B, HID), W[f"wo{l}"], xt)
            xt = _mlp(_rms(y, W[f"n2{l}"]), W[f"wg{l}"], W[f"wu{l}"], W[f"wd{l}"], y)
        logits.append(_lin(_rms(xt, W["nf"]), W["head"]))
    torch.cuda.synchronize()
    assert cache.status() == 0
    lens = [cache.layer_info(l)["len_now"] for l in range(nL)]
    cache.close()
    return torch.stack(logits, 1), (torch.stack(tokens, 1) if tokens else None), kepts, scores, lens


@pytest.mark.parametrize("ratio", [[1.0, 0.5], [1.0, 1.0]], ids=["pyramid", "ratio1"])
def test_tiny_llama_against_oracle(ratio):
    Wt = synth.tiny_llama_weights(hidden=HID, n_layers=2, inter=768, vocab=1000, seed=1)
    ids = synth.uniform_token_ids(B, N, 1000, seed=0)
    Wg = {k: v.to(DEV) for k, v in Wt.items()}
    logits, tokens, kepts, scores, lens = _gpu_generate(Wg, ids.to(DEV), ratio, STEPS)
    Wn = {k: v.numpy() for k, v in Wt.items()}
    budgets = oracle.layer_budgets(N, L, ratio)
    assert lens == [b["n_out"] + STEPS for b in budgets]           # 256 + 16 and 144 + 16 for the pyramid
    # per call: the oracle driven through the GPU's kept sets and tokens
    forced = tl.pyramid_generate(Wn, ids.numpy(), H, L, ratio, STEPS, kept_override=[k.cpu().numpy() for k in kepts],
                                 tokens_override=tokens.cpu().numpy())
    for l, bud in enumerate(budgets):
        np.testing.assert_allclose(synth.widen(scores[l][:, 0]), forced["scores"][l], rtol=2e-4, atol=1e-30)
        for b in range(B):
            check_kept(kepts[l][b].cpu().numpy(), forced["scores"][l][b], bud["k"], bud["n_in"], L)
    scale = float(np.abs(forced["logits"]).max())
    tol = 1e-4 * scale
    err = float(np.abs(synth.widen(logits) - forced["logits"]).max())
    assert err <= tol, (err, tol)
    # greedy tokens: equal to the oracle's argmax unless its two best logits are closer than the tolerance
    got_tok = np.concatenate([tokens.cpu().numpy(), logits[:, -1].argmax(-1).cpu().numpy()[:, None]], 1)
    for b in range(B):
        for t in range(STEPS + 1):
            if got_tok[b, t] != forced["tokens"][b, t]:
                top2 = np.sort(forced["logits"][b, t])[-2:]
                assert top2[1] - top2[0] <= tol
    # the oracle left to itself makes the same choices (no tie was met on this input)
    free = tl.pyramid_generate(Wn, ids.numpy(), H, L, ratio, STEPS)
    np.testing.assert_array_equal(free["tokens"], got_tok)
    for l in range(len(ratio)):
        np.testing.assert_array_equal(free["kept"][l], kepts[l].cpu().numpy())
    if ratio == [1.0, 1.0]:
        plain = tl.plain_generate(Wn, ids.numpy(), H, STEPS)
        assert np.abs(synth.widen(logits) - plain["logits"]).max() <= tol
