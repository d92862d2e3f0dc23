"""Pins of the decoder glue in the oracle (the tiny Llama-style workload)."""
import numpy as np
import pytest

import oracle
from oracle import tiny_llama as tl
from paper_2405_12532_b200 import synth

rng = np.random.default_rng(11)


def test_rope_depends_on_relative_position_and_keeps_norms():
    D = 16
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))
    def dot(m, n):
        return float((tl.rope(q, [m])[0, 0] * tl.rope(k, [n])[0, 0]).sum())
    assert abs(dot(7, 3) - dot(104, 100)) < 1e-12
    assert abs(dot(7, 3) - dot(3, 7)) > 1e-3                  # it is the signed difference that matters
    assert abs(dot(5, 5) - float((q * k).sum())) < 1e-12      # no rotation at equal positions
    x = rng.standard_normal((3, 2, D))
    np.testing.assert_allclose(np.linalg.norm(tl.rope(x, [0, 9, 250]), axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)
    # position 1, pair (0, D/2) turns by theta_0 = 1 radian
    e = np.zeros((1, 1, D)); e[0, 0, 0] = 1.0
    r = tl.rope(e, [1])[0, 0]
    assert abs(r[0] - np.cos(1.0)) < 1e-15 and abs(r[D // 2] - np.sin(1.0)) < 1e-15
    # pair (1, D/2 + 1) turns by 10000^(-2/D)
    e = np.zeros((1, 1, D)); e[0, 0, 1] = 1.0
    r = tl.rope(e, [1])[0, 0]
    assert abs(r[1] - np.cos(10000.0 ** (-2.0 / D))) < 1e-15


def test_rmsnorm_and_swiglu_on_hand_values():
    x = np.array([3.0, 4.0])                                  # mean square 12.5
    np.testing.assert_allclose(tl.rmsnorm(x, [1.0, 2.0], eps=0.0), [3 / np.sqrt(12.5), 8 / np.sqrt(12.5)], rtol=1e-15)
    assert abs(tl.rmsnorm(np.array([1.0, 1.0]), [1.0, 1.0])[0] - 1 / np.sqrt(1 + 1e-5)) < 1e-15
    Wg, Wu, Wd = np.array([[2.0]]), np.array([[3.0]]), np.array([[0.5]])
    got = tl.swiglu_mlp(np.array([[1.0]]), Wg, Wu, Wd)[0, 0]
    assert abs(got - (2.0 / (1 + np.exp(-2.0))) * 3.0 * 0.5) < 1e-15


@pytest.fixture(scope="module")
def small_model():
    W = {k: v.numpy() for k, v in synth.tiny_llama_weights(hidden=32, n_layers=2, inter=48, vocab=50, seed=3, std=0.3).items()}
    ids = rng.integers(0, 50, size=(2, 24))
    return W, ids


def test_ratio_one_equals_a_plain_full_cache_forward(small_model):
    W, ids = small_model
    pyr = tl.pyramid_generate(W, ids, n_heads=4, recent_len=6, ratio=[1.0, 1.0], steps=5)
    ref = tl.plain_generate(W, ids, n_heads=4, steps=5)
    np.testing.assert_allclose(pyr["logits"], ref["logits"], rtol=1e-9, atol=1e-12)
    np.testing.assert_array_equal(pyr["tokens"], ref["tokens"])
    assert pyr["cache_len"] == [24 + 5, 24 + 5]


def test_pyramid_drops_rows_and_keeps_positions(small_model):
    W, ids = small_model
    out = tl.pyramid_generate(W, ids, n_heads=4, recent_len=6, ratio=[1.0, 0.5], steps=3)
    assert out["kept"][0].shape == (2, 24) and out["kept"][1].shape == (2, 9 + 6)
    assert out["cache_len"] == [24 + 3, 15 + 3]
    full = tl.pyramid_generate(W, ids, n_heads=4, recent_len=6, ratio=[1.0, 1.0], steps=3)
    # the second layer's cut changes nothing before it: first-layer scores are the same
    np.testing.assert_allclose(out["scores"][0], full["scores"][0], rtol=1e-12)
    assert np.abs(out["logits"] - full["logits"]).max() > 1e-6        # but the compression is felt
    # a kept-set override is honoured (per-call comparison hook)
    forced = [None, np.stack([np.concatenate([np.arange(9), np.arange(18, 24)])] * 2)]
    o2 = tl.pyramid_generate(W, ids, n_heads=4, recent_len=6, ratio=[1.0, 0.5], steps=0, kept_override=forced)
    np.testing.assert_array_equal(o2["kept"][1], forced[1])
