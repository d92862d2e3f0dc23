"""Host side of the C ABI, no GPU: the library loads, exports what the header
declares, validates arguments, orders calls, and turns the ratio schedule into
the same integer budgets as the oracle."""
import ctypes as C
import os
import re

import pytest

import oracle
from paper_2405_12532_b200 import binding as pb
from paper_2405_12532_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE_DEV = 0x7F0000000000          # never dereferenced on the host


def _cfg(**over):
    kw = dict(n_layers=4, n_q_heads=8, n_kv_heads=4, head_dim=128, sel_groups=4, dtype="bf16", batch=2,
              prompt_len=512, recent_len=64, max_new_tokens=8, ratio=[1.0, 0.8, 0.5, 0.5])
    kw.update(over)
    return pb.make_config(**kw)


def _alloc(**over):
    cfg, keep = _cfg(**over)
    nbytes, align = pb.pyr_cache_bytes(cfg)
    h = C.c_void_p()
    st = pb.lib().pyr_cache_alloc(C.byref(cfg), C.c_void_p(FAKE_DEV), nbytes, C.byref(h))
    assert st == pb.PYR_OK
    return h, cfg, keep, nbytes


def test_library_exports_every_declared_symbol():
    with open(os.path.join(ROOT, "include", "pyr.h")) as f:
        text = f.read()
    declared = set(re.findall(r"\b(pyr_[a-z_]+)\s*\(", text))
    assert declared == set(pb.EXPORTS)
    L = pb.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert L.pyr_version() >= 100
    assert pb.status_string(pb.PYR_ERR_ORDER) == "call out of sequence"


@pytest.mark.parametrize("over,want", [
    (dict(n_q_heads=6, n_kv_heads=4), pb.PYR_ERR_INVALID),
    (dict(sel_groups=2), pb.PYR_ERR_INVALID),
    (dict(head_dim=96), pb.PYR_ERR_UNSUPPORTED),
    (dict(dtype=7), pb.PYR_ERR_UNSUPPORTED),
    (dict(ratio=[1.0, 0.8, 0.9, 0.5]), pb.PYR_ERR_INVALID),      # increasing
    (dict(ratio=[1.2, 0.8, 0.5, 0.5]), pb.PYR_ERR_INVALID),
    (dict(ratio=[1.0, 0.8, 0.5, -0.1]), pb.PYR_ERR_INVALID),
    (dict(recent_len=0), pb.PYR_ERR_INVALID),
    (dict(batch=0), pb.PYR_ERR_INVALID),
    (dict(prompt_len=1 << 20), pb.PYR_ERR_UNSUPPORTED),
    (dict(recent_w=[-1.0] * 64), pb.PYR_ERR_INVALID),
    (dict(softmax_scale=-1.0), pb.PYR_ERR_INVALID),
    (dict(min_len=[0, 0, -3, 0]), pb.PYR_ERR_INVALID),
    (dict(ratio=None), pb.PYR_ERR_NULL),
])
def test_config_validation(over, want):
    cfg, keep = _cfg(**over)
    b = C.c_size_t(0)
    assert pb.lib().pyr_cache_bytes(C.byref(cfg), C.byref(b), None) == want


def test_null_and_small_buffer():
    L = pb.lib()
    cfg, keep = _cfg()
    b = C.c_size_t(0)
    assert L.pyr_cache_bytes(None, C.byref(b), None) == pb.PYR_ERR_NULL
    assert L.pyr_cache_bytes(C.byref(cfg), None, None) == pb.PYR_ERR_NULL
    nbytes, align = pb.pyr_cache_bytes(cfg)
    assert align == 256
    h = C.c_void_p()
    assert L.pyr_cache_alloc(C.byref(cfg), None, nbytes, C.byref(h)) == pb.PYR_ERR_NULL
    assert L.pyr_cache_alloc(C.byref(cfg), C.c_void_p(FAKE_DEV), nbytes - 1, C.byref(h)) == pb.PYR_ERR_BUFFER_TOO_SMALL
    assert L.pyr_cache_alloc(C.byref(cfg), C.c_void_p(FAKE_DEV + 8), nbytes, C.byref(h)) == pb.PYR_ERR_INVALID
    assert L.pyr_cache_free(None) == pb.PYR_ERR_NULL


def _info(h, layer):
    v = [C.c_int32(0) for _ in range(4)]
    st = pb.lib().pyr_cache_layer_info(h, layer, *[C.byref(x) for x in v])
    return st, [x.value for x in v]


@pytest.mark.parametrize("name", list(synth.CONFIGS))
def test_budgets_equal_oracle_on_all_workloads(name):
    w = synth.CONFIGS[name]
    ratio = synth.ratio_schedule(w)
    h, cfg, keep, nbytes = _alloc(**pb.config_from_workload(w, ratio))
    want = oracle.layer_budgets(w["prompt_len"], w["recent_len"], ratio)
    for l, b in enumerate(want):
        st, (n_in, k, len_now, cap) = _info(h, l)
        assert st == pb.PYR_OK
        assert (n_in, k, len_now, cap) == (b["n_in"], b["k"], 0, b["n_out"] + w["max_new_tokens"])
    eb = 2 if w["dtype"] == "bf16" else 4
    kv = oracle.cache_bytes(w["batch"], w["n_kv_heads"], w["head_dim"], eb, w["prompt_len"], w["recent_len"],
                            ratio, w["max_new_tokens"])
    assert kv <= nbytes <= kv * 1.08 + (64 << 20)
    assert _info(h, w["n_layers"])[0] == pb.PYR_ERR_INVALID
    pb.lib().pyr_cache_free(h)


def test_budget_edges_match_oracle():
    for N, L, ratio, ml in [(20, 32, [0.5, 0.1], None), (100, 10, [0.0], None),
                            (100, 10, [0.1, 0.1], [50, 60]), (100, 10, [0.9, 0.5], None),
                            (4097, 1, [1.0, 0.33333, 0.001], None)]:
        h, cfg, keep, _ = _alloc(n_layers=len(ratio), prompt_len=N, recent_len=L, ratio=ratio, min_len=ml)
        for l, b in enumerate(oracle.layer_budgets(N, L, ratio, ml)):
            st, (n_in, k, _, cap) = _info(h, l)
            assert (n_in, k, cap) == (b["n_in"], b["k"], b["n_out"] + 8)
        pb.lib().pyr_cache_free(h)


def test_call_order_and_pointer_checks_before_any_launch():
    L = pb.lib()
    h, cfg, keep, _ = _alloc()
    p = C.c_void_p(FAKE_DEV)
    st = [64 * 8 * 128, 8 * 128, 128, 64 * 4 * 128, 4 * 128, 128, 64 * 8 * 128, 8 * 128, 128]
    # wrong layer, select before prefill, decode before the prompt is done
    assert L.pyr_prefill_layer(h, 1, p, p, p, p, *st, None) == pb.PYR_ERR_ORDER
    assert L.pyr_select_compact(h, 0, p, p, st[3], st[4], st[5], None, 0, 0, 0, 0, None, None) == pb.PYR_ERR_ORDER
    assert L.pyr_decode_attn(h, 0, p, p, p, p, None) == pb.PYR_ERR_ORDER
    assert L.pyr_prefill_layer(h, 0, None, p, p, p, *st, None) == pb.PYR_ERR_NULL
    assert L.pyr_prefill_layer(h, 9, p, p, p, p, *st, None) == pb.PYR_ERR_INVALID
    bad = list(st); bad[2] = 64                      # head stride smaller than D
    assert L.pyr_prefill_layer(h, 0, p, p, p, p, *bad, None) == pb.PYR_ERR_INVALID
    bad = list(st); bad[1] = 8 * 128 + 3             # bf16 rows must stay 16-byte aligned
    assert L.pyr_prefill_layer(h, 0, p, p, p, p, *bad, None) == pb.PYR_ERR_INVALID
    ip, pp = C.c_void_p(), C.c_void_p()
    assert L.pyr_cache_kept(h, 0, C.byref(ip), C.byref(pp)) == pb.PYR_ERR_ORDER
    assert L.pyr_cache_scores(h, 0, C.byref(ip)) == pb.PYR_ERR_ORDER
    L.pyr_cache_free(h)


def test_shard_batch_covers_batch():
    for B, W in [(64, 8), (10, 4), (3, 4)]:
        spans = [synth.shard_batch(B, W, r) for r in range(W)]
        assert spans[0][0] == 0 and spans[-1][1] == B
        assert all(spans[i][1] == spans[i + 1][0] for i in range(W - 1))


def test_recent_len_from_ratio_matches_the_oracle():
    for N in (1, 7, 512, 2048, 8191):
        for r in (0.0, 0.001, 0.3, 0.4, 0.5, 0.9999, 1.0, 1.7):
            assert pb.recent_len_from_ratio(N, r) == oracle.recent_len_from_ratio(N, r)
    assert pb.recent_len_from_ratio(2048, 0.4) == 819 and pb.recent_len_from_ratio(10, 0.0) == 1
    assert pb.recent_len_from_ratio(0, 0.4) == 0 and pb.recent_len_from_ratio(100, -0.1) == 0


def _cache_gb(w, ratio, batch, flags=0):
    cfg, keep = pb.make_config(**pb.config_from_workload(dict(w, batch=batch), ratio, flags=flags))
    return pb.pyr_cache_bytes(cfg)[0] / 1e9


def test_max_batch_under_a_memory_cap_table2_shape():
    """Table 2's setting as byte accounting: the largest batch whose cache buffer fits beside the
    13B model's 26 GB of 2-byte weights on an 80 GB device, with every layer keeping everything and
    with the pyramid schedule (no GPU: pyr_cache_bytes is host arithmetic). The paper reports batch
    42 for the full cache and 88 for PyramidInfer, a factor 2.1; its schedule is not in its text, so
    only the direction and rough size of the gain are checked."""
    w = synth.CONFIGS["13b_table_32x512"]
    budget_gb = 80.0 - 26.0

    def max_batch(ratio, generated_rows):
        lo, hi = 1, 4096
        while lo < hi:
            mid = (lo + hi + 1) // 2
            if _cache_gb(dict(w, max_new_tokens=generated_rows), ratio, mid) <= budget_gb:
                lo = mid
            else:
                hi = mid - 1
        return lo

    full = max_batch([1.0] * w["n_layers"], 256)
    # with the generation-phase update every 16 steps a layer never holds more than its budget + window + 16 rows
    pyr = max_batch(synth.ratio_schedule(w), 16)
    assert 60 <= full <= 90             # 2 * 40 layers * 5120 * 2 B * 768 rows = 0.63 GB per sequence
    assert pyr / full > 1.8


def test_glue_entry_points_validate_before_any_launch():
    """The decoder-glue calls refuse bad arguments on the host: null pointers, unknown dtypes, sizes out
    of range, and the shapes the fused forms do not cover - none of which reaches a kernel launch."""
    L = pb.lib()
    P = C.c_void_p(FAKE_DEV)
    NULL = C.c_void_p(None)
    i64, i32, f32 = C.c_int64, C.c_int32, C.c_float
    L.pyr_glue_linear.restype = L.pyr_glue_rope.restype = L.pyr_glue_linear_swiglu.restype = C.c_int
    L.pyr_glue_rmsnorm_rows.restype = L.pyr_glue_linear_rows.restype = C.c_int
    assert L.pyr_glue_linear(NULL, P, NULL, P, i64(4), i32(8), i32(8), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_NULL
    assert L.pyr_glue_linear(P, P, NULL, P, i64(4), i32(0), i32(8), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_INVALID
    assert L.pyr_glue_linear(P, P, NULL, P, i64(4), i32(8), i32(8), i32(9), NULL) == pb.PYR_ERR_UNSUPPORTED
    assert L.pyr_glue_linear(P, P, NULL, P, i64(0), i32(8), i32(8), i32(pb.PYR_BF16), NULL) == pb.PYR_OK      # nothing to do
    # the gated form: bf16, k a multiple of 64, n a multiple of 8
    assert L.pyr_glue_linear_swiglu(P, P, NULL, P, i64(4), i32(8), i32(64), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_NULL
    assert L.pyr_glue_linear_swiglu(P, P, P, P, i64(4), i32(8), i32(64), i32(pb.PYR_F32), NULL) == pb.PYR_ERR_UNSUPPORTED
    assert L.pyr_glue_linear_swiglu(P, P, P, P, i64(4), i32(8), i32(48), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_UNSUPPORTED
    assert L.pyr_glue_linear_swiglu(P, P, P, P, i64(-1), i32(8), i32(64), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_INVALID
    # rotary embedding: even head_dim up to 256
    assert L.pyr_glue_rope(P, P, i64(4), i32(2), i32(7), i32(pb.PYR_F32), NULL) == pb.PYR_ERR_INVALID
    assert L.pyr_glue_rope(P, P, i64(4), i32(2), i32(512), i32(pb.PYR_F32), NULL) == pb.PYR_ERR_UNSUPPORTED
    # row lists: a list stride shorter than the list, empty sources
    assert L.pyr_glue_rmsnorm_rows(P, P, i64(3), P, P, i32(2), i32(10), i32(4), i32(16), f32(1e-5), i32(pb.PYR_F32), NULL) == pb.PYR_ERR_INVALID
    assert L.pyr_glue_rmsnorm_rows(P, NULL, i64(4), P, P, i32(2), i32(10), i32(4), i32(16), f32(1e-5), i32(pb.PYR_F32), NULL) == pb.PYR_ERR_NULL
    assert L.pyr_glue_linear_rows(P, P, P, P, i64(4), P, i32(2), i32(0), i32(4), i32(16), i32(16), i32(pb.PYR_F32), NULL) == pb.PYR_ERR_INVALID
    assert L.pyr_glue_linear_rows(P, P, NULL, P, i64(4), P, i32(2), i32(10), i32(4), i32(16), i32(16), i32(pb.PYR_F32), NULL) == pb.PYR_ERR_NULL
    assert L.pyr_glue_linear_rows(P, P, P, P, i64(4), P, i32(0), i32(10), i32(4), i32(16), i32(16), i32(pb.PYR_F32), NULL) == pb.PYR_OK
    # stacked projections: one to four parts, every part's pointer given
    L.pyr_glue_linear_split.restype = L.pyr_glue_status.restype = C.c_int
    two = (C.c_void_p * 2)(FAKE_DEV, FAKE_DEV)
    hole = (C.c_void_p * 2)(FAKE_DEV, None)
    assert L.pyr_glue_linear_split(P, P, None, i32(2), i64(4), i32(128), i32(64), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_NULL
    assert L.pyr_glue_linear_split(P, P, hole, i32(2), i64(4), i32(128), i32(64), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_NULL
    assert L.pyr_glue_linear_split(P, P, two, i32(5), i64(4), i32(128), i32(64), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_INVALID
    assert L.pyr_glue_linear_split(P, P, two, i32(2), i64(4), i32(0), i32(64), i32(pb.PYR_BF16), NULL) == pb.PYR_ERR_INVALID
    assert L.pyr_glue_linear_split(P, P, two, i32(2), i64(0), i32(128), i32(64), i32(pb.PYR_BF16), NULL) == pb.PYR_OK
    assert L.pyr_glue_status(NULL, None) == pb.PYR_ERR_NULL


def test_select_first_flag_adds_the_inverse_list_to_the_plan():
    """PYR_FLAG_SELECT_FIRST carves one more [B, G, N] int32 array (the inverse of the kept list), nothing else."""
    base_cfg, keep0 = _cfg()
    flag_cfg, keep1 = _cfg(flags=pb.PYR_FLAG_SELECT_FIRST)
    b0, _ = pb.pyr_cache_bytes(base_cfg)
    b1, _ = pb.pyr_cache_bytes(flag_cfg)
    want = 2 * 4 * 512 * 4                     # B * G * N * 4 bytes
    assert b1 - b0 == (want + 255) // 256 * 256


def test_header_is_plain_c(tmp_path):
    """include/pyr.h is the boundary: it must compile as C99 on its own (no C++ or CUDA types in the signatures)."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    src = tmp_path / "use_header.c"
    src.write_text('#include "pyr.h"\nint main(void) { pyr_config_t c; (void)c; return (int)PYR_OK; }\n')
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                    "-I", os.path.join(ROOT, "include"), str(src)], check=True)
