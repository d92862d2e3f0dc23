"""ctypes binding of libpyr.so: the same names as the C ABI (include/pyr.h),
argument marshalling only. torch supplies device memory and streams; every
step of the path runs inside the library's kernels. There is no fallback: if
the library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpyr.so")

PYR_OK, PYR_ERR_INVALID, PYR_ERR_NULL, PYR_ERR_UNSUPPORTED, PYR_ERR_BUFFER_TOO_SMALL, \
    PYR_ERR_CAPACITY, PYR_ERR_ORDER, PYR_ERR_CUDA, PYR_ERR_TIMEOUT = range(9)
PYR_ERR_SCRATCH_LIMIT = 9
PYR_ERR_HOST_MEMORY = 10
PYR_BF16, PYR_F32 = 0, 1
PYR_FLAG_CUDA_CORE_PREFILL = 1
PYR_FLAG_GEN_RESELECT = 2
PYR_FLAG_POS_REENCODE = 4
PYR_FLAG_SELECT_FIRST = 8

EXPORTS = [
    "pyr_cache_layer_info", "pyr_cache_bytes", "pyr_cache_alloc", "pyr_cache_free", "pyr_cache_reset",
    "pyr_cache_kept", "pyr_cache_scores", "pyr_cache_lse", "pyr_cache_kv", "pyr_cache_status",
    "pyr_prefill_layer", "pyr_select_compact", "pyr_decode_attn", "pyr_decode_reselect", "pyr_cache_arm_wait_test", "pyr_recent_len_from_ratio", "pyr_glue_embed", "pyr_glue_rmsnorm", "pyr_glue_status", "pyr_glue_linear", "pyr_glue_linear_split", "pyr_glue_linear_swiglu", "pyr_glue_rmsnorm_rows", "pyr_glue_linear_rows",
    "pyr_glue_rope", "pyr_glue_swiglu", "pyr_glue_argmax", "pyr_status_string", "pyr_version", "pyr_launch_count",
    "pyr_decode_attn_noalloc", "pyr_decode_attn_noalloc_status",
]


class PyrConfig(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("sel_groups", C.c_int32), ("dtype", C.c_int32),
        ("batch", C.c_int32), ("prompt_len", C.c_int32), ("recent_len", C.c_int32),
        ("max_new_tokens", C.c_int32),
        ("ratio", C.POINTER(C.c_double)), ("min_len", C.POINTER(C.c_int32)),
        ("recent_w", C.POINTER(C.c_float)), ("softmax_scale", C.c_float), ("flags", C.c_uint32),
    ]


class PyrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> C.CDLL:
    """The loaded library. Raises if libpyr.so is missing (build it with
    `python -m paper_2405_12532_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: the CUDA library is not built and there is no "
                               "other implementation to fall back to")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        pi32 = C.POINTER(C.c_int32)
        L.pyr_status_string.restype = C.c_char_p
        L.pyr_status_string.argtypes = [C.c_int]
        L.pyr_version.restype = i32
        L.pyr_launch_count.restype = C.c_uint64
        L.pyr_launch_count.argtypes = []
        L.pyr_cache_bytes.argtypes = [C.POINTER(PyrConfig), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        L.pyr_cache_alloc.argtypes = [C.POINTER(PyrConfig), vp, C.c_size_t, C.POINTER(vp)]
        L.pyr_cache_free.argtypes = [vp]
        L.pyr_cache_reset.argtypes = [vp, vp]
        L.pyr_cache_layer_info.argtypes = [vp, i32, pi32, pi32, pi32, pi32]
        L.pyr_cache_kept.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp)]
        L.pyr_cache_scores.argtypes = [vp, i32, C.POINTER(vp)]
        L.pyr_cache_lse.argtypes = [vp, i32, C.POINTER(vp)]
        L.pyr_cache_kv.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp)]
        L.pyr_cache_status.argtypes = [vp, vp, pi32]
        L.pyr_prefill_layer.argtypes = [vp, i32, vp, vp, vp, vp] + [i64] * 9 + [vp]
        L.pyr_select_compact.argtypes = [vp, i32, vp, vp, i64, i64, i64, vp, i64, i64, i64, i64, pi32, vp]
        L.pyr_decode_attn.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        L.pyr_decode_reselect.argtypes = [vp, i32, pi32, pi32, vp]
        L.pyr_cache_arm_wait_test.argtypes = [vp]
        L.pyr_glue_embed.argtypes = [vp, vp, vp, i64, i32, i32, i32, vp, vp]
        L.pyr_glue_rmsnorm.argtypes = [vp, vp, vp, i64, i32, C.c_float, i32, vp]
        L.pyr_glue_linear.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, vp]
        L.pyr_glue_linear_swiglu.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, vp]
        L.pyr_glue_linear_split.argtypes = [vp, vp, vp, i32, i64, i32, i32, i32, vp]
        L.pyr_glue_rmsnorm_rows.argtypes = [vp, vp, i64, vp, vp, i32, i32, i32, i32, C.c_float, i32, vp]
        L.pyr_glue_linear_rows.argtypes = [vp, vp, vp, vp, i64, vp, i32, i32, i32, i32, i32, i32, vp]
        L.pyr_glue_rope.argtypes = [vp, vp, i64, i32, i32, i32, vp]
        L.pyr_glue_swiglu.argtypes = [vp, vp, vp, i64, i32, vp]
        L.pyr_glue_argmax.argtypes = [vp, vp, i64, i32, i32, vp]
        L.pyr_recent_len_from_ratio.argtypes = [i32, C.c_double]
        L.pyr_recent_len_from_ratio.restype = i32
        L.pyr_decode_attn_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                              C.c_float, vp]
        L.pyr_decode_attn_noalloc_status.argtypes = [vp, pi32]
        for name in EXPORTS:
            fn = getattr(L, name)
            if name not in ("pyr_status_string", "pyr_version", "pyr_launch_count", "pyr_recent_len_from_ratio"):
                fn.restype = C.c_int
        _lib = L
    return _lib


def launch_count() -> int:
    return int(lib().pyr_launch_count())


def status_string(status: int) -> str:
    return lib().pyr_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != PYR_OK:
        raise PyrError(status, where)


def make_config(*, n_layers, n_q_heads, n_kv_heads, head_dim, sel_groups, dtype, batch, prompt_len,
                recent_len, max_new_tokens, ratio, min_len=None, recent_w=None, softmax_scale=0.0,
                flags=0):
    """Returns (PyrConfig, keepalive): the ctypes arrays the struct points to."""
    cfg = PyrConfig()
    cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
    cfg.sel_groups = sel_groups
    cfg.dtype = {"bf16": PYR_BF16, "f32": PYR_F32, torch.bfloat16: PYR_BF16, torch.float32: PYR_F32}.get(dtype, dtype)
    cfg.batch, cfg.prompt_len, cfg.recent_len, cfg.max_new_tokens = batch, prompt_len, recent_len, max_new_tokens
    keep = []
    if ratio is not None:
        r = (C.c_double * len(ratio))(*[float(x) for x in ratio])
        keep.append(r)
        cfg.ratio = C.cast(r, C.POINTER(C.c_double))
    if min_len is not None:
        ml = (C.c_int32 * len(min_len))(*[int(x) for x in min_len])
        keep.append(ml)
        cfg.min_len = C.cast(ml, C.POINTER(C.c_int32))
    if recent_w is not None:
        w = (C.c_float * len(recent_w))(*[float(x) for x in recent_w])
        keep.append(w)
        cfg.recent_w = C.cast(w, C.POINTER(C.c_float))
    cfg.softmax_scale = float(softmax_scale)
    cfg.flags = int(flags)
    return cfg, keep


def pyr_cache_bytes(cfg: PyrConfig) -> tuple[int, int]:
    b, a = C.c_size_t(0), C.c_size_t(0)
    _check(lib().pyr_cache_bytes(C.byref(cfg), C.byref(b), C.byref(a)), "pyr_cache_bytes")
    return b.value, a.value


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def decode_attn_noalloc(q, k_new, v_new, out, k_cache, v_cache, length: int, softmax_scale: float = 0.0,
                        stream=None) -> int:
    """pyr_decode_attn_noalloc on torch tensors (q [B,Hq,D], k_new/v_new [B,Hkv,D],
    caches [B,Hkv,cap,D], `length` rows filled). Returns the status code; the
    library allocates nothing and the binding only reads pointers and shapes."""
    B, Hq, D = q.shape
    Hkv, cap = k_cache.shape[1], k_cache.shape[2]
    dt = PYR_BF16 if q.dtype == torch.bfloat16 else PYR_F32
    return lib().pyr_decode_attn_noalloc(q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
                                         k_cache.data_ptr(), v_cache.data_ptr(), B, Hq, Hkv, D, dt, int(length),
                                         cap, float(softmax_scale), C.c_void_p(_stream_ptr(stream)))


def _dt(t: torch.Tensor) -> int:
    return PYR_BF16 if t.dtype == torch.bfloat16 else PYR_F32


def glue_embed(ids, table):
    """ids int32 [...], table [V, d] -> [..., d] (pyr_glue_embed)."""
    assert ids.dtype == torch.int32 and ids.is_contiguous() and table.is_contiguous()
    out = torch.empty(*ids.shape, table.shape[1], dtype=table.dtype, device=table.device)
    _check(lib().pyr_glue_embed(ids.data_ptr(), table.data_ptr(), out.data_ptr(), ids.numel(), table.shape[1],
                                table.shape[0], _dt(table), None, C.c_void_p(_stream_ptr(None))), "pyr_glue_embed")
    return out


def glue_rmsnorm(x, gain, eps=1e-5):
    assert x.is_contiguous()
    out = torch.empty_like(x)
    _check(lib().pyr_glue_rmsnorm(x.data_ptr(), gain.data_ptr(), out.data_ptr(), x.numel() // x.shape[-1], x.shape[-1],
                                  float(eps), _dt(x), C.c_void_p(_stream_ptr(None))), "pyr_glue_rmsnorm")
    return out


def glue_linear(x, w, residual=None):
    """x [..., K] . w [N, K] (+ residual [..., N]) -> [..., N] (pyr_glue_linear)."""
    assert x.is_contiguous() and w.is_contiguous() and (residual is None or residual.is_contiguous())
    N, K = w.shape
    y = torch.empty(*x.shape[:-1], N, dtype=x.dtype, device=x.device)
    _check(lib().pyr_glue_linear(x.data_ptr(), w.data_ptr(), residual.data_ptr() if residual is not None else None,
                                 y.data_ptr(), x.numel() // K, N, K, _dt(x), C.c_void_p(_stream_ptr(None))), "pyr_glue_linear")
    return y


def glue_rmsnorm_rows(x, rows, gain, eps: float = 1e-5):
    """rmsnorm of the rows rows[b, i] of x [B, n_src, d] -> [B, n_dst, d] (pyr_glue_rmsnorm_rows); rows int32 [B, n_dst], last dim contiguous."""
    assert x.is_contiguous() and x.dim() == 3 and rows.dtype == torch.int32 and rows.dim() == 2 and rows.stride(1) == 1
    B, n_src, d = x.shape
    n_dst = rows.shape[1]
    out = torch.empty(B, n_dst, d, dtype=x.dtype, device=x.device)
    _check(lib().pyr_glue_rmsnorm_rows(x.data_ptr(), rows.data_ptr(), rows.stride(0), gain.data_ptr(), out.data_ptr(), B, n_src, n_dst, d,
                                       float(eps), _dt(x), C.c_void_p(_stream_ptr(None))), "pyr_glue_rmsnorm_rows")
    return out


def glue_linear_rows(x, w, residual, res_rows):
    """x [B, n_dst, K] . w [N, K]^T + residual[b, res_rows[b, i]] for residual [B, n_src, N] -> [B, n_dst, N] (pyr_glue_linear_rows)."""
    assert x.is_contiguous() and w.is_contiguous() and residual.is_contiguous() and x.dim() == 3 and residual.dim() == 3
    assert res_rows.dtype == torch.int32 and res_rows.dim() == 2 and res_rows.stride(1) == 1 and res_rows.shape[1] == x.shape[1]
    N, K = w.shape
    B, n_dst, _ = x.shape
    y = torch.empty(B, n_dst, N, dtype=x.dtype, device=x.device)
    _check(lib().pyr_glue_linear_rows(x.data_ptr(), w.data_ptr(), residual.data_ptr(), res_rows.data_ptr(), res_rows.stride(0),
                                      y.data_ptr(), B, residual.shape[1], n_dst, N, K, _dt(x), C.c_void_p(_stream_ptr(None))),
           "pyr_glue_linear_rows")
    return y


def glue_linear_split(x, w, n_parts: int):
    """x [..., K] . w [n_parts * part_n, K]^T as n_parts tensors [..., part_n] (pyr_glue_linear_split)."""
    assert x.is_contiguous() and w.is_contiguous() and w.shape[0] % n_parts == 0
    K = w.shape[1]
    part_n = w.shape[0] // n_parts
    ys = [torch.empty(*x.shape[:-1], part_n, dtype=x.dtype, device=x.device) for _ in range(n_parts)]
    arr = (C.c_void_p * n_parts)(*[y.data_ptr() for y in ys])
    _check(lib().pyr_glue_linear_split(x.data_ptr(), w.data_ptr(), arr, n_parts, x.numel() // K, part_n, K, _dt(x),
                                       C.c_void_p(_stream_ptr(None))), "pyr_glue_linear_split")
    return ys


def glue_status() -> int:
    """0, or PYR_ERR_TIMEOUT if a linear layer's bounded wait ran out on this GPU since the last call (pyr_glue_status)."""
    word = C.c_int32(0)
    lib().pyr_glue_status(C.c_void_p(_stream_ptr(None)), C.byref(word))
    return int(word.value)


def glue_linear_swiglu(x, w_gate, w_up):
    """silu(x . w_gate^T) * (x . w_up^T) -> [..., N] in one pass (pyr_glue_linear_swiglu; bf16, K a multiple of 64)."""
    assert x.is_contiguous() and w_gate.is_contiguous() and w_up.is_contiguous() and w_gate.shape == w_up.shape
    N, K = w_gate.shape
    out = torch.empty(*x.shape[:-1], N, dtype=x.dtype, device=x.device)
    _check(lib().pyr_glue_linear_swiglu(x.data_ptr(), w_gate.data_ptr(), w_up.data_ptr(), out.data_ptr(), x.numel() // K, N, K,
                                        _dt(x), C.c_void_p(_stream_ptr(None))), "pyr_glue_linear_swiglu")
    return out


def glue_rope_(x, pos):
    """In place on x [..., H, D] with pos int32 [...] (pyr_glue_rope)."""
    assert x.is_contiguous() and pos.dtype == torch.int32 and pos.is_contiguous()
    _check(lib().pyr_glue_rope(x.data_ptr(), pos.data_ptr(), pos.numel(), x.shape[-2], x.shape[-1], _dt(x),
                               C.c_void_p(_stream_ptr(None))), "pyr_glue_rope")
    return x


def glue_swiglu(gate, up):
    assert gate.is_contiguous() and up.is_contiguous()
    out = torch.empty_like(gate)
    _check(lib().pyr_glue_swiglu(gate.data_ptr(), up.data_ptr(), out.data_ptr(), gate.numel(), _dt(gate),
                                 C.c_void_p(_stream_ptr(None))), "pyr_glue_swiglu")
    return out


def glue_argmax(x):
    assert x.is_contiguous() and x.dim() == 2
    out = torch.empty(x.shape[0], dtype=torch.int32, device=x.device)
    _check(lib().pyr_glue_argmax(x.data_ptr(), out.data_ptr(), x.shape[0], x.shape[1], _dt(x),
                                 C.c_void_p(_stream_ptr(None))), "pyr_glue_argmax")
    return out


def recent_len_from_ratio(prompt_len: int, ratio: float) -> int:
    return int(lib().pyr_recent_len_from_ratio(int(prompt_len), float(ratio)))


def decode_attn_noalloc_status(stream=None) -> int:
    """pyr_decode_attn_noalloc_status: 0, or PYR_ERR_TIMEOUT if a wait of an earlier
    no-alloc call ran out (synchronises the stream; reading clears the record)."""
    w = C.c_int32(0)
    lib().pyr_decode_attn_noalloc_status(C.c_void_p(_stream_ptr(stream)), C.byref(w))
    return w.value


def config_from_workload(w: dict, ratio, **over) -> dict:
    """Keyword arguments of PyrCache for a workload dict (see synth.CONFIGS)."""
    kw = dict(n_layers=w["n_layers"], n_q_heads=w["n_q_heads"], n_kv_heads=w["n_kv_heads"],
              head_dim=w["head_dim"], sel_groups=w["sel_groups"], dtype=w["dtype"], batch=w["batch"],
              prompt_len=w["prompt_len"], recent_len=w["recent_len"], max_new_tokens=w["max_new_tokens"],
              ratio=list(ratio))
    kw.update(over)
    return kw


class PyrCache:
    """A cache handle plus the torch buffer that backs it."""

    def __init__(self, device="cuda", **kw):
        self.cfg, self._keep = make_config(**kw)
        self.kw = dict(kw)
        nbytes, align = pyr_cache_bytes(self.cfg)
        self.nbytes = nbytes
        self.device = torch.device(device)
        self.buf = torch.empty(nbytes + align, dtype=torch.uint8, device=self.device)
        base = self.buf.data_ptr()
        self._off = (-base) % align
        self.handle = C.c_void_p()
        _check(lib().pyr_cache_alloc(C.byref(self.cfg), C.c_void_p(base + self._off), nbytes,
                                     C.byref(self.handle)), "pyr_cache_alloc")
        self.tdtype = torch.bfloat16 if self.cfg.dtype == PYR_BF16 else torch.float32

    def close(self):
        if getattr(self, "handle", None):
            lib().pyr_cache_free(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- host-side queries -------------------------------------------------
    def layer_info(self, layer: int):
        v = [C.c_int32(0) for _ in range(4)]
        _check(lib().pyr_cache_layer_info(self.handle, layer, *[C.byref(x) for x in v]), "pyr_cache_layer_info")
        return {"n_in": v[0].value, "k_ctx": v[1].value, "len_now": v[2].value, "cap": v[3].value}

    def _view(self, ptr: int, shape, dtype):
        """A torch view of library-carved memory inside self.buf."""
        off = ptr - self.buf.data_ptr()
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        return self.buf[off: off + nbytes].view(dtype).view(*shape)

    def kept(self, layer: int):
        i, p = C.c_void_p(), C.c_void_p()
        _check(lib().pyr_cache_kept(self.handle, layer, C.byref(i), C.byref(p)), "pyr_cache_kept")
        info = self.layer_info(layer)
        n_out = info["k_ctx"] + min(self.cfg.recent_len, info["n_in"])
        shape = (self.cfg.batch, self.cfg.sel_groups, n_out)
        return self._view(i.value, shape, torch.int32), self._view(p.value, shape, torch.int32)

    def scores(self, layer: int):
        p = C.c_void_p()
        _check(lib().pyr_cache_scores(self.handle, layer, C.byref(p)), "pyr_cache_scores")
        info = self.layer_info(layer)
        c = max(info["n_in"] - self.cfg.recent_len, 0)
        return self._view(p.value, (self.cfg.batch, self.cfg.sel_groups, c), torch.float32)

    def lse(self, layer: int):
        p = C.c_void_p()
        _check(lib().pyr_cache_lse(self.handle, layer, C.byref(p)), "pyr_cache_lse")
        info = self.layer_info(layer)
        return self._view(p.value, (self.cfg.batch, self.cfg.n_q_heads, info["n_in"]), torch.float32)

    def kv(self, layer: int):
        k, v = C.c_void_p(), C.c_void_p()
        _check(lib().pyr_cache_kv(self.handle, layer, C.byref(k), C.byref(v)), "pyr_cache_kv")
        info = self.layer_info(layer)
        shape = (self.cfg.batch, self.cfg.n_kv_heads, info["cap"], self.cfg.head_dim)
        return self._view(k.value, shape, self.tdtype), self._view(v.value, shape, self.tdtype)

    def status(self, stream=None) -> int:
        w = C.c_int32(0)
        lib().pyr_cache_status(self.handle, C.c_void_p(_stream_ptr(stream)), C.byref(w))
        return w.value

    # --- the path ------------------------------------------------------------
    def reset(self, stream=None):
        _check(lib().pyr_cache_reset(self.handle, C.c_void_p(_stream_ptr(stream))), "pyr_cache_reset")

    def prefill_layer(self, layer: int, q, k, v, out, stream=None):
        """q/out [B, n, Hq, D], k/v [B, n, Hkv, D] (any strides with D contiguous)."""
        assert q.stride(-1) == 1 and k.stride(-1) == 1 and v.stride(-1) == 1 and out.stride(-1) == 1
        assert k.stride() == v.stride()
        _check(lib().pyr_prefill_layer(
            self.handle, layer, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
            q.stride(0), q.stride(1), q.stride(2), k.stride(0), k.stride(1), k.stride(2),
            out.stride(0), out.stride(1), out.stride(2), C.c_void_p(_stream_ptr(stream))), "pyr_prefill_layer")

    def select_compact(self, layer: int, k, v, rows=None, row_elems=0, rows_stride_b=0, rows_stride_n=0,
                       rows_stride_g=0, stream=None) -> int:
        n_out = C.c_int32(0)
        _check(lib().pyr_select_compact(
            self.handle, layer, k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1), k.stride(2),
            C.c_void_p(rows.data_ptr() if rows is not None else None), row_elems, rows_stride_b, rows_stride_n,
            rows_stride_g, C.byref(n_out), C.c_void_p(_stream_ptr(stream))), "pyr_select_compact")
        return n_out.value

    def arm_wait_test(self):
        _check(lib().pyr_cache_arm_wait_test(self.handle), "pyr_cache_arm_wait_test")

    def decode_reselect(self, layer: int, stream=None):
        """pyr_decode_reselect: returns (context rows scored, rows the cache holds afterwards)."""
        c_ctx, n_out = C.c_int32(0), C.c_int32(0)
        _check(lib().pyr_decode_reselect(self.handle, layer, C.byref(c_ctx), C.byref(n_out),
                                         C.c_void_p(_stream_ptr(stream))), "pyr_decode_reselect")
        return c_ctx.value, n_out.value

    def reselect_views(self, layer: int, c_ctx: int, n_out: int):
        """(kept [B, G, n_out] int32, pooled scores [B, G, c_ctx] f32) of the last pyr_decode_reselect
        of `layer` that selected."""
        i, p = C.c_void_p(), C.c_void_p()
        _check(lib().pyr_cache_kept(self.handle, layer, C.byref(i), C.byref(p)), "pyr_cache_kept")
        sp = C.c_void_p()
        _check(lib().pyr_cache_scores(self.handle, layer, C.byref(sp)), "pyr_cache_scores")
        shape = (self.cfg.batch, self.cfg.sel_groups)
        return self._view(i.value, shape + (n_out,), torch.int32), self._view(sp.value, shape + (c_ctx,), torch.float32)

    def decode_attn(self, layer: int, q, k_new, v_new, out, stream=None):
        assert q.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous() and out.is_contiguous()
        _check(lib().pyr_decode_attn(self.handle, layer, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                                     out.data_ptr(), C.c_void_p(_stream_ptr(stream))), "pyr_decode_attn")
