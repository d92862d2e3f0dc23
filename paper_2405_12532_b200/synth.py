"""Seeded synthetic inputs: shapes, schedules and value distributions of the
workloads. Holds none of the method's arithmetic (no attention, no scoring, no
budget rounding): it only draws tensors and lists caller-side parameters, so
both the CUDA library's tests and the CPU checker can be fed from it.
"""
from __future__ import annotations

import torch

# The five workloads. "stack" = attention-only stack with fresh Q/K/V per layer
# drawn at the layer's surviving length; ratio = (start, end) of a geometric
# per-layer retention schedule clamped at `end`, or an explicit list.
CONFIGS = {
    "tiny_fp32": dict(kind="stack", n_layers=2, n_q_heads=4, n_kv_heads=4, head_dim=64,
                      dtype="f32", batch=2, prompt_len=256, recent_len=32,
                      ratio=[1.0, 0.5], sel_groups=1, max_new_tokens=16,
                      hitter_frac=0.02, hitter_mag=3.0),
    "7b_stack_8x2k": dict(kind="stack", n_layers=32, n_q_heads=32, n_kv_heads=32, head_dim=128,
                          dtype="bf16", batch=8, prompt_len=2048, recent_len=256,
                          ratio=(1.0, 0.3), sel_groups=32, max_new_tokens=0,
                          hitter_frac=0.02, hitter_mag=3.0),
    "7b_64x2k": dict(kind="stack", n_layers=32, n_q_heads=32, n_kv_heads=32, head_dim=128,
                     dtype="bf16", batch=64, prompt_len=2048, recent_len=256,
                     ratio=(1.0, 0.3), sel_groups=1, max_new_tokens=128,
                     hitter_frac=0.02, hitter_mag=3.0, hidden=4096),
    "13b_stack_32x4k": dict(kind="stack", n_layers=40, n_q_heads=40, n_kv_heads=40, head_dim=128,
                            dtype="bf16", batch=32, prompt_len=4096, recent_len=512,
                            ratio=(1.0, 0.25), sel_groups=40, max_new_tokens=256,
                            hitter_frac=0.02, hitter_mag=3.0),
    "70b_gqa_16x8k": dict(kind="stack", n_layers=80, n_q_heads=64, n_kv_heads=8, head_dim=128,
                          dtype="bf16", batch=16, prompt_len=8192, recent_len=1024,
                          ratio=(1.0, 0.2), sel_groups=8, max_new_tokens=512,
                          hitter_frac=0.01, hitter_mag=4.0),
    # The shapes of the paper's efficiency tables (Table 1 / Table 2: LLaMA-2-13B at batch 32 with
    # 512 prompt + 256 generated tokens, LLaMA-2-70B at batch 8 with 256 + 128), as attention stacks.
    # The paper's text does not give the schedule or the window behind its numbers: the window is
    # 40 % of the prompt (its Section 5.2 trade-off) and the retention falls geometrically to 0.2.
    "13b_table_32x512": dict(kind="stack", n_layers=40, n_q_heads=40, n_kv_heads=40, head_dim=128,
                             dtype="bf16", batch=32, prompt_len=512, recent_len=204,
                             ratio=(1.0, 0.2), sel_groups=40, max_new_tokens=256,
                             hitter_frac=0.02, hitter_mag=3.0),
    "70b_table_8x256": dict(kind="stack", n_layers=80, n_q_heads=64, n_kv_heads=8, head_dim=128,
                            dtype="bf16", batch=8, prompt_len=256, recent_len=102,
                            ratio=(1.0, 0.2), sel_groups=8, max_new_tokens=128,
                            hitter_frac=0.01, hitter_mag=4.0),
    # The 7B workload as a whole model: the same attention geometry, window and schedule as 7b_64x2k with
    # the public Llama-2-7B block around it (hidden 4096, MLP 11008, vocabulary 32000), random-init weights,
    # uniform random token ids for the prompt and for the decode steps.
    "7b_model_64x2k": dict(kind="model", n_layers=32, n_q_heads=32, n_kv_heads=32, head_dim=128,
                           dtype="bf16", batch=64, prompt_len=2048, recent_len=256,
                           ratio=(1.0, 0.3), sel_groups=1, max_new_tokens=128,
                           hitter_frac=0.0, hitter_mag=0.0, hidden=4096, inter=11008, vocab=32000),
}


def geometric_ratio(n_layers: int, r_start: float, r_end: float) -> list[float]:
    """ratio[l] = max(r_end, r_start * g**l) with g chosen so the last layer
    lands on r_end; the clamp keeps rounding of g**(layers-1) from dipping
    below r_end."""
    if n_layers == 1:
        return [float(r_start)]
    g = (r_end / r_start) ** (1.0 / (n_layers - 1))
    return [max(float(r_end), float(r_start) * g ** l) for l in range(n_layers)]


def ratio_schedule(cfg: dict) -> list[float]:
    r = cfg["ratio"]
    if isinstance(r, tuple):
        return geometric_ratio(cfg["n_layers"], r[0], r[1])
    return [float(x) for x in r]


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[name]


def widen(x: torch.Tensor):
    """The stored (bf16 or fp32) values as float64 numpy, exactly."""
    return x.detach().to("cpu").to(torch.float64).numpy()


def stack_layer_inputs(cfg: dict, layer: int, n: int, device="cpu", batch: int | None = None,
                       seed_base: int = 1000, boost_queries: bool = False):
    """Q [B, n, Hq, D], K, V [B, n, Hkv, D] of one layer of an attention stack.

    Entries are N(0,1). One unit direction u per layer is added, scaled by
    hitter_mag, to the keys at a random hitter_frac of positions (drawn per
    sequence, shared by all heads). boost_queries also adds hitter_mag * u to
    every query, which separates the hitters' scores from the rest.
    """
    B = cfg["batch"] if batch is None else batch
    Hq, Hkv, D = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    dt = torch_dtype(cfg["dtype"])
    gen = torch.Generator(device=device)
    gen.manual_seed(seed_base + layer)
    Q = torch.randn(B, n, Hq, D, generator=gen, device=device, dtype=torch.float32)
    K = torch.randn(B, n, Hkv, D, generator=gen, device=device, dtype=torch.float32)
    V = torch.randn(B, n, Hkv, D, generator=gen, device=device, dtype=torch.float32)
    u = torch.randn(D, generator=gen, device=device, dtype=torch.float32)
    u = u / u.norm()
    hit = torch.rand(B, n, generator=gen, device=device) < cfg["hitter_frac"]
    K = K + cfg["hitter_mag"] * hit[:, :, None, None].to(torch.float32) * u
    if boost_queries:
        Q = Q + cfg["hitter_mag"] * u
    return Q.to(dt).contiguous(), K.to(dt).contiguous(), V.to(dt).contiguous()


def decode_step_inputs(cfg: dict, layer: int, step: int, device="cpu", batch: int | None = None,
                       seed_base: int = 500000):
    """q [B, Hq, D], k_new, v_new [B, Hkv, D] ~ N(0,1) for one decode step."""
    B = cfg["batch"] if batch is None else batch
    Hq, Hkv, D = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    dt = torch_dtype(cfg["dtype"])
    gen = torch.Generator(device=device)
    gen.manual_seed(seed_base + 4096 * layer + step)
    q = torch.randn(B, Hq, D, generator=gen, device=device, dtype=torch.float32).to(dt)
    k = torch.randn(B, Hkv, D, generator=gen, device=device, dtype=torch.float32).to(dt)
    v = torch.randn(B, Hkv, D, generator=gen, device=device, dtype=torch.float32).to(dt)
    return q, k, v


def scaled_config(cfg: dict, **over) -> dict:
    """A copy of a workload with some fields replaced (smaller batch, fewer
    layers, shorter prompt) for cases a CPU check can finish in seconds."""
    out = dict(cfg)
    out.update(over)
    return out


def uniform_token_ids(batch: int, prompt_len: int, vocab: int, seed: int = 0) -> torch.Tensor:
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    return torch.randint(0, vocab, (batch, prompt_len), generator=gen, dtype=torch.int64)


def tiny_llama_weights(hidden: int = 256, n_layers: int = 2, inter: int = 768, vocab: int = 1000, seed: int = 1,
                       std: float = 0.02) -> dict:
    """Random-init weights of the tiny Llama-style decoder as fp32 CPU tensors: every matrix
    N(0, std^2) from one seeded generator in a fixed order, norm gains 1. Matrices are stored
    [in, out]. Draws values only."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    rn = lambda *shape: torch.randn(*shape, generator=gen, dtype=torch.float32) * std
    W = {"emb": rn(vocab, hidden)}
    for l in range(n_layers):
        for nm in ("wq", "wk", "wv", "wo"):
            W[f"{nm}{l}"] = rn(hidden, hidden)
        W[f"wg{l}"] = rn(hidden, inter)
        W[f"wu{l}"] = rn(hidden, inter)
        W[f"wd{l}"] = rn(inter, hidden)
        W[f"n1{l}"] = torch.ones(hidden)
        W[f"n2{l}"] = torch.ones(hidden)
    W["nf"] = torch.ones(hidden)
    W["head"] = rn(hidden, vocab)
    return W


def shard_batch(batch: int, world_size: int, rank: int) -> tuple[int, int]:
    """[start, stop) of the sequences rank `rank` owns when a batch is split
    across data-parallel ranks (sequences are independent: no exchange)."""
    base, rem = divmod(batch, world_size)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)
