#!/usr/bin/env python
"""Benchmark of the pyramid prefill-selection path.

One step = one pass of the whole path over one synthetic batch: for every layer
attention + recent-window score, then top-k + K/V gather + in-place compaction
of the hidden rows; then T decode steps over the ragged per-layer caches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line. Under torchrun every rank runs the same per-GPU workload
(sequences are independent: weak scaling, no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2405_12532_b200 import dist as pdist
from paper_2405_12532_b200 import synth

METRIC = "prefill tokens/s + decode tokens/s at 7B shapes 64x2k"
UNIT = "tokens/s (prefill of the attention path, all layers incl. select+compact; no linear layers, no weight reads)"
SCOPE = ("attention path only: per-layer Q/K/V are inputs; a full model's projections, MLP and weight reads "
         "are not in the step")
DEFAULT_WORKLOAD = "7b_64x2k"
MODEL_WORKLOAD = "7b_model_64x2k"      # the same shapes as a whole model; reported beside the default line
PROFILES = os.path.join(ROOT, "profiles")


def traffic_ratio(summary: str):
    """DRAM bytes per algorithmic byte of a kernel, from the ncu summary under profiles/ that
    states it (`traffic_ratio: R`) together with the hash of the source file the kernel was
    built from (`source_sha1: FILE HASH`). None when there is no such line or the source has
    changed since the capture."""
    import hashlib
    import re
    path = os.path.join(PROFILES, summary)
    if not os.path.exists(path):
        return None
    text = open(path).read()
    m = re.search(r"^traffic_ratio:\s*([0-9.]+)", text, re.M)
    h = re.search(r"^source_sha1:\s*(\S+)\s+([0-9a-f]{40})", text, re.M)
    if not m or not h:
        return None
    src = os.path.join(ROOT, "paper_2405_12532_b200", "csrc", h.group(1))
    if not os.path.exists(src) or hashlib.sha1(open(src, "rb").read()).hexdigest() != h.group(2):
        return None
    return float(m.group(1))


def measured_peaks():
    """(hbm GB/s, bf16 TFLOP/s burst, source)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p["bf16_tflops"]), float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "measured"
    return 6650.0, 1590.0, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ ours
class Workload:
    """Device-resident synthetic inputs and the call sequence of one step."""

    def __init__(self, name: str, device, pool: int = 2, layers: int = 0, decode_steps: int = -1, batch: int = 0,
                 reselect_every: int = 0, select_first: str = "auto"):
        from paper_2405_12532_b200 import binding as pb
        self.pb = pb
        self.name = name
        self.w = w = dict(synth.CONFIGS[name])
        self.device = device
        self.ratio = synth.ratio_schedule(w)
        if layers > 0:            # profiling aid: the first `layers` layers of the schedule only
            self.ratio = self.ratio[:layers]
            w["n_layers"] = layers
        if decode_steps >= 0:
            w["max_new_tokens"] = decode_steps
        if batch > 0:             # profiling aid: a smaller batch keeps an ncu capture small
            w["batch"] = batch
        self.reselect_every = reselect_every      # generation-phase PvC update every so many decode steps (0: never)
        flags = pb.PYR_FLAG_GEN_RESELECT if reselect_every else 0
        # Select-first ordering where the rows that select + compact moves are the attention output itself (one kept
        # set per head group): the kept rows are then written in place by the attention kernel. With one kept set per
        # sequence the compacted rows are the hidden states, which attention does not produce. "auto": on for prompts
        # of 4096 tokens and more, where it was measured to win (its two attention launches cost more on short ones).
        want = select_first == "on" or (select_first == "auto" and w["prompt_len"] >= 4096)
        self.select_first = bool(want and w["sel_groups"] > 1 and w["dtype"] == "bf16" and w["head_dim"] == 128)
        if self.select_first:
            flags |= pb.PYR_FLAG_SELECT_FIRST
        self.cache = pb.PyrCache(device=device, **pb.config_from_workload(w, self.ratio, flags=flags))
        self.layers = [self.cache.layer_info(l) for l in range(w["n_layers"])]
        B, N, Hq, Hkv, D = w["batch"], w["prompt_len"], w["n_q_heads"], w["n_kv_heads"], w["head_dim"]
        self.dt = synth.torch_dtype(w["dtype"])
        self.eb = 2 if w["dtype"] == "bf16" else 4
        # a small pool of full-length Q/K/V sets; layer l reads the first n_in rows of set l % pool
        # (values do not change the work done; every tensor is far larger than L2)
        self.pool = [synth.stack_layer_inputs(w, l, N, device=device) for l in range(pool)]
        self.out = torch.empty(B, N, Hq, D, dtype=self.dt, device=device)
        self.G = w["sel_groups"]
        if self.G == 1:
            self.hidden = w.get("hidden", Hq * D)
            self.rows = torch.randn(B, N, self.hidden, device=device).to(self.dt)
        else:
            self.rows = None
        self.T = w["max_new_tokens"]
        self.dec_in = [synth.decode_step_inputs(w, 0, t, device=device) for t in range(4)]
        self.dec_out = torch.empty(B, Hq, D, dtype=self.dt, device=device)

    def release(self):
        """Give the device memory back (the schedule-derived accounting below stays usable)."""
        if self.cache is not None:
            self.cache.close()
        self.cache = self.pool = self.out = self.rows = self.dec_in = self.dec_out = None
        torch.cuda.empty_cache()

    def layer_views(self, l):
        n = self.layers[l]["n_in"]
        Q, K, V = self.pool[l % len(self.pool)]
        return Q[:, :n], K[:, :n], V[:, :n], self.out[:, :n], n

    def select_args(self, l, n):
        w = self.w
        if self.G == 1:
            return (self.rows, self.hidden, self.rows.stride(0), self.hidden, 0)
        rep = w["n_q_heads"] // w["n_kv_heads"]
        D = w["head_dim"]
        return (self.out, rep * D, self.out.stride(0), self.out.stride(1), rep * D)

    def prefill(self, events=None):
        c = self.cache
        c.reset()
        for l in range(self.w["n_layers"]):
            Q, K, V, O, n = self.layer_views(l)
            if events is not None:
                events[l][0].record()
            c.prefill_layer(l, Q, K, V, O)
            if events is not None:
                events[l][1].record()
            c.select_compact(l, K, V, *self.select_args(l, n))
            if events is not None:
                events[l][2].record()

    def decode(self):
        c = self.cache
        for t in range(self.T):
            q, kn, vn = self.dec_in[t % len(self.dec_in)]
            for l in range(self.w["n_layers"]):
                c.decode_attn(l, q, kn, vn, self.dec_out)
            if self.reselect_every and (t + 1) % self.reselect_every == 0:
                for l in range(self.w["n_layers"]):
                    c.decode_reselect(l)

    # ---- algorithmic work, from the schedule
    def prefill_flops(self):
        w = self.w
        return sum(w["batch"] * w["n_q_heads"] * 2 * w["head_dim"] * L["n_in"] * (L["n_in"] + 1) for L in self.layers)

    def prefill_roofline_seconds(self, tflops: float, hbm_gbs: float):
        """Sum over layers of max(flops / tensor peak, compulsory Q+K+V+O bytes / HBM bandwidth):
        the short layers deep in the pyramid are bound by their traffic, not by the contraction."""
        w = self.w
        B, Hq, Hkv, D = w["batch"], w["n_q_heads"], w["n_kv_heads"], w["head_dim"]
        t = 0.0
        for L in self.layers:
            n = L["n_in"]
            flops = B * Hq * 2 * D * n * (n + 1)
            byts = B * n * (2 * Hq + 2 * Hkv) * D * self.eb
            t += max(flops / (tflops * 1e12), byts / (hbm_gbs * 1e9))
        return t

    def prefill_bytes(self):
        w = self.w
        return sum(w["batch"] * L["n_in"] * (2 * w["n_q_heads"] + 2 * w["n_kv_heads"]) * w["head_dim"] * self.eb
                   for L in self.layers)

    def select_compact_bytes(self):
        w = self.w
        B, Hkv, D, G, Lw = w["batch"], w["n_kv_heads"], w["head_dim"], self.G, w["recent_len"]
        tot = 0
        for L in self.layers:
            n = L["n_in"]
            c = max(n - Lw, 0)
            n_out = L["k_ctx"] + (n - c)
            tot += B * G * c * 4 + B * G * n_out * 4                        # scores in, indices out
            tot += 2 * 2 * B * Hkv * n_out * D * self.eb                    # K and V, read + write
            if n_out < n:
                row_b = (self.hidden if G == 1 else (w["n_q_heads"] // Hkv) * D) * self.eb
                # select-first ordering: only the window's rows (and the few kept rows of the tile that holds the
                # window's start, not counted here) are still moved; the others were written in place
                moved = min(Lw, n) if (self.select_first and c > 0) else n_out
                tot += 2 * B * G * moved * row_b                            # compacted rows, read + write
            tot += 2 * B * G * n_out * 4                                    # positions
        return tot

    def decode_bytes(self):
        w = self.w
        tot = 0
        for L in self.layers:
            n_out = L["k_ctx"] + min(w["recent_len"], L["n_in"])
            for t in range(self.T):
                grown = t % self.reselect_every if self.reselect_every else t   # rows appended since the last update
                tot += 2 * w["batch"] * w["n_kv_heads"] * (n_out + grown + 1) * w["head_dim"] * self.eb
        return tot


class ModelWorkload(Workload):
    """The 7B-shaped workload as a whole model on the library's kernels: embedding, RMSNorm, the
    projections and the MLP on the tcgen05 GEMM, rotary embedding at original positions, the pyramid
    path, o_proj on all rows, then the MLP on the kept rows read where they lie (the hidden states are
    never compacted: the norm and the residual of the down projection go through the kept list),
    greedy head. torch holds the tensors."""

    def __init__(self, name: str, device, layers: int = 0, decode_steps: int = -1, batch: int = 0, reselect_every: int = 0):
        from paper_2405_12532_b200 import binding as pb
        self.pb = pb
        self.name = name
        self.w = w = dict(synth.CONFIGS[name])
        self.device = device
        self.ratio = synth.ratio_schedule(w)
        if layers > 0:
            self.ratio = self.ratio[:layers]
            w["n_layers"] = layers
        if decode_steps >= 0:
            w["max_new_tokens"] = decode_steps
        if batch > 0:
            w["batch"] = batch
        self.reselect_every = reselect_every
        flags = pb.PYR_FLAG_GEN_RESELECT if reselect_every else 0
        self.cache = pb.PyrCache(device=device, **pb.config_from_workload(w, self.ratio, flags=flags))
        self.layers = [self.cache.layer_info(l) for l in range(w["n_layers"])]
        self.dt = torch.bfloat16
        self.eb = 2
        self.G = 1
        self.T = w["max_new_tokens"]
        B, N, d, f, V = w["batch"], w["prompt_len"], w["hidden"], w["inter"], w["vocab"]
        g = torch.Generator(device=device)
        g.manual_seed(1)
        rn = lambda *s: (torch.randn(*s, generator=g, device=device, dtype=torch.float32) * 0.02).to(torch.bfloat16)
        self.W = {"emb": rn(V, d), "head": rn(V, d), "nf": torch.ones(d, device=device, dtype=torch.bfloat16)}
        for l in range(w["n_layers"]):
            # q, k, v and gate, up are stored stacked: a decode step streams each stack through one launch, the
            # prefill uses the row blocks as separate weights
            self.W[f"wqkv{l}"] = rn(3 * d, d)
            self.W[f"wgu{l}"] = rn(2 * f, d)
            for i, nm in enumerate(("wq", "wk", "wv")):
                self.W[f"{nm}{l}"] = self.W[f"wqkv{l}"][i * d:(i + 1) * d]
            self.W[f"wg{l}"], self.W[f"wu{l}"] = self.W[f"wgu{l}"][:f], self.W[f"wgu{l}"][f:]
            self.W[f"wo{l}"], self.W[f"wd{l}"] = rn(d, d), rn(d, f)
            self.W[f"n1{l}"] = torch.ones(d, device=device, dtype=torch.bfloat16)
            self.W[f"n2{l}"] = torch.ones(d, device=device, dtype=torch.bfloat16)
        self.ids = synth.uniform_token_ids(B, N, V, seed=0).to(torch.int32).to(device)
        self.dec_ids = synth.uniform_token_ids(B, max(self.T, 1), V, seed=2).to(torch.int32).to(device)
        self.out = None
        self.rows = None

    def prefill(self, events=None):
        pb, W, w = self.pb, self.W, self.w
        B, N, H, D, d = w["batch"], w["prompt_len"], w["n_q_heads"], w["head_dim"], w["hidden"]
        c = self.cache
        c.reset()
        x = pb.glue_embed(self.ids, W["emb"])
        pos = torch.arange(N, device=self.device, dtype=torch.int32).expand(B, N).contiguous()
        for l in range(w["n_layers"]):
            n = x.shape[1]
            if events is not None:
                events[l][0].record()
            h = pb.glue_rmsnorm(x, W[f"n1{l}"])
            q = pb.glue_rope_(pb.glue_linear(h, W[f"wq{l}"]).view(B, n, H, D), pos)
            k = pb.glue_rope_(pb.glue_linear(h, W[f"wk{l}"]).view(B, n, H, D), pos)
            v = pb.glue_linear(h, W[f"wv{l}"]).view(B, n, H, D)
            o = torch.empty_like(q)
            c.prefill_layer(l, q, k, v, o)
            y = pb.glue_linear(o.view(B, n, d), W[f"wo{l}"], x)
            if events is not None:
                events[l][1].record()
            c.select_compact(l, k, v, None, 0, 0, 0, 0)      # K/V into the cache, kept list, positions; y stays where it is
            if events is not None:
                events[l][2].record()
            kept, kept_pos = c.kept(l)
            rows = kept[:, 0]                                # [B, n_out]: the kept rows of every sequence
            pos = kept_pos[:, 0].contiguous()
            h2 = pb.glue_rmsnorm_rows(y, rows, W[f"n2{l}"])
            x = pb.glue_linear_rows(pb.glue_linear_swiglu(h2, W[f"wg{l}"], W[f"wu{l}"]), W[f"wd{l}"], y, rows)
        logits = pb.glue_linear(pb.glue_rmsnorm(x[:, -1].contiguous(), W["nf"]), W["head"])
        self.first_token = pb.glue_argmax(logits)

    def decode(self):
        pb, W, w = self.pb, self.W, self.w
        B, N, H, D, d = w["batch"], w["prompt_len"], w["n_q_heads"], w["head_dim"], w["hidden"]
        c = self.cache
        for t in range(self.T):
            xt = pb.glue_embed(self.dec_ids[:, t].contiguous(), W["emb"])      # pre-drawn ids: the timing does not hang on ties
            p = torch.full((B,), N + t, device=self.device, dtype=torch.int32)
            for l in range(w["n_layers"]):
                h = pb.glue_rmsnorm(xt, W[f"n1{l}"])
                q, k, v = pb.glue_linear_split(h, W[f"wqkv{l}"], 3)
                q, k, v = pb.glue_rope_(q.view(B, H, D), p), pb.glue_rope_(k.view(B, H, D), p), v.view(B, H, D)
                o = torch.empty_like(q)
                c.decode_attn(l, q, k, v, o)
                y = pb.glue_linear(o.view(B, d), W[f"wo{l}"], xt)
                h2 = pb.glue_rmsnorm(y, W[f"n2{l}"])
                g, u = pb.glue_linear_split(h2, W[f"wgu{l}"], 2)
                xt = pb.glue_linear(pb.glue_swiglu(g, u), W[f"wd{l}"], y)
            self.last_token = pb.glue_argmax(pb.glue_linear(pb.glue_rmsnorm(xt, W["nf"]), W["head"]))
            if self.reselect_every and (t + 1) % self.reselect_every == 0:
                for l in range(w["n_layers"]):
                    c.decode_reselect(l)

    def linear_flops(self):
        w = self.w
        B, d, f = w["batch"], w["hidden"], w["inter"]
        tot = 0
        for L in self.layers:
            n_out = L["k_ctx"] + min(w["recent_len"], L["n_in"])
            tot += 2 * B * L["n_in"] * 4 * d * d + 2 * B * n_out * 3 * d * f
        return tot + 2 * B * d * w["vocab"]

    def weight_bytes(self):
        w = self.w
        d, f = w["hidden"], w["inter"]
        return (w["n_layers"] * (4 * d * d + 3 * d * f) + d * w["vocab"]) * 2

    def select_args(self, l, n):
        raise NotImplementedError


def run_model(args, rank, world, local_rank, name, emit=True):
    """One line for the whole-model workload: the same step (prefill of all layers, then T decode steps),
    now with the model's linear layers, norms, rotary embedding and head inside it. With emit=False the
    line is returned (rank 0; None elsewhere) instead of printed."""
    from paper_2405_12532_b200 import binding as pb
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    wl = ModelWorkload(name, device, layers=args.layers, decode_steps=args.decode_steps, batch=args.batch,
                       reselect_every=args.reselect_every)
    w = wl.w
    hbm, tf_burst, tf_sust, peak_src = measured_peaks()
    for _ in range(args.warmup):
        wl.prefill(); wl.decode()
    pdist.barrier(world)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = pb.launch_count()
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    pdist.barrier(world)
    for s in range(args.steps):
        marks[s][0].record(); wl.prefill(); marks[s][1].record(); wl.decode(); marks[s][2].record()
    pdist.barrier(world)
    launches = pb.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    assert wl.cache.status() == 0 and pb.glue_status() == 0, "device-side wait timed out"
    t_pre = sum(m[0].elapsed_time(m[1]) for m in marks) / 1e3
    t_dec = sum(m[1].elapsed_time(m[2]) for m in marks) / 1e3
    t_pre, t_dec = pdist.max_over_ranks([t_pre, t_dec], world, device)
    wl.cache.close()
    wl.cache = wl.W = None
    torch.cuda.empty_cache()
    if rank != 0:
        return None
    K, B, N, T = args.steps, w["batch"], w["prompt_len"], w["max_new_tokens"]
    flops = wl.linear_flops() + wl.prefill_flops()
    dec_bytes = wl.decode_bytes() + T * wl.weight_bytes()
    ach = K * flops / t_pre / 1e12
    line = {"metric": METRIC, "value": world * K * B * N / t_pre,
            "unit": "tokens/s (prefill, whole model: linear layers, norms, rotary embedding and the attention path)",
            "decode_tokens_per_s": world * K * B * T / t_dec if T > 0 else None,
            "n_gpus": world, "steps": K, "warmup": args.warmup, "ms_per_step": (t_pre + t_dec) / K * 1e3,
            "ms_prefill": t_pre / K * 1e3, "ms_decode": t_dec / K * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name, "scope": "whole model on the library's kernels; random-init weights, uniform random token ids",
                       "layers": w["n_layers"], "batch_per_gpu": B, "prompt_len": N, "recent_len": w["recent_len"],
                       "decode_steps": T, "hidden": w["hidden"], "inter": w["inter"], "vocab": w["vocab"],
                       "ratio": "geometric 1.0->%.2f" % wl.ratio[-1], "reselect_every": args.reselect_every or None,
                       "l2": "weights (13.5 GB) and activations are far larger than L2"},
            "roofline": {"kernel": "prefill: linear layers (tcgen05 GEMM) + attention path", "bound": "tensor", "achieved": ach,
                         "peak": tf_burst, "unit": "TFLOP/s", "frac": ach / tf_burst, "frac_of_sustained": ach / tf_sust,
                         "traffic": None, "peak_source": f"of {peak_src}"},
            "roofline_decode": ({"kernel": "decode: weights streamed once per step + K/V caches", "bound": "hbm",
                                 "achieved": K * dec_bytes / t_dec / 1e9, "peak": hbm, "unit": "GB/s",
                                 "frac": K * dec_bytes / t_dec / 1e9 / hbm, "traffic": None, "peak_source": f"of {peak_src}"}
                                if T > 0 else None),
            "gpu_launches": launches, "clocks": clocks, "e2e": None, "cpu_baseline": None}
    if emit:
        print(json.dumps(line), flush=True)
    return line


def run_ours(args, rank, world, local_rank, workload=None):
    from paper_2405_12532_b200 import binding as pb
    name = workload or args.workload
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    wl = Workload(name, device, layers=args.layers, decode_steps=args.decode_steps, batch=args.batch,
                  reselect_every=args.reselect_every, select_first=args.select_first)
    w = wl.w
    nL = w["n_layers"]
    hbm, tf_burst, tf_sust, peak_src = measured_peaks()

    def barrier():
        pdist.barrier(world)

    for _ in range(args.warmup):
        wl.prefill(); wl.decode()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = pb.launch_count()
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(nL)] for _ in range(args.steps)]
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    t0 = time.perf_counter()
    for s in range(args.steps):
        marks[s][0].record()
        wl.prefill(ev[s])
        marks[s][1].record()
        wl.decode()
        marks[s][2].record()
    barrier()
    wall = time.perf_counter() - t0
    launches = pb.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    assert wl.cache.status() == 0, "device-side wait timed out"

    t_pre = sum(m[0].elapsed_time(m[1]) for m in marks) / 1e3
    t_dec = sum(m[1].elapsed_time(m[2]) for m in marks) / 1e3
    t_attn = sum(e[0].elapsed_time(e[1]) for st in ev for e in st) / 1e3
    t_sel = sum(e[1].elapsed_time(e[2]) for st in ev for e in st) / 1e3
    t_pre, t_dec, t_attn, t_sel, t_all = pdist.max_over_ranks([t_pre, t_dec, t_attn, t_sel, t_pre + t_dec], world, device)

    K = args.steps
    B, N, T = w["batch"], w["prompt_len"], w["max_new_tokens"]
    prefill_tps = pdist.whole_job_rate(K * B * N, world, t_pre)
    decode_tps = world * K * B * T / t_dec if T > 0 and t_dec > 0 else None

    # ---- end to end: host buffers, copies inside the timed region
    e2e = run_e2e(wl, args, barrier, world) if not args.no_e2e else None
    wl.release()

    # the same 7B shapes as a whole model (linear layers, norms, rotary embedding, head), reported beside the
    # attention-path numbers of the headline line
    model = None
    if name == DEFAULT_WORKLOAD and not args.no_model and not (args.layers or args.batch or args.decode_steps >= 0):
        # an auxiliary figure: a few steps are enough, however long the headline run is asked to be
        margs = argparse.Namespace(**vars(args))
        margs.steps, margs.warmup = min(args.steps, 5), min(args.warmup, 3)
        model = run_model(margs, rank, world, local_rank, MODEL_WORKLOAD, emit=False)

    if rank != 0:
        return
    dec_bytes = wl.decode_bytes()
    dec_launches = nL * T
    roof_dec = None
    if T > 0:
        ach = K * dec_bytes / t_dec / 1e9
        rr = traffic_ratio("decode_kernel_7b_2k_batch16.txt")
        roof_dec = {"kernel": "decode_kernel", "bound": "hbm", "achieved": ach, "peak": hbm, "unit": "GB/s",
                    "frac": ach / hbm, "traffic": rr * dec_bytes / dec_launches if rr else None,
                    "traffic_note": "dram read+write bytes per launch, scaled from one ncu capture at batch 16 "
                                    "(profiles/decode_kernel_7b_2k_batch16.txt) by the rows streamed",
                    "peak_source": f"of {peak_src}",
                    "launches": K * dec_launches, "avg_launch_us": t_dec / (K * dec_launches) * 1e6,
                    "algorithmic_bytes_per_launch": dec_bytes / dec_launches,
                    "reselect_every": args.reselect_every or None}
    ach_tf = K * wl.prefill_flops() / t_attn / 1e12
    t_roof = wl.prefill_roofline_seconds(tf_burst, hbm)
    t_roof_s = wl.prefill_roofline_seconds(tf_sust, hbm)
    rr = traffic_ratio("attn_tc_kernel_7b_2k_batch16.txt")
    roof_pre = {"kernel": "prefill attention + score", "bound": "tensor", "achieved": ach_tf, "peak": tf_burst,
                "unit": "TFLOP/s", "frac": ach_tf / tf_burst, "frac_of_sustained": ach_tf / tf_sust,
                # per layer max(flops / tensor peak, Q+K+V+O bytes / HBM bandwidth), summed, over the measured time
                "frac_of_layer_roofline": K * t_roof / t_attn, "frac_of_layer_roofline_sustained": K * t_roof_s / t_attn,
                "traffic": rr * wl.prefill_bytes() / nL if rr else None,
                "traffic_note": "dram bytes of the attention kernel per launch (average layer), scaled from one ncu "
                                "capture at batch 16 by the Q+K+V+O bytes",
                "peak_source": f"of {peak_src}", "launches": K * nL * 2, "avg_layer_us": t_attn / (K * nL) * 1e6}
    ach_sel = K * wl.select_compact_bytes() / t_sel / 1e9
    rr = traffic_ratio("select_compact_7b_2k_batch16.txt")
    roof_sel = {"kernel": "select + gather + compact", "bound": "hbm", "achieved": ach_sel, "peak": hbm,
                "unit": "GB/s", "frac": ach_sel / hbm,
                "traffic": rr * wl.select_compact_bytes() / nL if rr else None,
                "traffic_note": "dram bytes per layer (average), scaled from the ncu captures of the call's three kernels at "
                                "batch 16 (profiles/select_compact_7b_2k_batch16.txt)",
                "peak_source": f"of {peak_src}", "avg_layer_us": t_sel / (K * nL) * 1e6}
    dominant = roof_dec if (roof_dec and t_dec >= t_attn) else roof_pre
    line = {
        "metric": METRIC, "value": prefill_tps, "unit": UNIT,
        "decode_tokens_per_s": decode_tps,
        "n_gpus": world, "steps": K, "warmup": args.warmup, "ms_per_step": t_all / K * 1e3,
        "ms_prefill": t_pre / K * 1e3, "ms_decode": t_dec / K * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w["dtype"], "data": "synthetic",
        "config": {"workload": name, "scope": SCOPE, "layers": nL, "batch_per_gpu": B, "prompt_len": N,
                   "recent_len": w["recent_len"], "decode_steps": T, "sel_groups": w["sel_groups"],
                   "heads": w["n_q_heads"], "kv_heads": w["n_kv_heads"], "head_dim": w["head_dim"],
                   "ratio": "geometric 1.0->%.2f" % wl.ratio[-1],
                   "reselect_every": args.reselect_every or None,
                   "ordering": ("select-first: the window's query tiles, scores and selection, then the other tiles writing "
                                "kept rows in place (the selection is timed with the attention)") if wl.select_first else "default",
                   "l2": "inputs larger than L2 (each of Q, K, V and the cache is >= 1 GB)"},
        "roofline": dominant, "roofline_prefill": roof_pre, "roofline_select_compact": roof_sel,
        "roofline_decode": roof_dec,
        "gpu_launches": launches, "wall_s": wall, "clocks": clocks, "e2e": e2e,
        "cpu_baseline": cpu_baseline(name) if not args.no_cpu else None,
    }
    if model is not None:
        line["whole_model"] = {k: model[k] for k in ("value", "unit", "decode_tokens_per_s", "ms_prefill", "ms_decode",
                                                      "roofline", "roofline_decode", "gpu_launches", "clocks")}
        line["whole_model"]["workload"] = MODEL_WORKLOAD
        line["whole_model"]["steps"], line["whole_model"]["warmup"] = model["steps"], model["warmup"]
    print(json.dumps(line), flush=True)


def run_e2e(wl, args, barrier, world):
    """The same step driven from pinned host buffers: each layer's Q/K/V are
    copied host->device before its calls, the last layer's attention output and
    every decode output are copied back. `value` is the headline metric (prefill
    tokens/s) with those copies inside the timed region."""
    w = wl.w
    steps = max(1, min(args.steps, args.e2e_steps))
    host_pool = [tuple(x.to("cpu").pin_memory() for x in qkv) for qkv in wl.pool[:1]]
    hq, hk, hv = host_pool[0]
    dq, dk, dv = wl.pool[0]
    dec_host = [tuple(x.to("cpu").pin_memory() for x in d) for d in wl.dec_in[:1]]
    out_host = torch.empty(wl.out.shape, dtype=wl.out.dtype).pin_memory()
    dec_out_host = torch.empty(wl.dec_out.shape, dtype=wl.dec_out.dtype).pin_memory()
    c = wl.cache
    nL = w["n_layers"]
    h2d = d2h = 0
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]

    def step(count, mk=None):
        nonlocal h2d, d2h
        c.reset()
        if mk:
            mk[0].record()
        for l in range(nL):
            n = wl.layers[l]["n_in"]
            for src, dst in ((hq, dq), (hk, dk), (hv, dv)):
                # one contiguous copy per sequence: a [:, :n] slice of the pinned tensor is strided across
                # the batch, and a strided host->device copy goes through a slow staging path
                for bi in range(src.shape[0]):
                    dst[bi, :n].copy_(src[bi, :n], non_blocking=True)
                if count:
                    h2d += src[:, :n].numel() * src.element_size()
            O = wl.out[:, :n]
            c.prefill_layer(l, dq[:, :n], dk[:, :n], dv[:, :n], O)
            c.select_compact(l, dk[:, :n], dv[:, :n], *wl.select_args(l, n))
        n_last = wl.layers[-1]["n_in"]
        for bi in range(out_host.shape[0]):
            out_host[bi, :n_last].copy_(wl.out[bi, :n_last], non_blocking=True)
        if count:
            d2h += wl.out[:, :n_last].numel() * wl.out.element_size()
        if mk:
            mk[1].record()
        q, kn, vn = wl.dec_in[0]
        hq1, hk1, hv1 = dec_host[0]
        for t in range(wl.T):
            for l in range(nL):
                q.copy_(hq1, non_blocking=True); kn.copy_(hk1, non_blocking=True); vn.copy_(hv1, non_blocking=True)
                c.decode_attn(l, q, kn, vn, wl.dec_out)
                dec_out_host.copy_(wl.dec_out, non_blocking=True)
                if count:
                    h2d += (q.numel() + kn.numel() + vn.numel()) * q.element_size()
                    d2h += wl.dec_out.numel() * wl.dec_out.element_size()
            if wl.reselect_every and (t + 1) % wl.reselect_every == 0:
                for l in range(nL):
                    c.decode_reselect(l)
        if mk:
            mk[2].record()

    step(False)
    barrier()
    for i in range(steps):
        step(True, marks[i])
    barrier()
    t_pre = sum(m[0].elapsed_time(m[1]) for m in marks) / 1e3
    t_dec = sum(m[1].elapsed_time(m[2]) for m in marks) / 1e3
    t_pre, t_dec = pdist.max_over_ranks([t_pre, t_dec], world, wl.device)
    B, N, T = w["batch"], w["prompt_len"], w["max_new_tokens"]
    return {"value": world * steps * B * N / t_pre, "unit": UNIT,
            "decode_tokens_per_s": world * steps * B * T / t_dec if T > 0 and t_dec > 0 else None,
            "steps": steps, "ms_per_step": (t_pre + t_dec) / steps * 1e3, "ms_prefill": t_pre / steps * 1e3,
            "h2d_bytes_per_step": h2d // steps, "d2h_bytes_per_step": d2h // steps}


# ------------------------------------------------------------------------------------------ oracle
def oracle_sample(workload: str, layers=None):
    """Times the fp64 oracle, as it stands, on ONE sequence of the workload at a
    few layers; returns (seconds, description, est. prefill tokens/s for a full pass)."""
    import numpy as np
    import oracle
    w = synth.CONFIGS[workload]
    ratio = synth.ratio_schedule(w)
    budgets = oracle.layer_budgets(w["prompt_len"], w["recent_len"], ratio)
    nL = len(budgets)
    if layers is None:
        # evenly spaced layers, as many (3 to 16) as keep the sample near 10-15 s of host time:
        # about 8e9 head x key x query x dim products per second on the hosts measured so far
        cost = lambda ls: sum(budgets[l]["n_in"] ** 2 for l in ls) * w["n_q_heads"] * w["head_dim"]
        spaced = lambda k: sorted({round(i * (nL - 1) / (k - 1)) for i in range(k)})
        layers = spaced(min(3, nL)) if nL > 1 else [0]
        for k in range(4, min(nL, 16) + 1):
            if cost(spaced(k)) > 1.3e11:
                break
            layers = spaced(k)
    cores = len(os.sched_getaffinity(0))
    torch.set_num_threads(cores)
    t_total = 0.0
    for l in layers:
        bud = budgets[l]
        Q, K, V = synth.stack_layer_inputs(w, l, bud["n_in"], device="cpu", batch=1)
        Qn, Kn, Vn = synth.widen(Q), synth.widen(K), synth.widen(V)
        t0 = time.perf_counter()
        oracle.prefill_layer(Qn, Kn, Vn, w["recent_len"], bud["k"], w["sel_groups"])
        t_total += time.perf_counter() - t0
    work = lambda ls: sum(budgets[l]["n_in"] ** 2 for l in ls)
    t_full = t_total * work(range(nL)) / work(layers)
    desc = (f"1 of {w['batch']} sequences, layers {layers} of {nL} (attention + score + top-k + gather), "
            f"scaled to all layers by sum of n_in^2")
    return t_total, desc, w["prompt_len"] / t_full, cores


def cpu_baseline(workload: str):
    t, desc, tps, cores = oracle_sample(workload)
    return {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "sample_seconds": t,
            "note": "estimated from the sample"}


def run_reference(args, rank, world):
    if rank != 0:
        return
    w = synth.CONFIGS[args.workload]
    nL = w["n_layers"]
    per_step = []
    desc = cores = None
    for i in range(args.warmup + args.steps):
        layers = [0] if i < args.warmup else [nL - 1]      # warm-up: one layer; timed: the smallest layer
        t0 = time.perf_counter()
        t, desc, tps, cores = oracle_sample(args.workload, layers)
        if i >= args.warmup:
            per_step.append((time.perf_counter() - t0, tps))
    value = statistics.mean(x[1] for x in per_step)
    ms = statistics.mean(x[0] for x in per_step) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "scope": SCOPE},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                             "note": "estimated from the sample"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_dry(args, rank, world):
    """Launch-path check without a GPU: the ranks meet on gloo, agree on the slowest rank's time
    as the timed run does, and rank 0 prints what the launch looked like."""
    pdist.init("gloo") if world > 1 else None
    pdist.barrier(world)
    mx = pdist.max_over_ranks([1.0 + rank], world)
    lo, hi = synth.shard_batch(synth.CONFIGS[args.workload]["batch"] * world, world, rank)
    pdist.barrier(world)
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "slowest_rank_seconds": mx[0],
                          "rank0_sequences": [lo, hi], "workload": args.workload}), flush=True)


def run(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.dry_run:
        try:
            run_dry(args, rank, world)
        finally:
            if world > 1 and torch.distributed.is_initialized():
                torch.distributed.destroy_process_group()
        return
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if world > 1:
        pdist.init("nccl", torch.device("cuda", local_rank))
    try:
        names = list(synth.CONFIGS) if args.workload == "all" else [args.workload]
        if args.workload == "all":
            args.no_model = True    # the whole-model workload has its own line in this mode
        for name in names:          # "all": one line per workload, back to back
            if synth.CONFIGS[name]["kind"] == "model":
                run_model(args, rank, world, local_rank, name)
            else:
                run_ours(args, rank, world, local_rank, name)
            torch.cuda.empty_cache()
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


def _spawned(rank, args, port):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(args.gpus), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    run(args)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(synth.CONFIGS) + ["all"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--select-first", default="auto", choices=["auto", "on", "off"],
                    help="select-first ordering on the per-head workloads: the window's query tiles, the scores and the "
                         "selection first, then the other tiles writing kept rows in place (auto: prompts of 4096 tokens and more)")
    ap.add_argument("--no-model", action="store_true", help="skip the whole-model run that the default workload reports beside its line")
    ap.add_argument("--reselect-every", type=int, default=0,
                    help="generation-phase PvC update of every layer every so many decode steps (0: never)")
    ap.add_argument("--dry-run", action="store_true", help="launch path only (gloo, no GPU work)")
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: only the first LAYERS layers")
    ap.add_argument("--decode-steps", type=int, default=-1, help="profiling aid: override the decode steps")
    ap.add_argument("--batch", type=int, default=0, help="profiling aid: override the batch size")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        # not under a launcher: start one rank per GPU here (each rank reads RANK / WORLD_SIZE as under torchrun)
        import socket
        import torch.multiprocessing as mp
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        mp.spawn(_spawned, args=(args, port), nprocs=args.gpus, join=True)
        return
    run(args)


if __name__ == "__main__":
    main()
