"""Seeded synthetic inputs shaped like the paper's long chain-of-thought decode workloads.

This module only draws random tensors; it contains none of the method's arithmetic and is the one
module that both the tests' CPU oracle and the CUDA path take inputs from.

Recipe (per layer): K, V, Q ~ N(0, 1) in bf16.  Four of the 128 key channels per (layer, KV head) are
outlier channels scaled by a factor uniform in [10, 30]; query channels carry a per-(KV head, channel)
gain log-uniform in [0.5, 4] shared by the heads of the GQA group, times a per-head jitter in
[0.8, 1.25]; values have no outliers.  Tokens are produced in fixed chunks of CHUNK tokens, each
chunk from its own generator seed, so a token range is the same however it is requested.  With
``drift=True`` (the long-CoT stream) each outlier slot lives 16384 tokens (staggered by 4096), ramps
its gain 1 -> a -> 1 over its life and then moves to another seeded channel.
"""
from __future__ import annotations

import dataclasses
import math

import torch

CHUNK = 1024
D = 128


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    tokens: int                 # cached tokens at the timed state
    seed: int
    residual_len: int = 128
    group_size: int = 32
    tau_bf16: float = 6.5
    tau_u4: float = 1e30
    score_bits: int = 2
    drift: bool = False
    n_outliers: int = 4

    @property
    def g(self):
        return self.n_q_heads // self.n_kv_heads


# thresholds calibrated once on this distribution with the CPU oracle and frozen
P24 = dict(tau_bf16=6.5, tau_u4=1e30, score_bits=2)          # ~4 promoted channels, UINT4 tier empty
P27 = dict(tau_bf16=6.5, tau_u4=3.8, score_bits=2)           # three tiers
P4BASE = dict(tau_bf16=1.3, tau_u4=-1.0, score_bits=4)      # 4-bit base: nothing stays at 2 bits

CONFIGS = {
    "tiny":      Workload("tiny", 1, 1, 1, 1, 1024, 0x5EED0001),
    "qwen7b":    Workload("qwen2.5-7b-decode", 28, 8, 28, 4, 32768, 0x5EED0002),
    "llama8b":   Workload("llama-3.1-8b-decode", 32, 16, 32, 8, 16384, 0x5EED0003),
    "qwen32b":   Workload("qwen2.5-32b-decode", 64, 64, 40, 8, 32768, 0x5EED0004, group_size=128),
    "longcot":   Workload("long-cot-stream", 28, 4, 28, 4, 131072, 0x5EED0005, drift=True),
}


def _gen(device, *keys):
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in keys:
        s = ((s ^ (int(k) & 0xFFFFFFFFFFFFFFFF)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        s ^= s >> 31
    g.manual_seed(s & 0x7FFFFFFFFFFFFFFF)
    return g


def layer_gains(w: Workload, layer: int):
    """CPU tensors: outlier channels [Hkv, n_out] (int64), outlier factors [Hkv, n_out], query gains [Hq, D]."""
    g = _gen("cpu", w.seed, layer, 0xA11)
    chans = torch.stack([torch.randperm(D, generator=g)[: w.n_outliers] for _ in range(w.n_kv_heads)])
    factors = 10.0 + 20.0 * torch.rand(w.n_kv_heads, w.n_outliers, generator=g)
    qg = 0.5 * torch.pow(8.0, torch.rand(w.n_kv_heads, D, generator=g))
    jitter = 0.8 + 0.45 * torch.rand(w.n_q_heads, 1, generator=g)
    qgain = qg.repeat_interleave(w.g, dim=0) * jitter
    return chans, factors, qgain


def _key_gain(w: Workload, layer: int, t0: int, n: int, device):
    """Per-token key gain [Hkv, n, D] (float32)."""
    chans, factors, _ = layer_gains(w, layer)
    gain = torch.ones(w.n_kv_heads, n, D, dtype=torch.float32)
    if not w.drift:
        for hk in range(w.n_kv_heads):
            gain[hk, :, chans[hk]] = factors[hk]
        return gain.to(device)
    life, stagger = 16384, 4096
    tok = torch.arange(t0, t0 + n)
    for hk in range(w.n_kv_heads):
        for slot in range(w.n_outliers):
            shifted = tok + slot * stagger
            epoch = shifted // life
            phase = (shifted % life).to(torch.float32) / life
            ramp = 1.0 - (2.0 * phase - 1.0).abs()                     # 0 -> 1 -> 0 over the life
            for ep in epoch.unique().tolist():
                ge = _gen("cpu", w.seed, layer, hk, slot, ep, 0xD21F7)
                ch = int(torch.randint(0, D, (1,), generator=ge))
                a = float(10.0 + 20.0 * torch.rand(1, generator=ge))
                m = epoch == ep
                gain[hk, m, ch] = torch.maximum(gain[hk, m, ch], 1.0 + (a - 1.0) * ramp[m])
    return gain.to(device)


def _chunk(w: Workload, layer: int, ci: int, device):
    g = _gen(device, w.seed, layer, ci, 0xC0DE)
    shape_kv = (w.batch, w.n_kv_heads, CHUNK, D)
    k = torch.randn(shape_kv, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(shape_kv, generator=g, device=device, dtype=torch.float32)
    q = torch.randn((w.batch, w.n_q_heads, CHUNK, D), generator=g, device=device, dtype=torch.float32)
    _, _, qgain = layer_gains(w, layer)
    k = k * _key_gain(w, layer, ci * CHUNK, CHUNK, device)[None]
    q = q * qgain.to(device)[None, :, None, :]
    return k.to(torch.bfloat16), v.to(torch.bfloat16), q.to(torch.bfloat16)


def tokens(w: Workload, layer: int, t0: int, n: int, device="cpu"):
    """(k [B,Hkv,n,D], v [B,Hkv,n,D], q [B,Hq,n,D]) bf16 for tokens [t0, t0+n) of a layer."""
    ks, vs, qs = [], [], []
    t = t0
    while t < t0 + n:
        ci, off = divmod(t, CHUNK)
        m = min(CHUNK - off, t0 + n - t)
        k, v, q = _chunk(w, layer, ci, device)
        ks.append(k[:, :, off:off + m]); vs.append(v[:, :, off:off + m]); qs.append(q[:, :, off:off + m])
        t += m
    cat = (lambda xs: xs[0].contiguous() if len(xs) == 1 else torch.cat(xs, dim=2))
    return cat(ks), cat(vs), cat(qs)


def decode_query(w: Workload, layer: int, step: int, device="cpu"):
    """One decode-step query [B, Hq, D] bf16 (same gains as the cached queries)."""
    g = _gen(device, w.seed, layer, step, 0xDEC0DE)
    q = torch.randn((w.batch, w.n_q_heads, D), generator=g, device=device, dtype=torch.float32)
    _, _, qgain = layer_gains(w, layer)
    return (q * qgain.to(device)[None]).to(torch.bfloat16)


def softmax_scale():
    return 1.0 / math.sqrt(D)


def small(w: Workload, **kw):
    """A reduced copy of a workload (fewer layers / batch / tokens) with the same distributions."""
    return dataclasses.replace(w, **kw)
