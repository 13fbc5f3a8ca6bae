"""Helpers for the GPU parity tests: feed the same seeded inputs to the CUDA path and to the oracle."""
import numpy as np
import torch

from oracle import mixkvq_oracle as O
from paper_2512_19206_b200 import workloads as W


def f32(t):
    return t.to(torch.float32).cpu().numpy()


def make_cache(binding, w, max_tokens=None, importance_mode=0, extras_budget_bytes=0, layout=0, budget_bf16=0,
               budget_u4=0, sink_len=0, v_bits=2):
    cfg = binding.make_config(w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, max_tokens or (w.tokens + 256),
                              residual_len=w.residual_len, group_size=w.group_size, tau_bf16=w.tau_bf16,
                              tau_u4=w.tau_u4, score_bits=w.score_bits, importance_mode=importance_mode,
                              extras_budget_bytes=extras_budget_bytes, block_layout=layout, budget_bf16=budget_bf16,
                              budget_u4=budget_u4, sink_len=sink_len, v_bits=v_bits)
    return binding.Cache(cfg)


def oracle_stream(w, importance_mode=0, budget_bf16=0, budget_u4=0, sink_len=0, v_bits=2):
    return O.OracleStream(g=w.g, R=w.residual_len, G=w.group_size, score_bits=w.score_bits, tau_bf16=w.tau_bf16,
                          tau_u4=w.tau_u4, importance_mode=importance_mode, budget_bf16=budget_bf16, budget_u4=budget_u4,
                          sink_len=sink_len, v_bits=v_bits)


def oracle_streams(w, layer, k, v, q, streams=None, importance_mode=0, budget_bf16=0, budget_u4=0, sink_len=0, v_bits=2):
    """Oracle caches of the requested (b, hk) streams after a bulk append of k, v, q (CPU bf16 tensors)."""
    out = {}
    kf, vf, qf = f32(k), f32(v), f32(q)
    for (b, hk) in streams or [(b, hk) for b in range(w.batch) for hk in range(w.n_kv_heads)]:
        st = oracle_stream(w, importance_mode, budget_bf16, budget_u4, sink_len, v_bits)
        st.append_many(kf[b, hk], vf[b, hk], qf[b, hk * w.g:(hk + 1) * w.g])
        out[(b, hk)] = st
    return out


def compare_regions(cache, layer, w, oracle):
    """Byte equality of every region of every oracle stream with the device cache."""
    for (b, hk), st in oracle.items():
        got = cache.stream_regions(layer, b * w.n_kv_heads + hk)
        want = O.pack_stream(st, layout=cache.cfg.block_layout)
        for key in ("table", "base", "extras", "state", "resK", "sinkK", "sinkV"):
            assert got[key] == want[key], f"stream {(b, hk)} region {key} differs"
        R = w.residual_len
        assert got["resV"] == want["resV"], f"stream {(b, hk)} region resV differs"


def oracle_attention(w, oracle, qd):
    """qd [B,Hq,128] CPU bf16 -> dict stream -> [g,128] float32."""
    qf = f32(qd)
    return {(b, hk): st.attention(qf[b, hk * w.g:(hk + 1) * w.g], W.softmax_scale()) for (b, hk), st in oracle.items()}


def max_abs_err(w, out, ref):
    o = out.cpu().numpy()
    return max(float(np.abs(o[b, hk * w.g:(hk + 1) * w.g] - r).max()) for (b, hk), r in ref.items())
