"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times.

One layer of each configuration is built at its full batch and context from the seeded generator (on the GPU, in
the prefill chunks bench.py uses).  A few sampled (batch, KV head) streams are copied to the host and fed to the
CPU oracle: their packed bytes must be identical and their attention outputs within 2e-3.  The remaining streams
are checked by properties that hold at any size: finite outputs inside the value range, and equal results from the
two independent attention kernels.
"""
import numpy as np
import pytest
import torch

import gpu_util as U
from oracle import mixkvq_oracle as O
from paper_2512_19206_b200 import workloads as W

pytestmark = pytest.mark.gpu
ATTN_TOL = 2e-3
CHUNK = 4096


@pytest.fixture(scope="module")
def binding():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19206_b200 import build
    build.build()
    from paper_2512_19206_b200 import binding as b
    b.lib()
    return b


def _build(binding, w, streams, layout=0, layer=0):
    """Fills one layer on the GPU; returns the cache and the oracle streams of the sampled (b, hk)."""
    # with a 4-bit base every channel has a high plane: give the promoted-channel arena room for it
    budget = ((w.tokens + 2 * w.residual_len) // w.residual_len + 1) * 8192 if w.score_bits == 4 else 0
    cache = U.make_cache(binding, w, max_tokens=w.tokens + 2 * w.residual_len, layout=layout, extras_budget_bytes=budget)
    orc = {s: U.oracle_stream(w) for s in streams}
    t = 0
    while t < w.tokens:
        n = min(CHUNK, w.tokens - t)
        k, v, q = W.tokens(w, layer, t, n, device="cuda")
        cache.quantize_append(0, k, v, q)
        for (b, hk), st in orc.items():
            st.append_many(U.f32(k[b, hk]), U.f32(v[b, hk]), U.f32(q[b, hk * w.g:(hk + 1) * w.g]))
        t += n
    torch.cuda.synchronize()
    assert cache.status() == 0
    return cache, orc


def _check(binding, w, cache, orc, layer=0, kinds=(0,)):
    qd = W.decode_query(w, layer, 0, device="cuda")
    outs = []
    for kind in kinds:
        cache.set_attention_kernel(kind)
        outs.append(cache.decode_attention(0, qd, W.softmax_scale()))
    torch.cuda.synchronize()
    out = outs[0]
    assert torch.isfinite(out).all()
    ref = U.oracle_attention(w, orc, qd.cpu())
    err = U.max_abs_err(w, out, ref)
    assert err <= ATTN_TOL, err
    for other in outs[1:]:                        # every stream: the independent kernel agrees
        assert float((other - out).abs().max()) <= ATTN_TOL
    U.compare_regions(cache, 0, w, orc)           # packed bytes of the sampled streams
    assert cache.status() == 0
    return err


def test_qwen7b_32k_full_batch(binding):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, **W.P24)                   # B = 8, Hkv = 4, g = 7, T = 32768
    cache, orc = _build(binding, w, [(0, 0), (3, 2), (7, 3)])
    _check(binding, w, cache, orc, kinds=(0, 1))


def test_qwen7b_32k_tile_layout(binding):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, **W.P27)
    cache, orc = _build(binding, w, [(1, 1), (6, 0)], layout=1)
    _check(binding, w, cache, orc)


@pytest.mark.parametrize("preset", ["P24", "P4BASE"])
def test_llama8b_16k_full_batch(binding, preset):
    w = W.small(W.CONFIGS["llama8b"], n_layers=1, **getattr(W, preset))     # B = 16, Hkv = 8, g = 4, T = 16384
    cache, orc = _build(binding, w, [(0, 7), (15, 3)])
    _check(binding, w, cache, orc)


def test_qwen32b_32k_full_batch(binding):
    w = W.small(W.CONFIGS["qwen32b"], n_layers=1, **W.P24)                  # B = 64, Hkv = 8, g = 5, T = 32768, G = 128
    cache, orc = _build(binding, w, [(0, 0), (63, 7)])
    _check(binding, w, cache, orc)


def test_long_cot_stream_checkpoints(binding):
    # batch 4, prefill 8192, then the context grows; attention is checked at 8K, 32K, 64K and 128K cached tokens
    w = W.small(W.CONFIGS["longcot"], n_layers=1, **W.P24)
    streams = [(2, 1)]
    cache = U.make_cache(binding, w, max_tokens=w.tokens + 256)
    orc = {s: U.oracle_stream(w) for s in streams}
    t = 0
    for checkpoint in (8192, 32768, 65536, 131072):
        while t < checkpoint:
            # after the prefill the tokens arrive in ragged pieces, as a run of decode steps would leave them
            n = min(CHUNK if t < 8192 else 4096 - 37, checkpoint - t)
            k, v, q = W.tokens(w, 0, t, n, device="cuda")
            cache.quantize_append(0, k, v, q)
            for (b, hk), st in orc.items():
                st.append_many(U.f32(k[b, hk]), U.f32(v[b, hk]), U.f32(q[b, hk * w.g:(hk + 1) * w.g]))
            t += n
        qd = W.decode_query(w, 0, checkpoint, device="cuda")
        out = cache.decode_attention(0, qd, W.softmax_scale())
        err = U.max_abs_err(w, out, U.oracle_attention(w, orc, qd.cpu()))
        assert err <= ATTN_TOL, (checkpoint, err)
    U.compare_regions(cache, 0, w, orc)
    # the drifting outliers move the promoted set: more than one distinct channel list over the stream
    lists = {tuple(np.flatnonzero(b.tiers == O.TIER_BF16)) for b in orc[streams[0]].blocks}
    assert len(lists) > 4
    assert cache.status() == 0


def test_long_cot_streamed_decode_steps(binding):
    """The long chain-of-thought stream as it is produced: from 32K cached tokens, 2100 fused decode steps (one token
    per step through mixkvq_decode_step, 16 flushes with drifting outlier channels).  Two sampled streams follow on the
    CPU oracle token by token: attention at 16 seeded steps within the tolerance, all their bytes equal at the end."""
    w = W.small(W.CONFIGS["longcot"], n_layers=1, batch=2, tokens=32768, **W.P24)
    n_steps = 2100
    streams = [(0, 3), (1, 0)]
    cache = U.make_cache(binding, w, max_tokens=w.tokens + n_steps + 256)
    orc = {s: U.oracle_stream(w) for s in streams}
    t = 0
    while t < w.tokens:
        k, v, q = W.tokens(w, 0, t, CHUNK, device="cuda")
        cache.quantize_append(0, k, v, q)
        for (b, hk), st in orc.items():
            st.append_many(U.f32(k[b, hk]), U.f32(v[b, hk]), U.f32(q[b, hk * w.g:(hk + 1) * w.g]))
        t += CHUNK
    checked = set(np.random.default_rng(0x5EED).choice(n_steps, size=16, replace=False).tolist()) | {n_steps - 1}
    k, v, q = W.tokens(w, 0, w.tokens, n_steps, device="cuda")
    kc, vc, qc = U.f32(k), U.f32(v), U.f32(q)
    flushes0 = {s: st.n_flushes for s, st in orc.items()}
    scale = W.softmax_scale()
    worst = 0.0
    for i in range(n_steps):
        out = cache.decode_step(0, k[:, :, i:i + 1].contiguous(), v[:, :, i:i + 1].contiguous(), q[:, :, i:i + 1].contiguous(), scale)
        for (b, hk), st in orc.items():
            st.append(kc[b, hk, i], vc[b, hk, i], qc[b, hk * w.g:(hk + 1) * w.g, i])
        if i in checked:
            ref = {(b, hk): st.attention(qc[b, hk * w.g:(hk + 1) * w.g, i], scale) for (b, hk), st in orc.items()}
            worst = max(worst, U.max_abs_err(w, out, ref))
    assert worst <= ATTN_TOL, worst
    assert all(st.n_flushes - flushes0[s] >= 16 for s, st in orc.items())
    U.compare_regions(cache, 0, w, orc)
    assert cache.status() == 0
