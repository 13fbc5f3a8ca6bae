"""GPU parity of ragged batches: sequences of one batch hold different numbers of tokens.  Every sequence's streams
must hold the bytes a batch-1 oracle stream holds after the same tokens, and decode attention must match the oracle's
per-stream attention; a sequence without tokens gets zeros."""
import numpy as np
import pytest
import torch

import gpu_util as U
from oracle import mixkvq_oracle as O
from paper_2512_19206_b200 import workloads as W

pytestmark = pytest.mark.gpu
ATTN_TOL = 2e-3


@pytest.fixture(scope="module")
def binding():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19206_b200 import build
    build.build()
    from paper_2512_19206_b200 import binding as b
    b.lib()
    return b


def feed(cache, oracle, w, layer, k, v, q, counts):
    """One ragged append of the first counts[b] tokens of sequence b, to the device cache and to the oracle streams."""
    cache.quantize_append_ragged(layer, k.cuda(), v.cuda(), q.cuda(), counts)
    kf, vf, qf = U.f32(k), U.f32(v), U.f32(q)
    for (b, hk), st in oracle.items():
        if counts[b]:
            st.append_many(kf[b, hk, :counts[b]], vf[b, hk, :counts[b]], qf[b, hk * w.g:(hk + 1) * w.g, :counts[b]])


def check_attention(cache, oracle, w, layer, seed_t, lengths):
    qd = W.decode_query(w, layer, seed_t)
    out = cache.decode_attention(layer, qd.cuda(), W.softmax_scale()).cpu().numpy()
    qf = U.f32(qd)
    for (b, hk), st in oracle.items():
        got = out[b, hk * w.g:(hk + 1) * w.g]
        if lengths[b] == 0:
            assert not got.any()
        else:
            ref = st.attention(qf[b, hk * w.g:(hk + 1) * w.g], W.softmax_scale())
            assert float(np.abs(got - ref).max()) <= ATTN_TOL, (b, hk)


@pytest.mark.parametrize("preset,kwargs", [("P27", {}), ("P24", {"sink_len": 32}), ("P4BASE", {"importance_mode": 1})])
def test_ragged_appends_and_attention(binding, preset, kwargs):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=5, tokens=1024, **getattr(W, preset))
    R = w.residual_len
    cache = U.make_cache(binding, w, max_tokens=1200, **kwargs)
    oracle = {(b, hk): U.oracle_stream(w, **kwargs) for b in range(w.batch) for hk in range(w.n_kv_heads)}
    lengths = [0] * w.batch
    sink = kwargs.get("sink_len", 0)
    # lengths differ by several blocks; sequence 0 stays empty; sequence 1 ends exactly on a full window
    for step, counts in enumerate([[0, 200 + sink, 500, 37, 500], [0, 2 * R - 200, 317, 0, 317], [0, 0, 1, 1, 1]]):
        k, v, q = W.tokens(w, 0, 1000 * step, max(counts))
        feed(cache, oracle, w, 0, k, v, q, counts)
        lengths = [a + c for a, c in zip(lengths, counts)]
        for b in range(w.batch):
            nb, r, ns = cache.sequence_fill(0, b)
            assert ns + nb * R + r == lengths[b]
        U.compare_regions(cache, 0, w, oracle)
        check_attention(cache, oracle, w, 0, 7 + step, lengths)
    assert cache.sequence_fill(0, 1) == (1, R, sink)          # full window, not flushed yet (lazy)
    assert cache.status() == 0
    # a fused decode step for all sequences (the empty one gets its first token, the full window is flushed first)
    k, v, q = W.tokens(w, 0, 5000, 1)
    out = cache.decode_step(0, k.cuda(), v.cuda(), q.cuda(), W.softmax_scale()).cpu().numpy()
    kf, vf, qf = U.f32(k), U.f32(v), U.f32(q)
    for (b, hk), st in oracle.items():
        st.append(kf[b, hk, 0], vf[b, hk, 0], qf[b, hk * w.g:(hk + 1) * w.g, 0])
        ref = st.attention(qf[b, hk * w.g:(hk + 1) * w.g, 0], W.softmax_scale())
        assert float(np.abs(out[b, hk * w.g:(hk + 1) * w.g] - ref).max()) <= ATTN_TOL, (b, hk)
    U.compare_regions(cache, 0, w, oracle)
    # channel selection on the ragged windows
    tiers, sal = cache.select_channels(0)
    for (b, hk), st in oracle.items():
        if st.r == 0:                  # an empty window has no scores: the call leaves these rows alone
            continue
        t_ref, a_ref = st.current_tiers()
        assert np.array_equal(tiers[b, hk].cpu().numpy(), t_ref)
        assert np.array_equal(sal[b, hk].cpu().numpy(), a_ref)


def test_ragged_decode_steps_flush_each_sequence_at_its_own_step(binding):
    """140 fused decode steps on a batch whose windows fill up at different steps: every step is one attention launch,
    a step in which some windows are full adds ONE flush launch for those sequences only."""
    w = W.small(W.CONFIGS["llama8b"], n_layers=1, batch=4, tokens=1024, **W.P27)
    R = w.residual_len
    cache = U.make_cache(binding, w, max_tokens=1024)
    oracle = {(b, hk): U.oracle_stream(w) for b in range(w.batch) for hk in (0, w.n_kv_heads - 1)}
    k, v, q = W.tokens(w, 0, 0, 300)
    feed(cache, oracle, w, 0, k, v, q, [300, 120, 7, 0])
    flush_steps = 0
    for step in range(140):
        k, v, q = W.tokens(w, 0, 2000 + step, 1)
        n0 = cache.launch_count()
        due = any(cache.sequence_fill(0, b)[1] == R for b in range(w.batch))
        out = cache.decode_step(0, k.cuda(), v.cuda(), q.cuda(), W.softmax_scale())
        # table + split + merge, and table + flush before them when a window is full
        assert cache.launch_count() - n0 == (5 if due else 3)
        flush_steps += due
        kf, vf, qf = U.f32(k), U.f32(v), U.f32(q)
        for (b, hk), st in oracle.items():
            st.append(kf[b, hk, 0], vf[b, hk, 0], qf[b, hk * w.g:(hk + 1) * w.g, 0])
        if step % 35 == 34 or due:
            o = out.cpu().numpy()
            for (b, hk), st in oracle.items():
                ref = st.attention(qf[b, hk * w.g:(hk + 1) * w.g, 0], W.softmax_scale())
                assert float(np.abs(o[b, hk * w.g:(hk + 1) * w.g] - ref).max()) <= ATTN_TOL, (step, b, hk)
    assert flush_steps >= 4                       # the four sequences reach a full window at four different steps
    U.compare_regions(cache, 0, w, oracle)
    assert cache.status() == 0


@pytest.mark.parametrize("R,G,v_bits", [(256, 128, 2), (64, 64, 4), (128, 32, 4)])
def test_ragged_other_geometries(binding, R, G, v_bits):
    """Ragged appends, decode steps and attention with other window and group sizes and with 4-bit values."""
    w = W.small(W.CONFIGS["llama8b"], n_layers=1, batch=3, tokens=1024, residual_len=R, group_size=G, **W.P24)
    cache = U.make_cache(binding, w, max_tokens=1100, v_bits=v_bits)
    oracle = {(b, hk): U.oracle_stream(w, v_bits=v_bits) for b in range(w.batch) for hk in (0, w.n_kv_heads - 1)}
    k, v, q = W.tokens(w, 0, 0, 900)
    feed(cache, oracle, w, 0, k, v, q, [900, 2 * R, 33])
    lengths = [900, 2 * R, 33]
    U.compare_regions(cache, 0, w, oracle)
    check_attention(cache, oracle, w, 0, 3, lengths)
    for step in range(3):
        k, v, q = W.tokens(w, 0, 3000 + step, 1)
        out = cache.decode_step(0, k.cuda(), v.cuda(), q.cuda(), W.softmax_scale()).cpu().numpy()
        kf, vf, qf = U.f32(k), U.f32(v), U.f32(q)
        for (b, hk), st in oracle.items():
            st.append(kf[b, hk, 0], vf[b, hk, 0], qf[b, hk * w.g:(hk + 1) * w.g, 0])
            ref = st.attention(qf[b, hk * w.g:(hk + 1) * w.g, 0], W.softmax_scale())
            assert float(np.abs(out[b, hk * w.g:(hk + 1) * w.g] - ref).max()) <= ATTN_TOL, (step, b, hk)
    U.compare_regions(cache, 0, w, oracle)
    assert cache.status() == 0


def test_equal_counts_are_one_run(binding):
    """A ragged call with equal counts on a uniform batch launches what the plain append launches."""
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=3, tokens=400, **W.P27)
    k, v, q = W.tokens(w, 0, 0, 300)
    a, b = U.make_cache(binding, w), U.make_cache(binding, w)
    n0 = a.launch_count()
    a.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    na = a.launch_count() - n0
    n0 = b.launch_count()
    b.quantize_append_ragged(0, k.cuda(), v.cuda(), q.cuda(), [300, 300, 300])
    assert b.launch_count() - n0 == na
    for s in range(w.batch * w.n_kv_heads):
        assert a.stream_regions(0, s) == b.stream_regions(0, s)


def test_ragged_argument_checks(binding):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=2, tokens=300, **W.P27)
    k, v, q = W.tokens(w, 0, 0, 100)
    cache = U.make_cache(binding, w, max_tokens=150)
    with pytest.raises(binding.MixKVQError):
        cache.quantize_append_ragged(0, k.cuda(), v.cuda(), q.cuda(), [101, 5])      # more than the tensors hold
    with pytest.raises(binding.MixKVQError):
        cache.quantize_append_ragged(0, k.cuda(), v.cuda(), q.cuda(), [-1, 5])
    cache.quantize_append_ragged(0, k.cuda(), v.cuda(), q.cuda(), [100, 20])
    with pytest.raises(binding.MixKVQError):                                          # sequence 0 would exceed max_tokens;
        cache.quantize_append_ragged(0, k.cuda(), v.cuda(), q.cuda(), [60, 1])       # nothing is appended to sequence 1 either
    assert cache.sequence_fill(0, 0) == (0, 100, 0) and cache.sequence_fill(0, 1) == (0, 20, 0)
