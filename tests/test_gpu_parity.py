"""GPU parity: the CUDA path through the C ABI against the CPU oracle on the same seeded inputs.

Codes, packed bytes, selected channels and accumulator state must be bit-exact; attention outputs
within 2e-3 max-abs (the stated tolerance for fp32 outputs on bf16 inputs)."""
import dataclasses

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


def small(name="qwen7b", **kw):
    base = dict(n_layers=1, batch=2, tokens=300)
    base.update(kw)
    return W.small(W.CONFIGS[name], **base)


# ------------------------------------------------------------------------------------------ selection
@pytest.mark.parametrize("bits,preset", [(2, W.P27), (4, W.P4BASE)])
def test_select_channels_raw_bit_exact(binding, bits, preset):
    w = small(tokens=128, **{k: v for k, v in preset.items()})
    k, v, q = W.tokens(w, 0, 0, 128)
    tiers, sal = binding.select_channels_raw(q.cuda(), k.cuda(), bits, w.tau_bf16, w.tau_u4)
    for b in range(w.batch):
        for hk in range(w.n_kv_heads):
            acc, cnt = O.importance_from_queries(U.f32(q[b, hk * w.g:(hk + 1) * w.g]))
            _, _, A = O.salience(acc, cnt, U.f32(k[b, hk]), bits)
            assert np.array_equal(sal[b, hk].cpu().numpy(), A)                       # fp64, bit for bit
            assert np.array_equal(tiers[b, hk].cpu().numpy(), O.assign_tiers(A, w.tau_bf16, w.tau_u4))
    assert int((tiers == 2).sum()) >= 4 * w.batch * w.n_kv_heads - 4


def test_select_channels_of_current_window(binding):
    w = small(tokens=128 + 57, **W.P27)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    tiers, sal = cache.select_channels(0)
    orc = U.oracle_streams(w, 0, k, v, q)
    for (b, hk), st in orc.items():
        t, A = st.current_tiers()
        assert st.r == 57
        assert np.array_equal(tiers[b, hk].cpu().numpy(), t)
        assert np.array_equal(sal[b, hk].cpu().numpy(), A)


# --------------------------------------------------------------------------------- quantize + pack bytes
GEOMS = [(128, 32), (128, 128), (128, 64), (64, 32), (96, 32), (256, 64), (32, 32)]


TILE_GEOMS = [(128, 32, 1), (128, 64, 1), (128, 128, 1)]      # the optional tile layout exists for R = 128 only


@pytest.mark.parametrize("R,G,layout", [(r, g, 0) for r, g in GEOMS] + TILE_GEOMS)
@pytest.mark.parametrize("preset", ["P24", "P27", "P4BASE"])
def test_packed_cache_is_byte_exact(binding, R, G, layout, preset):
    w = small(tokens=2 * R + 41, residual_len=R, group_size=G, **getattr(W, preset))
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w, layout=layout)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    assert cache.status() == 0
    orc = U.oracle_streams(w, 0, k, v, q)
    U.compare_regions(cache, 0, w, orc)
    d = cache.describe(0)
    nb = (w.tokens - 1) // R
    assert (d.n_blocks, d.residual_tokens) == (nb, w.tokens - nb * R)
    if preset == "P27":
        assert any((b.tiers == O.TIER_U4).any() for st in orc.values() for b in st.blocks)
    if preset == "P4BASE":
        assert all(not (b.tiers == O.TIER_U2).any() for st in orc.values() for b in st.blocks)


@pytest.mark.parametrize("layout", [0, 1])
def test_tiny_config_full_parity(binding, layout):
    # configuration 1: 1 layer, batch 1, 1 KV head, 1 query head, 1024 cached tokens, then one decode step
    w = W.CONFIGS["tiny"]
    w = dataclasses.replace(w, **W.P27)
    k, v, q = W.tokens(w, 0, 0, 1025)
    cache = U.make_cache(binding, w, layout=layout)
    cache.quantize_append(0, k[:, :, :1024].cuda(), v[:, :, :1024].cuda(), q[:, :, :1024].cuda())
    orc = U.oracle_streams(w, 0, k[:, :, :1024], v[:, :, :1024], q[:, :, :1024])
    U.compare_regions(cache, 0, w, orc)
    assert cache.describe(0).n_blocks == 7 and cache.describe(0).residual_tokens == 128
    # the decode step: append (triggers the flush of block 8), then attention
    cache.quantize_append(0, k[:, :, 1024:].cuda().contiguous(), v[:, :, 1024:].cuda().contiguous(),
                          q[:, :, 1024:].cuda().contiguous())
    st = orc[(0, 0)]
    st.append(U.f32(k[0, 0, 1024]), U.f32(v[0, 0, 1024]), U.f32(q[0, :, 1024]))
    U.compare_regions(cache, 0, w, orc)
    qd = q[:, :, 1024].contiguous()
    ref = U.oracle_attention(w, orc, qd)
    for kind in (0, 1):
        cache.set_attention_kernel(kind)
        out = cache.decode_attention(0, qd.cuda(), W.softmax_scale())
        assert U.max_abs_err(w, out, ref) <= ATTN_TOL, kind
    assert cache.status() == 0


@pytest.mark.parametrize("mode", [0, 1])
def test_streamed_appends_equal_bulk(binding, mode):
    # window importance and cumulative importance (whose bulk path carries the running sums across the windows)
    w = small(batch=1, tokens=(128 + 70) if mode == 0 else (3 * 128 + 70), **W.P27)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    kc, vc, qc = k.cuda(), v.cuda(), q.cuda()
    bulk = U.make_cache(binding, w, importance_mode=mode)
    bulk.quantize_append(0, kc, vc, qc)
    one = U.make_cache(binding, w, importance_mode=mode)
    for t in range(w.tokens):
        one.quantize_append(0, kc[:, :, t:t + 1].contiguous(), vc[:, :, t:t + 1].contiguous(),
                            qc[:, :, t:t + 1].contiguous())
    # in two ragged pieces as well
    two = U.make_cache(binding, w, importance_mode=mode)
    two.quantize_append(0, kc[:, :, :93].contiguous(), vc[:, :, :93].contiguous(), qc[:, :, :93].contiguous())
    two.quantize_append(0, kc[:, :, 93:].contiguous(), vc[:, :, 93:].contiguous(), qc[:, :, 93:].contiguous())
    for s in range(w.n_kv_heads):
        a, b, c = bulk.stream_regions(0, s), one.stream_regions(0, s), two.stream_regions(0, s)
        r = bulk.describe(0).residual_tokens
        for key in ("table", "base", "extras", "state", "resK", "resV"):
            assert a[key] == b[key] == c[key], key
    U.compare_regions(bulk, 0, w, U.oracle_streams(w, 0, k, v, q, importance_mode=mode))


@pytest.mark.parametrize("mode", [1, 2])
def test_other_importance_modes(binding, mode):
    # 1: cumulative |q| accumulator (Appendix D.2); 2: error-only ablation, A = S (Appendix E)
    w = small(batch=1, tokens=2 * 128 + 9, **W.P27)
    if mode == 2:
        w = dataclasses.replace(w, tau_bf16=12.0, tau_u4=1.8)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w, importance_mode=mode)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    orc = U.oracle_streams(w, 0, k, v, q, importance_mode=mode)
    U.compare_regions(cache, 0, w, orc)
    tiers, sal = cache.select_channels(0)
    for (b, hk), st in orc.items():
        t, A = st.current_tiers()
        assert np.array_equal(tiers[b, hk].cpu().numpy(), t) and np.array_equal(sal[b, hk].cpu().numpy(), A)
    assert len({int(x) for st in orc.values() for blk in st.blocks for x in blk.tiers}) == 3


def test_rounding_ties_are_bit_exact(binding):
    # keys and values on a grid of half-steps of their scale: every group spans 0 .. 3 (2-bit scale exactly 1, a
    # second stream 0 .. 3 * 0.75 with a scale that is not a power of two), so (x - z) / s falls on exact half-integers
    # for about half of the elements; the codes must follow round-half-even of the IEEE quotient like the oracle's
    w = small("qwen7b", batch=2, tokens=4 * 128 + 40, **W.P24)
    gen = torch.Generator().manual_seed(1234)
    shape = (w.batch, w.n_kv_heads, w.tokens, 128)
    k = torch.randint(0, 7, shape, generator=gen).float() * 0.5
    v = torch.randint(0, 7, shape, generator=gen).float() * 0.5
    k[:, :, 0::32] = 0.0; k[:, :, 1::32] = 3.0          # every 32-token key group holds its extremes
    v[..., 0::32] = 0.0; v[..., 1::32] = 3.0            # every 32-channel value group too
    k[1] *= 0.75; v[1] *= 0.75
    k, v = k.to(torch.bfloat16), v.to(torch.bfloat16)
    _, _, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    orc = U.oracle_streams(w, 0, k, v, q)
    U.compare_regions(cache, 0, w, orc)
    codes = np.concatenate([blk.kcodes.ravel() for st in orc.values() for blk in st.blocks] +
                           [blk.vcodes.ravel() for st in orc.values() for blk in st.blocks])
    assert set(np.unique(codes)) == {0, 1, 2, 3}
    assert cache.status() == 0


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("k16,k4", [(4, 0), (3, 24), (0, 9)])
def test_fixed_budget_tiering(binding, layout, k16, k4):
    # the top k16 channels by salience in BF16, the next k4 in UINT4, whatever the thresholds say: constant tier counts per
    # block, bytes and scores equal to the oracle's, attention within tolerance
    w = small("qwen7b", batch=2, tokens=5 * 128 + 33, **W.P24)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w, layout=layout, budget_bf16=k16, budget_u4=k4)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    orc = U.oracle_streams(w, 0, k, v, q, budget_bf16=k16, budget_u4=k4)
    U.compare_regions(cache, 0, w, orc)
    tiers, sal = cache.select_channels(0)
    for (b, hk), st in orc.items():
        t, A = st.current_tiers()
        assert np.array_equal(tiers[b, hk].cpu().numpy(), t) and np.array_equal(sal[b, hk].cpu().numpy(), A)
        assert all(int((blk.tiers == O.TIER_BF16).sum()) == k16 and int((blk.tiers == O.TIER_U4).sum()) == k4
                   for blk in st.blocks)
    qd = W.decode_query(w, 0, 0)
    out = cache.decode_attention(0, qd.cuda(), W.softmax_scale())
    assert U.max_abs_err(w, out, U.oracle_attention(w, orc, qd)) <= ATTN_TOL
    assert cache.status() == 0


@pytest.mark.parametrize("kind,layout", [(0, 0), (1, 0), (0, 1)])
@pytest.mark.parametrize("tokens", [20, 37, 32 + 2 * 128 + 17])
def test_sink_tokens(binding, kind, layout, tokens):
    # the first 32 tokens stay in bf16 outside the residual window, the scoring and the blocks; attention sees them
    w = small("qwen7b", batch=2, tokens=tokens, **W.P27)
    k, v, q = W.tokens(w, 0, 0, tokens)
    cache = U.make_cache(binding, w, layout=layout, sink_len=32)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    cache.set_attention_kernel(kind)
    orc = U.oracle_streams(w, 0, k, v, q, sink_len=32)
    U.compare_regions(cache, 0, w, orc)
    d = cache.describe(0)
    assert d.sink_tokens == min(tokens, 32) and d.n_blocks * 128 + d.residual_tokens == max(tokens - 32, 0)
    qd = W.decode_query(w, 0, 0)
    out = cache.decode_attention(0, qd.cuda(), W.softmax_scale())
    assert U.max_abs_err(w, out, U.oracle_attention(w, orc, qd)) <= ATTN_TOL
    assert cache.status() == 0


@pytest.mark.parametrize("kind", [0, 1])
def test_decode_steps_through_the_sink(binding, kind):
    # decode steps from a short prompt: the sink fills first (plain append + attention), then the fused step takes over
    w = small("qwen7b", batch=1, tokens=10 + 60, **W.P24)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    kc, vc, qc = k.cuda(), v.cuda(), q.cuda()
    cache = U.make_cache(binding, w, sink_len=32)
    cache.set_attention_kernel(kind)
    cache.quantize_append(0, kc[:, :, :10].contiguous(), vc[:, :, :10].contiguous(), qc[:, :, :10].contiguous())
    orc = U.oracle_streams(w, 0, k[:, :, :10], v[:, :, :10], q[:, :, :10], sink_len=32)
    for t in range(10, w.tokens):
        out = cache.decode_step(0, kc[:, :, t:t + 1].contiguous(), vc[:, :, t:t + 1].contiguous(),
                                qc[:, :, t:t + 1].contiguous(), W.softmax_scale())
        for (b, hk), st in orc.items():
            st.append(U.f32(k[b, hk, t]), U.f32(v[b, hk, t]), U.f32(q[b, hk * w.g:(hk + 1) * w.g, t]))
        if t in (10, 31, 32, 33, 69):
            qd = q[:, :, t]
            assert U.max_abs_err(w, out, U.oracle_attention(w, orc, qd)) <= ATTN_TOL, t
    U.compare_regions(cache, 0, w, orc)
    assert cache.status() == 0


@pytest.mark.parametrize("kind", [0, 1])
@pytest.mark.parametrize("R,G,preset", [(128, 32, "P24"), (128, 32, "P27"), (64, 64, "P24"), (128, 128, "P4BASE"), (256, 32, "P24")])
def test_four_bit_values(binding, kind, R, G, preset):
    # values at 4 bits per token group: two 2-bit planes per unit, bytes equal to the oracle's, attention within tolerance,
    # and a few fused decode steps on top (one of them flushes a window when R = 64)
    w = small("llama8b", batch=2, tokens=2 * R + 61, residual_len=R, group_size=G, **getattr(W, preset))
    k, v, q = W.tokens(w, 0, 0, w.tokens + 6)
    kc, vc, qc = k.cuda(), v.cuda(), q.cuda()
    budget = 16 * 8192 if preset == "P4BASE" else 0
    cache = U.make_cache(binding, w, v_bits=4, extras_budget_bytes=budget)
    n = w.tokens
    cache.quantize_append(0, kc[:, :, :n].contiguous(), vc[:, :, :n].contiguous(), qc[:, :, :n].contiguous())
    cache.set_attention_kernel(kind)
    orc = U.oracle_streams(w, 0, k[:, :, :n], v[:, :, :n], q[:, :, :n], v_bits=4)
    U.compare_regions(cache, 0, w, orc)
    qd = W.decode_query(w, 0, 0)
    out = cache.decode_attention(0, qd.cuda(), W.softmax_scale())
    assert U.max_abs_err(w, out, U.oracle_attention(w, orc, qd)) <= ATTN_TOL
    for t in range(n, n + 6):
        out = cache.decode_step(0, kc[:, :, t:t + 1].contiguous(), vc[:, :, t:t + 1].contiguous(),
                                qc[:, :, t:t + 1].contiguous(), W.softmax_scale())
        for (b, hk), st in orc.items():
            st.append(U.f32(k[b, hk, t]), U.f32(v[b, hk, t]), U.f32(q[b, hk * w.g:(hk + 1) * w.g, t]))
    assert U.max_abs_err(w, out, U.oracle_attention(w, orc, q[:, :, n + 5])) <= ATTN_TOL
    U.compare_regions(cache, 0, w, orc)
    assert cache.status() == 0


def test_four_bit_values_need_the_fragment_layout(binding):
    cfg = binding.make_config(1, 1, 4, 1, 1024, block_layout=1, v_bits=4)
    with pytest.raises(binding.MixKVQError):
        binding.cache_bytes(cfg)


def test_stream_order_around_the_early_started_kernels(binding):
    # the attention and combine kernels may start before their predecessor in the stream has finished and wait for it on
    # the device: a query rewritten by an ordinary kernel right before the call, and an output copied right after it,
    # must behave as in plain stream order, call after call without host synchronization
    w = small("qwen7b", batch=2, tokens=6 * 128 + 50, **W.P24)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    queries = [W.decode_query(w, 0, i).cuda() for i in range(6)]
    want = [cache.decode_attention(0, qi, W.softmax_scale()).clone() for qi in queries]
    torch.cuda.synchronize()
    q_dev = torch.empty_like(queries[0])
    out = torch.empty_like(want[0])
    got = []
    for rep in range(3):
        for qi in queries:
            q_dev.copy_(qi)                                   # ordinary kernel writes the input
            cache.decode_attention(0, q_dev, W.softmax_scale(), out=out)
            got.append(out.clone())                           # ordinary kernel reads the output
    torch.cuda.synchronize()
    for i, g in enumerate(got):
        assert torch.equal(g, want[i % len(queries)]), i
    assert cache.status() == 0


# ------------------------------------------------------------------------------------------- attention
@pytest.mark.parametrize("kind,layout", [(0, 0), (1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("name,tokens,preset", [
    ("qwen7b", 1, "P24"), ("qwen7b", 31, "P24"), ("qwen7b", 128, "P24"), ("qwen7b", 129, "P24"),
    ("qwen7b", 1153, "P27"), ("llama8b", 700, "P27"), ("llama8b", 700, "P4BASE"), ("qwen32b", 1000, "P24"),
    ("tiny", 2500, "P27"),
])
def test_attention_matches_oracle(binding, kind, layout, name, tokens, preset):
    w = small(name, batch=2 if name != "tiny" else 1, tokens=tokens, **getattr(W, preset))
    k, v, q = W.tokens(w, 0, 0, tokens)
    cache = U.make_cache(binding, w, layout=layout)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    cache.set_attention_kernel(kind)
    orc = U.oracle_streams(w, 0, k, v, q)
    for step in range(2):
        qd = W.decode_query(w, 0, step)
        out = cache.decode_attention(0, qd.cuda(), W.softmax_scale())
        err = U.max_abs_err(w, out, U.oracle_attention(w, orc, qd))
        assert err <= ATTN_TOL, (err, step)
    assert cache.status() == 0


@pytest.mark.parametrize("kind", [0, 1])
def test_attention_large_magnitudes(binding, kind):
    # values 64 times larger (stored value scales around 170: inside the documented fp16 operand range of the default
    # kernel, s_v * 2^7 < 65504) and queries 4 times larger (logits of several tens, sharply peaked softmax rows, so the
    # reference maximum of the online softmax jumps by more than its slack); the error bound scales with the values
    # (the salience is linear in |q|: the threshold moves with it, so the tier mix stays that of the preset)
    w = small("qwen7b", batch=2, tokens=9 * 128 + 77, **{**W.P24, "tau_bf16": 4.0 * W.P24["tau_bf16"]})
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    v = (v.float() * 64.0).to(torch.bfloat16)
    q = (q.float() * 4.0).to(torch.bfloat16)
    cache = U.make_cache(binding, w)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    cache.set_attention_kernel(kind)
    orc = U.oracle_streams(w, 0, k, v, q)
    U.compare_regions(cache, 0, w, orc)
    for step in range(2):
        qd = (W.decode_query(w, 0, step).float() * 4.0).to(torch.bfloat16)
        out = cache.decode_attention(0, qd.cuda(), W.softmax_scale())
        assert torch.isfinite(out).all()
        err = U.max_abs_err(w, out, U.oracle_attention(w, orc, qd))
        assert err <= 64.0 * ATTN_TOL, (err, step)
    assert cache.status() == 0


@pytest.mark.parametrize("kind", [0, 1])
@pytest.mark.parametrize("R,G,layout", [(128, 128, 0), (64, 32, 0), (256, 64, 0), (32, 32, 0), (96, 32, 0), (128, 128, 1),
                                        (128, 64, 1)])
def test_attention_other_geometries(binding, kind, R, G, layout):
    w = small("llama8b", batch=1, tokens=3 * R + 17, residual_len=R, group_size=G, **W.P27)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w, layout=layout)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    cache.set_attention_kernel(kind)
    orc = U.oracle_streams(w, 0, k, v, q)
    qd = W.decode_query(w, 0, 0)
    out = cache.decode_attention(0, qd.cuda(), W.softmax_scale())
    assert U.max_abs_err(w, out, U.oracle_attention(w, orc, qd)) <= ATTN_TOL


def test_layers_are_independent(binding):
    w = small(n_layers=3, batch=1, tokens=200, **W.P27)
    cache = U.make_cache(binding, w)
    data = [W.tokens(w, l, 0, 150 + 20 * l) for l in range(3)]
    for l in (2, 0, 1):
        k, v, q = data[l]
        cache.quantize_append(l, k.cuda(), v.cuda(), q.cuda())
    for l in range(3):
        k, v, q = data[l]
        orc = U.oracle_streams(w, l, k, v, q)
        U.compare_regions(cache, l, w, orc)
        qd = W.decode_query(w, l, 0)
        out = cache.decode_attention(l, qd.cuda(), W.softmax_scale())
        assert U.max_abs_err(w, out, U.oracle_attention(w, orc, qd)) <= ATTN_TOL


# ------------------------------------------------------------------------------------- errors and status
def test_capacity_and_empty_errors(binding):
    w = small(batch=1, tokens=100)
    cache = U.make_cache(binding, w, max_tokens=128)
    qd = W.decode_query(w, 0, 0).cuda()
    with pytest.raises(binding.MixKVQError) as e:
        cache.decode_attention(0, qd, 1.0)
    assert e.value.code == -7
    k, v, q = W.tokens(w, 0, 0, 129)
    with pytest.raises(binding.MixKVQError) as e:
        cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    assert e.value.code == -5
    assert cache.describe(0).residual_tokens == 0
    with pytest.raises(binding.MixKVQError) as e:         # misaligned device pointer
        cache.quantize_append(0, k.cuda().view(-1)[1:1 + 128 * 4].view(1, 4, 1, 128), v.cuda()[:, :, :1].contiguous(),
                              q.cuda()[:, :, :1].contiguous())
    assert e.value.code == -3


def test_extras_arena_exhaustion_sets_status(binding):
    w = small(batch=1, tokens=3 * 128 + 1, **W.P27)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w, extras_budget_bytes=2048)     # room for about one block's promoted channels
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    assert cache.status() & binding.DEV_EXTRAS_FULL
    # the stated behaviour: blocks that fitted equal the oracle's; a block that did not fit has a table entry without
    # promoted channels, nothing of it in the arena, and its base part written as usual
    oracle = U.oracle_streams(w, 0, k, v, q)
    st = oracle[(0, 0)]
    got = cache.stream_regions(0, 0)
    want = O.pack_stream(st)
    assert got["base"] == want["base"]
    fitted = 0
    for i in range(len(st.blocks)):
        entry = got["table"][8 * i:8 * i + 8]
        if entry == want["table"][8 * i:8 * i + 8] and fitted == i:
            fitted += 1
        else:
            assert entry[4] == 0 and entry[5] == 0                 # n16 = n4 = 0
    assert 1 <= fitted < len(st.blocks)
    used = 16 * int.from_bytes(got["state"][1028:1032], "little")      # the arena holds the fitted blocks only
    assert 0 < used <= 2048 and used < len(want["extras"])
    assert got["extras"] == want["extras"][:used]
    cache.reset()
    assert cache.status() == 0 and cache.describe(0).n_blocks == 0


# ------------------------------------------------------------------------------- degenerate cases of the method
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("kind", [0, 1])
def test_all_channels_promoted_is_unquantized_key_attention(binding, kind, layout):
    # every key channel in the BF16 tier: the logits are those of the raw bf16 keys (library attention on the
    # oracle's dequantized values), and the promoted-channel store carries all 128 channels of every block
    w = small("llama8b", batch=1, tokens=2 * 128 + 30, tau_bf16=-1.0, tau_u4=-1.0)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    cache = U.make_cache(binding, w, extras_budget_bytes=4 * 40000, layout=layout)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    cache.set_attention_kernel(kind)
    orc = U.oracle_streams(w, 0, k, v, q)
    U.compare_regions(cache, 0, w, orc)
    qd = W.decode_query(w, 0, 0)
    out = cache.decode_attention(0, qd.cuda(), W.softmax_scale()).cpu()
    assert cache.status() == 0
    for (b, hk), st in orc.items():
        assert all((blk.tiers == O.TIER_BF16).all() for blk in st.blocks)
        ref = torch.nn.functional.scaled_dot_product_attention(
            qd[b, hk * w.g:(hk + 1) * w.g].double()[None], k[b, hk].double()[None], torch.from_numpy(st.values())[None],
            scale=W.softmax_scale())[0]
        assert float((out[b, hk * w.g:(hk + 1) * w.g].double() - ref).abs().max()) <= ATTN_TOL


@pytest.mark.parametrize("layout", [0, 1])
def test_zero_keys_and_constant_groups(binding, layout):
    # all keys zero: every scale is 0 (codes 0, dequantized exactly) and the output is the mean of the values;
    # values constant inside each group of channels: their scale is 0 and the zero-point carries them exactly
    w = small("qwen7b", batch=1, tokens=3 * 128 + 5, **W.P27)
    k, v, q = W.tokens(w, 0, 0, w.tokens)
    k = torch.zeros_like(k)
    v = v[..., ::32].repeat_interleave(32, dim=-1).contiguous()
    cache = U.make_cache(binding, w, layout=layout)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    orc = U.oracle_streams(w, 0, k, v, q)
    U.compare_regions(cache, 0, w, orc)
    qd = W.decode_query(w, 0, 0)
    out = cache.decode_attention(0, qd.cuda(), W.softmax_scale()).cpu()
    mean_v = v.float().mean(dim=2)                                           # [B, Hkv, 128]
    for hk in range(w.n_kv_heads):
        got = out[0, hk * w.g:(hk + 1) * w.g]
        assert float((got - mean_v[0, hk][None]).abs().max()) <= 1e-4
    assert cache.status() == 0


# ------------------------------------------------------------------------------------------- fused decode step
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("kind", [0, 1])
def test_decode_step_equals_append_then_attention(binding, kind, layout):
    # 40 decode steps across a flush (the window fills at step 14): the fused entry point must leave the same bytes
    # and give the same outputs as quantize_append(1) + decode_attention, and both must match the oracle
    w = small("qwen7b", batch=2, tokens=2 * 128 + 114, **W.P27)
    steps = 40
    k, v, q = W.tokens(w, 0, 0, w.tokens + steps)
    kc, vc, qc = k.cuda(), v.cuda(), q.cuda()
    fused = U.make_cache(binding, w, max_tokens=w.tokens + steps + 8, layout=layout)
    plain = U.make_cache(binding, w, max_tokens=w.tokens + steps + 8, layout=layout)
    for c in (fused, plain):
        c.quantize_append(0, kc[:, :, :w.tokens].contiguous(), vc[:, :, :w.tokens].contiguous(), qc[:, :, :w.tokens].contiguous())
        c.set_attention_kernel(kind)
    orc = U.oracle_streams(w, 0, k[:, :, :w.tokens], v[:, :, :w.tokens], q[:, :, :w.tokens])
    for i in range(steps):
        t = w.tokens + i
        ks, vs, qs = (x[:, :, t:t + 1].contiguous() for x in (kc, vc, qc))
        out_f = fused.decode_step(0, ks, vs, qs, W.softmax_scale())
        plain.quantize_append(0, ks, vs, qs)
        out_p = plain.decode_attention(0, qs.view(w.batch, w.n_q_heads, 128), W.softmax_scale())
        assert float((out_f - out_p).abs().max()) <= 1e-6, i
        for (b, hk), st in orc.items():
            st.append(U.f32(k[b, hk, t]), U.f32(v[b, hk, t]), U.f32(q[b, hk * w.g:(hk + 1) * w.g, t]))
        if i in (0, 13, 14, 15, steps - 1):
            ref = U.oracle_attention(w, orc, q[:, :, t].contiguous())
            assert U.max_abs_err(w, out_f, ref) <= ATTN_TOL, i
    U.compare_regions(fused, 0, w, orc)
    U.compare_regions(plain, 0, w, orc)
    assert fused.status() == 0 and fused.describe(0).residual_tokens == plain.describe(0).residual_tokens


# --------------------------------------------------------------------------- guard bands around caller memory
@pytest.mark.parametrize("layout", [0, 1])
def test_no_write_outside_the_callers_buffers(binding, layout):
    # cache memory, workspace and output are carved out of larger tensors filled with a pattern; after a bulk append,
    # streamed steps across a flush and attention on both kernels, the bytes around them are untouched
    import ctypes as C
    w = small("qwen7b", batch=2, tokens=3 * 128 + 120, **W.P27)
    steps = 12
    cfg = binding.make_config(1, w.batch, w.n_q_heads, w.n_kv_heads, w.tokens + steps + 4, tau_bf16=w.tau_bf16,
                              tau_u4=w.tau_u4, block_layout=layout)
    nbytes, ws_bytes = binding.cache_bytes(cfg)
    pad = 4096
    def guarded(n):
        t = torch.full((n + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
        return t, t[pad:pad + n]
    mem_all, mem = guarded(nbytes)
    ws_all, ws = guarded(ws_bytes)
    out_all, out_b = guarded(w.batch * w.n_q_heads * 128 * 4)
    out = out_b.view(torch.float32).view(w.batch, w.n_q_heads, 128)
    assert mem.data_ptr() % 256 == 0 and ws.data_ptr() % 16 == 0
    lib, handle = binding.lib(), C.c_void_p()
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert lib.mixkvq_cache_init(C.byref(cfg), C.c_void_p(mem.data_ptr()), nbytes, stream, C.byref(handle)) == 0
    k, v, q = (x.cuda() for x in W.tokens(w, 0, 0, w.tokens + steps))
    p = lambda t: C.c_void_p(t.data_ptr())
    first = [x[:, :, :w.tokens].contiguous() for x in (k, v, q)]
    assert lib.mixkvq_quantize_append(handle, 0, p(first[0]), p(first[1]), p(first[2]), w.tokens, stream) == 0
    for i in range(steps):
        t = w.tokens + i
        ks, vs, qs = (x[:, :, t:t + 1].contiguous() for x in (k, v, q))
        assert lib.mixkvq_decode_step(handle, 0, p(ks), p(vs), p(qs), p(out), C.c_float(W.softmax_scale()), p(ws), ws_bytes,
                                      stream) == 0
    for kind in (1, 0):
        assert lib.mixkvq_set_attention_kernel(handle, kind) == 0
        qd = q[:, :, -1].contiguous()
        assert lib.mixkvq_decode_attention(handle, 0, p(qd), p(out), C.c_float(W.softmax_scale()), p(ws), ws_bytes, stream) == 0
    status = C.c_int(-1)
    assert lib.mixkvq_query_status(handle, C.byref(status), stream) == 0 and status.value == 0
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
    for whole, n in ((mem_all, nbytes), (ws_all, ws_bytes), (out_all, out_b.numel())):
        assert bool((whole[:pad] == 0xA5).all()) and bool((whole[pad + n:] == 0xA5).all())
    lib.mixkvq_cache_destroy(handle)
