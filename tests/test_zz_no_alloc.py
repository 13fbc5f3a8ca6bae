"""mixkvq_decode_attention_noalloc against mixkvq_decode_attention.

Some users of the library cannot allocate device memory: a plugin inside a serving engine whose memory pool
is sized once at start-up, or a host program whose language binding has no device allocator.  For them the
library offers one entry point that keeps the split partials of decode attention in a scratch array
compiled into the library.  This test calls it through the C ABI twice in a row (the second call on a
different, shorter cache, so stale partials of the first call are still lying in the array) and checks each
result against the ordinary entry point: both run the same kernels on the same grid, so the outputs must be equal
bit for bit (and within the attention tolerance of the other GPU tests, which follows).  It runs last so that a
failure here cannot hide another test's result.
"""
import ctypes as C

import pytest
import torch

import gpu_util as U
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


def _filled_cache(binding, name, batch, tokens, preset, layout=0):
    w = W.small(W.CONFIGS[name], n_layers=1, batch=batch, tokens=tokens, **preset)
    k, v, q = W.tokens(w, 0, 0, tokens)
    cache = U.make_cache(binding, w, layout=layout)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    return w, cache


def test_noalloc_entry_matches_workspace_entry_on_two_calls_in_a_row(binding):
    w1, c1 = _filled_cache(binding, "qwen7b", 3, 5 * 128 + 77, W.P27)
    w2, c2 = _filled_cache(binding, "llama8b", 2, 128 + 9, W.P24, layout=1)
    for step, (w, cache) in enumerate([(w1, c1), (w2, c2)]):
        qd = W.decode_query(w, 0, step).cuda()
        want = cache.decode_attention(0, qd, W.softmax_scale())
        out = torch.full(qd.shape, float("nan"), dtype=torch.float32, device="cuda")
        n_allocs = torch.cuda.memory_stats()["allocation.all.allocated"]
        got = cache.decode_attention_noalloc(0, qd, W.softmax_scale(), out=out)
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == n_allocs   # torch allocated nothing either
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert float((got - want).abs().max()) <= ATTN_TOL
        assert torch.equal(got, want)
        assert cache.status() == 0


def test_noalloc_entry_with_the_plain_alu_kernel(binding):
    # the comparison kernel lays its partials out differently in the same array
    w, cache = _filled_cache(binding, "qwen7b", 2, 3 * 128 + 50, W.P24)
    cache.set_attention_kernel(1)
    qd = W.decode_query(w, 0, 0).cuda()
    want = cache.decode_attention(0, qd, W.softmax_scale())
    got = cache.decode_attention_noalloc(0, qd, W.softmax_scale())
    assert torch.equal(got, want)
    assert cache.status() == 0


def test_noalloc_entry_rejects_more_streams_than_its_scratch_holds(binding):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=65, tokens=16)          # 65 * 4 = 260 streams > 256
    k, v, q = W.tokens(w, 0, 0, 16)
    cache = U.make_cache(binding, w, max_tokens=128)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    qd = W.decode_query(w, 0, 0).cuda()
    cache.decode_attention(0, qd, W.softmax_scale())                          # the ordinary entry point accepts it
    with pytest.raises(binding.MixKVQError) as e:
        cache.decode_attention_noalloc(0, qd, W.softmax_scale())
    assert e.value.code == -8
    assert "built-in scratch" in binding.status_string(-8)
    lib = binding.lib()
    assert lib.mixkvq_decode_attention_noalloc(None, 0, None, None, C.c_float(1.0), None) == -1
