"""GPU tests of the decode-attention kernel's behaviour off the happy path: a bounded wait that runs out, and the early
request of packed blocks ahead of the stream-order wait."""
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


def _filled(binding, tokens=5 * 128 + 40, **kw):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=2, tokens=tokens, **W.P27)
    k, v, q = W.tokens(w, 0, 0, tokens)
    cache = U.make_cache(binding, w, **kw)
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    return w, cache, (k, v, q)


def test_a_wait_that_runs_out_returns_with_the_status_bit(binding):
    """The barrier of every pair's first staged copy is armed for 16 bytes more than the copy delivers (the test hook
    of the C ABI), so no wait on it can succeed: every wait gives up after 64 polls, the call returns, the status word
    says so and the output is zero.  After a reset the same cache works again."""
    w, cache, (k, v, q) = _filled(binding)
    qd = W.decode_query(w, 0, 0).cuda()
    want = cache.decode_attention(0, qd, W.softmax_scale())
    assert cache.status() == 0
    cache.test_arm_copy_timeout(16, 64)
    got = cache.decode_attention(0, qd, W.softmax_scale())
    torch.cuda.synchronize()                                   # the call came back
    assert cache.status() & binding.DEV_COPY_TIMEOUT
    assert torch.isfinite(got).all()
    # the packed units gave nothing; what is left is the residual window alone, or zero for a stream whose pairs all gave up
    assert float((got - want).abs().max()) > ATTN_TOL
    cache.test_arm_copy_timeout(0, 0)
    cache.reset()
    assert cache.status() == 0
    cache.quantize_append(0, k.cuda(), v.cuda(), q.cuda())
    again = cache.decode_attention(0, qd, W.softmax_scale())
    assert cache.status() == 0
    assert torch.equal(again, want)


def test_a_prefill_wait_that_runs_out_returns_with_the_status_bit(binding):
    """The same for the prefill attention: the barrier of every CTA's first key tile never completes, every role of the
    CTA gives up after 64 polls, the call returns with the status bit and writes no output; after a reset the call works."""
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=1, tokens=600, **W.P24)
    k, v, q = [t.cuda() for t in W.tokens(w, 0, 0, 600)]
    cache = U.make_cache(binding, w)
    want = cache.prefill(0, k, v, q, W.softmax_scale())
    assert cache.status() == 0
    cache.reset()
    cache.test_arm_copy_timeout(16, 64)
    out = torch.full_like(want, 7.0)
    cache.prefill(0, k, v, q, W.softmax_scale(), out=out)
    torch.cuda.synchronize()                                   # the call came back
    assert cache.status() & binding.DEV_COPY_TIMEOUT
    assert bool((out == 7.0).all())                            # no row was written
    cache.test_arm_copy_timeout(0, 0)
    cache.reset()
    assert cache.status() == 0
    again = cache.prefill(0, k, v, q, W.softmax_scale())
    assert cache.status() == 0
    assert torch.equal(again, want)


def test_attention_right_after_a_flush_and_after_an_external_write(binding):
    """Packed blocks are requested ahead of the stream-order wait except right after a flush of the same layer (or
    when the caller says it wrote cache memory itself); the results do not depend on which path was taken."""
    w, cache, (k, v, q) = _filled(binding, tokens=6 * 128)          # the window is full: the next append flushes
    k1, v1, q1 = W.tokens(w, 0, w.tokens, 1)
    qd = W.decode_query(w, 0, 1).cuda()
    cache.quantize_append(0, k1.cuda(), v1.cuda(), q1.cuda())       # flush + append enqueued directly before the attention
    first = cache.decode_attention(0, qd, W.softmax_scale())        # waits before its first read
    second = cache.decode_attention(0, qd, W.softmax_scale())       # requests its first blocks early
    cache.written_externally()
    third = cache.decode_attention(0, qd, W.softmax_scale())        # waits again
    assert torch.equal(first, second) and torch.equal(first, third)
    kk = torch.cat([k, k1], 2); vv = torch.cat([v, v1], 2); qq = torch.cat([q, q1], 2)
    oracle = U.oracle_streams(w, 0, kk, vv, qq, **{})
    ref = U.oracle_attention(w, oracle, qd.cpu())
    assert U.max_abs_err(w, first, ref) <= ATTN_TOL
    assert cache.status() == 0
