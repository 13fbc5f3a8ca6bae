"""GPU parity of the rotating append (Appendix D: scores and keys are taken after the rotary embedding): the cache
after mixkvq_rope_append / mixkvq_rope_decode_step equals, byte for byte, the oracle's cache after rotating with the
oracle's rope and appending; the rotated tensors left in place equal the oracle's rotation bit for bit."""
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


def tables(n_pos, base=10000.0):
    inv = base ** (-np.arange(64, dtype=np.float64) / 64)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * inv[None]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def rotate_with_the_oracle(k, v, q, cos, sin, pos0):
    n = k.shape[2]
    kr = O.rope(U.f32(k), cos[pos0:pos0 + n], sin[pos0:pos0 + n])
    qr = O.rope(U.f32(q), cos[pos0:pos0 + n], sin[pos0:pos0 + n])
    return torch.from_numpy(kr).to(torch.bfloat16), v, torch.from_numpy(qr).to(torch.bfloat16)


@pytest.mark.parametrize("layout", [0, 1])
def test_bulk_then_decode_steps_with_rotation(binding, layout):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=2, tokens=3 * 128 + 57, **W.P27)
    n_dec = 140                                    # crosses a flush
    cos, sin = tables(w.tokens + n_dec + 8)
    cosd, sind = torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()
    k, v, q = W.tokens(w, 0, 0, w.tokens + n_dec)
    cache = U.make_cache(binding, w, max_tokens=w.tokens + n_dec + 256, layout=layout)
    # bulk append with rotation: the tensors come back rotated
    kd, vd, qd = k[:, :, :w.tokens].contiguous().cuda(), v[:, :, :w.tokens].contiguous().cuda(), q[:, :, :w.tokens].contiguous().cuda()
    cache.rope_append(0, kd, vd, qd, cosd, sind, 0)
    kr, vr, qr = rotate_with_the_oracle(k[:, :, :w.tokens], v[:, :, :w.tokens], q[:, :, :w.tokens], cos, sin, 0)
    assert torch.equal(kd.cpu(), kr) and torch.equal(qd.cpu(), qr)
    ks, vs, qs = [kr], [vr], [qr]
    scale = W.softmax_scale()
    out = None
    for i in range(n_dec):
        t = w.tokens + i
        k1, v1, q1 = k[:, :, t:t + 1].contiguous().cuda(), v[:, :, t:t + 1].contiguous().cuda(), q[:, :, t:t + 1].contiguous().cuda()
        if i % 2 == 0:
            out = cache.rope_decode_step(0, k1, v1, q1, cosd, sind, t, scale)
        else:                                      # the two-call form
            cache.rope_append(0, k1, v1, q1, cosd, sind, t)
            out = cache.decode_attention(0, q1.view(w.batch, w.n_q_heads, 128), scale)
        a, b, c = rotate_with_the_oracle(k[:, :, t:t + 1], v[:, :, t:t + 1], q[:, :, t:t + 1], cos, sin, t)
        assert torch.equal(q1.cpu(), c) and torch.equal(k1.cpu(), a)
        ks.append(a); vs.append(b); qs.append(c)
    kk, vv, qq = torch.cat(ks, 2), torch.cat(vs, 2), torch.cat(qs, 2)
    oracle = U.oracle_streams(w, 0, kk, vv, qq)
    U.compare_regions(cache, 0, w, oracle)
    ref = U.oracle_attention(w, oracle, qq[:, :, -1])
    assert U.max_abs_err(w, out, ref) <= ATTN_TOL
    assert cache.status() == 0


def test_rotation_errors(binding):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=1, tokens=40)
    cos, sin = tables(64)
    cosd, sind = torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()
    k, v, q = W.tokens(w, 0, 0, 40)
    cache = U.make_cache(binding, w, max_tokens=32)
    kd, qd = k.cuda(), q.cuda()
    with pytest.raises(binding.MixKVQError) as e:
        cache.rope_append(0, kd, v.cuda(), qd, cosd, sind, 0)         # more tokens than the cache holds
    assert e.value.code == -5
    assert torch.equal(kd.cpu(), k) and torch.equal(qd.cpu(), q)        # nothing was rotated
    lib = binding.lib()
    assert lib.mixkvq_rope_append(None, 0, None, None, None, None, None, 0, 1, None) == -1
