"""GPU parity of the prefill call: causal full-precision attention of the prompt against the oracle's plain definition
(within the attention tolerance), and the cache it leaves behind against the oracle's append_many (byte for byte)."""
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


@pytest.mark.parametrize("name,batch,tokens", [("qwen7b", 1, 1), ("qwen7b", 2, 127), ("qwen7b", 1, 128), ("llama8b", 1, 129),
                                               ("qwen7b", 1, 700), ("tiny", 1, 1024)])
def test_prefill_attention_and_cache(binding, name, batch, tokens):
    w = W.small(W.CONFIGS[name], n_layers=1, batch=batch, tokens=tokens, **W.P27)
    k, v, q = W.tokens(w, 0, 0, tokens)
    cache = U.make_cache(binding, w)
    out = cache.prefill(0, k.cuda(), v.cuda(), q.cuda(), W.softmax_scale()).cpu().numpy()
    assert cache.status() == 0
    kf, vf, qf = U.f32(k), U.f32(v), U.f32(q)
    streams = [(0, 0), (batch - 1, w.n_kv_heads - 1)]
    worst = 0.0
    for (b, hk) in set(streams):
        ref = O.causal_attention(qf[b, hk * w.g:(hk + 1) * w.g], kf[b, hk], vf[b, hk], W.softmax_scale())
        worst = max(worst, float(np.abs(out[b, hk * w.g:(hk + 1) * w.g] - ref).max()))
    assert worst <= ATTN_TOL, worst
    assert np.isfinite(out).all()
    U.compare_regions(cache, 0, w, U.oracle_streams(w, 0, k, v, q, streams=list(set(streams))))


def test_prefill_large_magnitudes_and_errors(binding):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=1, tokens=300)
    k, v, q = W.tokens(w, 0, 0, 300)
    v = (v.float() * 64).to(torch.bfloat16)
    q = (q.float() * 4).to(torch.bfloat16)
    cache = U.make_cache(binding, w)
    out = cache.prefill(0, k.cuda(), v.cuda(), q.cuda(), W.softmax_scale()).cpu().numpy()
    ref = O.causal_attention(U.f32(q)[0, :w.g], U.f32(k)[0, 0], U.f32(v)[0, 0], W.softmax_scale())
    assert float(np.abs(out[0, :w.g] - ref).max()) <= ATTN_TOL * 64
    with pytest.raises(binding.MixKVQError) as e:                      # the layer is no longer empty
        cache.prefill(0, k.cuda(), v.cuda(), q.cuda(), W.softmax_scale())
    assert e.value.code == -2
    cache.reset()
    small = torch.empty(cache.prefill_scratch_bytes(300) - 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.MixKVQError):                           # the scratch buffer is too small
        cache.prefill(0, k.cuda(), v.cuda(), q.cuda(), W.softmax_scale(), scratch=small)
    assert cache.prefill_scratch_bytes(300) == 2 * w.n_kv_heads * 3 * 32768
