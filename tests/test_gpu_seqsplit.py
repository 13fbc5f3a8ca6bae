"""GPU parity of the sequence-split decode on one GPU: one context split into two caches (the ranges two ranks would
hold), their partials merged by the library, against the oracle with the same sharding."""
import numpy as np
import pytest
import torch

import gpu_util as U
from oracle import mixkvq_oracle as O
from paper_2512_19206_b200 import seqsplit
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


@pytest.mark.parametrize("tokens,parts", [(1500, 2), (100, 2), (2600, 3)])
def test_split_caches_merge_to_the_oracles_result(binding, tokens, parts):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=2, tokens=tokens, **W.P27)
    k, v, q = W.tokens(w, 0, 0, tokens)
    kf, vf, qf = U.f32(k), U.f32(v), U.f32(q)
    qd = W.decode_query(w, 0, 11)
    qdf = U.f32(qd)
    ranges = seqsplit.shard_ranges(tokens, parts, w.residual_len)
    outs, lses, ref_parts = [], [], []
    for (t0, t1) in ranges:
        cache = U.make_cache(binding, w)
        if t1 > t0:
            cache.quantize_append(0, k[:, :, t0:t1].contiguous().cuda(), v[:, :, t0:t1].contiguous().cuda(),
                                  q[:, :, t0:t1].contiguous().cuda())
        o, l = cache.decode_attention_partial(0, qd.cuda(), W.softmax_scale())
        outs.append(o)
        lses.append(l)
        ro, rl = np.zeros((w.batch, w.n_q_heads, O.D)), np.zeros((w.batch, w.n_q_heads))
        for b in range(w.batch):
            for hk in range(w.n_kv_heads):
                st = U.oracle_stream(w)
                hs = slice(hk * w.g, (hk + 1) * w.g)
                if t1 > t0:
                    st.append_many(kf[b, hk, t0:t1], vf[b, hk, t0:t1], qf[b, hs, t0:t1])
                ro[b, hs], rl[b, hs] = st.attention_partial(qdf[b, hs], W.softmax_scale())
        ref_parts.append((ro, rl))
        # each part by itself: output and log-denominator
        assert float(np.abs(o.cpu().numpy() - ro).max()) <= ATTN_TOL
        fin = np.isfinite(rl)
        assert np.array_equal(np.isfinite(l.cpu().numpy()), fin)
        assert float(np.abs(l.cpu().numpy()[fin] - rl[fin]).max()) <= 2e-3 if fin.any() else True
        assert cache.status() == 0
    merged = binding.merge_partials(torch.stack(outs), torch.stack(lses)).cpu().numpy()
    want = O.merge_partials([p[0] for p in ref_parts], [p[1] for p in ref_parts])
    assert float(np.abs(merged - want).max()) <= ATTN_TOL
    # merging one part returns it
    one = binding.merge_partials(outs[-1][None].contiguous(), lses[-1][None].contiguous())
    assert float((one - outs[-1]).abs().max()) <= 1e-6


def test_partial_of_a_ragged_batch_and_merge_with_empty_rows(binding):
    """Sequence 0 holds no token in the first cache: its rows carry lse = -inf there and the merge takes the other
    cache's rows unchanged."""
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=2, tokens=400, **W.P27)
    k, v, q = W.tokens(w, 0, 0, 300)
    qd = W.decode_query(w, 0, 2)
    a, b = U.make_cache(binding, w), U.make_cache(binding, w)
    a.quantize_append_ragged(0, k.cuda(), v.cuda(), q.cuda(), [0, 300])
    b.quantize_append(0, k[:, :, :200].contiguous().cuda(), v[:, :, :200].contiguous().cuda(), q[:, :, :200].contiguous().cuda())
    oa, la = a.decode_attention_partial(0, qd.cuda(), W.softmax_scale())
    ob, lb = b.decode_attention_partial(0, qd.cuda(), W.softmax_scale())
    assert torch.isneginf(la[0]).all() and torch.isfinite(la[1]).all() and not oa[0].any()
    merged = binding.merge_partials(torch.stack([oa, ob]), torch.stack([la, lb]))
    assert torch.equal(merged[0], ob[0])
    want = O.merge_partials(np.stack([oa.cpu().numpy(), ob.cpu().numpy()]).astype(np.float64),
                            np.stack([la.cpu().numpy(), lb.cpu().numpy()]).astype(np.float64))
    assert float(np.abs(merged.cpu().numpy() - want).max()) <= 1e-5
