"""The threshold sweep tool: its bit-width formula on the CPU, its error ordering on the GPU."""
import pytest
import torch

from paper_2512_19206_b200 import fidelity as F
from paper_2512_19206_b200 import workloads as W


def test_effective_key_bits_matches_the_papers_formula():
    # Appendix C: B_eff = (16 n16 + 4 n4 + 2 n2) / D
    assert F.effective_key_bits(4, 0) == pytest.approx(2.4375)
    assert F.effective_key_bits(3, 24) == pytest.approx(2.703125)
    assert F.effective_key_bits(0, 0) == 2.0
    assert F.effective_key_bits(0, 128) == 4.0
    assert F.effective_key_bits(128, 0) == 16.0


def test_reference_attention_is_softmax_attention():
    torch.manual_seed(0)
    k = torch.randn(1, 2, 5, 128).bfloat16()
    v = torch.randn(1, 2, 5, 128).bfloat16()
    q = torch.randn(1, 4, 128).bfloat16()
    out = F.reference_attention(k, v, q, 0.1)
    for h in range(4):
        hk = h // 2
        p = torch.softmax((k[0, hk].double() @ q[0, h].double()) * 0.1, dim=0)
        assert torch.allclose(out[0, h].double(), p @ v[0, hk].double(), atol=1e-5)


@pytest.mark.gpu
def test_more_key_bits_mean_less_attention_error():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19206_b200 import build, binding
    build.build()
    binding.lib()
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=1, tokens=2048 + 40)
    inf = 1e30
    uniform = F.measure(w, inf, inf)
    two_tier = F.measure(w, 6.5, inf)
    all_bf16 = F.measure(w, -1.0, -1.0)
    assert uniform[0] == 2.0 and uniform[1] == 0 and uniform[2] == 0
    assert 2.0 < two_tier[0] < 3.0 and two_tier[1] > 0
    assert all_bf16[0] == 16.0
    # rms error of the attention output: promoting the salient channels helps, unquantized keys help more
    assert uniform[4] > two_tier[4] > all_bf16[4] > 0.0


@pytest.mark.gpu
def test_a_sweep_row_equals_the_oracles_numbers():
    """One setting of the sweep (three tiers) on a small workload: the tier counts and the key bit-width equal the
    oracle's exactly, the error columns equal the oracle's own (its quantized attention against its unquantized
    attention, both fp64) within twice the attention tolerance."""
    import numpy as np
    import gpu_util as U
    from oracle import mixkvq_oracle as O
    from paper_2512_19206_b200 import build, binding
    build.build()
    binding.lib()
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=1, tokens=1024 + 77, **W.P27)
    n_queries = 3
    beff, n16, n4, worst, rms = F.measure(w, w.tau_bf16, w.tau_u4, n_queries=n_queries)
    k, v, q = [x.cpu() for x in W.tokens(w, 0, 0, w.tokens, device="cuda")]      # the tool draws its inputs on the GPU
    orc = U.oracle_streams(w, 0, k, v, q)
    blocks = [b for st in orc.values() for b in st.blocks]
    o16 = float(np.mean([(b.tiers == O.TIER_BF16).sum() for b in blocks]))
    o4 = float(np.mean([(b.tiers == O.TIER_U4).sum() for b in blocks]))
    assert (n16, n4) == (o16, o4)
    assert beff == pytest.approx(O.effective_bits(o16, o4, 128 - o16 - o4))
    errs = []
    for i in range(n_queries):
        qd = U.f32(W.decode_query(w, 0, i, device="cuda"))
        for (b, hk), st in orc.items():
            qh = qd[b, hk * w.g:(hk + 1) * w.g]
            quant = st.attention(qh, W.softmax_scale())
            exact = O.unquantized_attention(qh, U.f32(k[b, hk]), U.f32(v[b, hk]), W.softmax_scale())
            errs.append(np.abs(np.asarray(quant, np.float64) - np.asarray(exact, np.float64)))
    errs = np.stack(errs)
    assert abs(worst - float(errs.max())) <= 4e-3
    assert abs(rms - float(np.sqrt((errs ** 2).mean()))) <= 4e-3
