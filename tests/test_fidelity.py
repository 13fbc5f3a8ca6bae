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
