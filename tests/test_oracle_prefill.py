"""Pins of the oracle's prompt attention (causal Eq. 1): special cases with a closed form, a library routine, and
independence from the future."""
import numpy as np
import torch

from conftest import to_bf16
from oracle import mixkvq_oracle as O


def data(rng, g=3, L=37, D=128):
    return to_bf16(rng.normal(size=(g, L, D))), to_bf16(rng.normal(size=(L, D))), to_bf16(rng.normal(size=(L, D)))


def test_first_position_returns_the_first_value_and_last_row_is_plain_attention(rng):
    q, K, V = data(rng)
    out = O.causal_attention(q, K, V, 0.11)
    assert np.allclose(out[:, 0], np.broadcast_to(V[0].astype(np.float64), out[:, 0].shape), atol=0, rtol=0)
    assert np.allclose(out[:, -1], O.unquantized_attention(q[:, -1], K, V, 0.11), atol=1e-12)


def test_equals_the_library_causal_attention(rng):
    q, K, V = data(rng, g=2, L=50)
    out = O.causal_attention(q, K, V, 0.07)
    tq = torch.from_numpy(q.astype(np.float64))[None]
    tk = torch.from_numpy(K.astype(np.float64))[None, None].expand(1, 2, -1, -1)
    tv = torch.from_numpy(V.astype(np.float64))[None, None].expand(1, 2, -1, -1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=0.07)[0].numpy()
    assert np.allclose(out, ref, atol=1e-10)


def test_rows_do_not_depend_on_later_tokens_and_sum_to_one(rng):
    q, K, V = data(rng, L=24)
    out = O.causal_attention(q, K, V, 0.2)
    K2, V2 = K.copy(), V.copy()
    K2[15:] += 3.0
    V2[15:] -= 5.0
    out2 = O.causal_attention(q, K2, V2, 0.2)
    assert np.array_equal(out[:, :15], out2[:, :15]) and not np.allclose(out[:, 15:], out2[:, 15:])
    ones = O.causal_attention(q, K, np.ones_like(V), 0.2)          # constant values: the weights of a row sum to one
    assert np.allclose(ones, 1.0, atol=1e-12)


def test_zero_keys_give_the_running_mean_of_the_values(rng):
    q, K, V = data(rng, L=16)
    out = O.causal_attention(q, np.zeros_like(K), V, 0.3)
    want = np.cumsum(V.astype(np.float64), axis=0) / np.arange(1, 17)[:, None]
    assert np.allclose(out, np.broadcast_to(want, out.shape), atol=1e-12)
