"""Pins for the oracle's attention (Eq. 1 over the mixed-precision cache)."""
import numpy as np
import pytest
import torch

from conftest import to_bf16
from oracle import mixkvq_oracle as O

SCALE = 1.0 / np.sqrt(128.0)


def _tokens(rng, n, g):
    k = rng.standard_normal((n, O.D)); k[:, [9, 50, 51]] *= 12
    v = rng.standard_normal((n, O.D))
    q = rng.standard_normal((g, n, O.D)) * rng.uniform(0.5, 4, (1, 1, O.D))
    return to_bf16(k), to_bf16(v), to_bf16(q)


def test_all_channels_bf16_reduces_to_library_attention_on_keys(rng):
    # every channel promoted (A >= 0 > tau): keys are exact, values stay 2-bit; with values also taken
    # from the dequantized store this must equal a library scaled-dot-product attention
    k, v, q = _tokens(rng, 300, 4)
    st = O.OracleStream(g=4, tau_bf16=-1.0, tau_u4=-1.0)
    st.append_many(k, v, q)
    assert all((b.tiers == O.TIER_BF16).all() for b in st.blocks)
    assert np.array_equal(st.keys(), k.astype(np.float64))
    qd = q[:, -1]
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(qd).double()[None], torch.from_numpy(st.keys())[None], torch.from_numpy(st.values())[None],
        scale=float(SCALE))[0].numpy()
    assert np.abs(st.attention(qd, SCALE) - ref).max() < 1e-6


def test_no_flushed_block_is_textbook_attention(rng):
    # fewer than R tokens: nothing is quantized at all -> unquantized attention, library routine
    k, v, q = _tokens(rng, 100, 7)
    st = O.OracleStream(g=7)
    st.append_many(k, v, q)
    qd = q[:, 5]
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(qd).double()[None], torch.from_numpy(k).double()[None], torch.from_numpy(v).double()[None],
        scale=float(SCALE))[0].numpy()
    assert np.abs(st.attention(qd, SCALE) - ref).max() < 1e-6
    assert np.abs(O.unquantized_attention(qd, k, v, SCALE) - ref).max() < 1e-12


def test_softmax_rows_sum_to_one(rng):
    k, v, q = _tokens(rng, 400, 5)
    st = O.OracleStream(g=5, tau_bf16=6.0, tau_u4=3.0)
    st.append_many(k, v, q)
    _, p = st.attention(q[:, -1], SCALE, return_probs=True)
    assert p.shape == (5, 400) and np.all(p >= 0)
    assert np.abs(p.sum(1) - 1).max() < 1e-12


def test_zero_keys_give_the_mean_value(rng):
    k, v, q = _tokens(rng, 260, 2)
    st = O.OracleStream(g=2)
    st.append_many(np.zeros_like(k), v, q)
    assert np.abs(st.attention(q[:, -1], SCALE) - st.values().mean(0)[None]).max() < 1e-6


def test_identical_value_rows_come_back(rng):
    k, v, q = _tokens(rng, 260, 2)
    v[:] = v[0]
    st = O.OracleStream(g=2, tau_bf16=6.0, tau_u4=3.0)
    st.append_many(k, v, q)
    vt = st.values()
    assert np.abs(vt[:256] - vt[0]).max() == 0                # per-token quantization of equal rows is equal
    assert np.array_equal(vt[256:], v[256:].astype(np.float64))   # the residual tokens are not quantized
    o, p = st.attention(q[:, -1], SCALE, return_probs=True)
    w = p[:, :256].sum(1, keepdims=True)
    assert np.abs(o - (w * vt[0][None] + (1 - w) * v[0][None].astype(np.float64))).max() < 1e-6
    assert np.abs(vt[0] - v[0]).max() <= (v[0].max() - v[0].min()) / 3 / 2 * 1.01 + 1e-6


def test_logit_error_bound(rng):
    # |q.k - q.k~| <= 1/2 sum_d |q_d| s_{d,group}  (logit error decomposition + the s/2 bound)
    k, v, q = _tokens(rng, 256 + 1, 3)
    st = O.OracleStream(g=3, tau_bf16=6.0, tau_u4=3.0)
    st.append_many(k, v, q)
    qd = q[:, -1].astype(np.float64)
    err = np.abs(qd @ k[:256].astype(np.float64).T - qd @ st.keys()[:256].T)      # [g, 256]
    for bi, blk in enumerate(st.blocks):
        s = np.repeat(blk.ks.astype(np.float64), st.G, axis=0)                    # [R, D]
        bound = 0.5 * np.abs(qd) @ s.T                                            # [g, R]
        assert np.all(err[:, bi * 128:(bi + 1) * 128] <= bound + 1e-9)
    assert err.max() > 0


def test_joint_channel_permutation_invariance(rng):
    k, v, q = _tokens(rng, 300, 2)
    perm = rng.permutation(O.D)
    a = O.OracleStream(g=2, tau_bf16=6.0, tau_u4=3.0); a.append_many(k, v, q)
    b = O.OracleStream(g=2, tau_bf16=6.0, tau_u4=3.0); b.append_many(k[:, perm], v, q[:, :, perm])
    assert np.array_equal(a.blocks[0].tiers[perm], b.blocks[0].tiers)
    assert np.abs(a.attention(q[:, -1], SCALE) - b.attention(q[:, -1][:, perm], SCALE)).max() < 1e-6


def test_promotion_reduces_logit_error(rng):
    # promoting the salient channels must shrink the attention-logit error versus plain 2-bit keys
    k, v, q = _tokens(rng, 257, 4)
    plain = O.OracleStream(g=4); plain.append_many(k, v, q)
    mixed = O.OracleStream(g=4, tau_bf16=6.0, tau_u4=3.0); mixed.append_many(k, v, q)
    qd = q[:, -1].astype(np.float64)
    exact = qd @ k[:256].astype(np.float64).T
    e_plain = np.abs(exact - qd @ plain.keys()[:256].T).mean()
    e_mixed = np.abs(exact - qd @ mixed.keys()[:256].T).mean()
    assert e_mixed < 0.5 * e_plain
