"""Pins of the oracle's sequence-split attention (partials per token set, log-sum-exp merge) against what the
mathematics fixes: the closed form for two tokens, Eq. 1 over the union, neutral empty parts, order independence."""
import math

import numpy as np

from oracle import mixkvq_oracle as O


def _bf16(x):
    return O.bf16_rne(np.asarray(x, np.float32))


def _stream(g=2, R=32, **kw):
    return O.OracleStream(g=g, R=R, G=32, score_bits=2, tau_bf16=1e9, tau_u4=1e9, **kw)


def test_two_tokens_closed_form():
    """One token per part, logits a and b: the merged output is (e^a v1 + e^b v2) / (e^a + e^b)."""
    a, b = 0.75, -1.25
    o = O.merge_partials(np.array([[[1.0, 0.0]], [[0.0, 2.0]]]), np.array([[a], [b]]))
    ea, eb = math.exp(a), math.exp(b)
    assert np.allclose(o, [[ea / (ea + eb), 2 * eb / (ea + eb)]], rtol=1e-15)


def test_merge_of_partials_is_attention_over_the_union():
    """Tokens split over three unflushed streams (nothing quantized): merging the three partials gives the textbook
    attention over all tokens; so does any order of the parts."""
    rng = np.random.default_rng(5)
    g, T = 2, 70
    K, V = _bf16(rng.normal(size=(T, O.D))), _bf16(rng.normal(size=(T, O.D)))
    q = _bf16(rng.normal(size=(g, O.D)) * 3)
    cuts = [(0, 11), (11, 43), (43, 70)]
    parts = []
    for (t0, t1) in cuts:
        st = _stream(g=g, R=32)
        # fewer than R tokens per stream or a window that is still unflushed: all tokens stay in full precision
        for t in range(t0, min(t1, t0 + 32)):
            st.append(K[t], V[t], np.zeros((g, O.D), np.float32))
        assert st.n_flushes == 0
        parts.append(st.attention_partial(q, 0.09))
    idx = np.concatenate([np.arange(t0, min(t1, t0 + 32)) for (t0, t1) in cuts])
    ref = O.unquantized_attention(q, K[idx], V[idx], 0.09)
    got = O.merge_partials([p[0] for p in parts], [p[1] for p in parts])
    assert np.abs(got - ref).max() < 1e-12
    rev = O.merge_partials([p[0] for p in parts[::-1]], [p[1] for p in parts[::-1]])
    assert np.abs(rev - got).max() < 1e-15


def test_partial_of_one_stream_is_its_attention_and_lse_is_the_log_denominator():
    rng = np.random.default_rng(6)
    st = _stream(g=3, R=32)
    K, V = _bf16(rng.normal(size=(100, O.D))), _bf16(rng.normal(size=(100, O.D)))
    Q = _bf16(rng.normal(size=(3, 100, O.D)))
    st.append_many(K, V, Q)                        # three flushed windows and a residual
    q = _bf16(rng.normal(size=(3, O.D)))
    o, lse = st.attention_partial(q, 0.1)
    assert np.abs(o - st.attention(q, 0.1)).max() < 1e-6            # attention() returns float32
    logits = (q.astype(np.float64) @ st.keys().T) * 0.1
    assert np.allclose(lse, np.log(np.exp(logits).sum(axis=1)), rtol=1e-13)
    assert np.abs(O.merge_partials([o], [lse]) - o).max() < 1e-15   # a single part is returned as it is


def test_empty_parts_are_neutral():
    st = _stream()
    o0, l0 = st.attention_partial(np.ones((2, O.D), np.float32), 0.1)
    assert not o0.any() and np.all(np.isneginf(l0))
    o1 = np.arange(2 * O.D, dtype=np.float64).reshape(2, O.D)
    l1 = np.array([0.3, -4.0])
    assert np.array_equal(O.merge_partials([o0, o1, o0], [l0, l1, l0]), o1)
    assert not O.merge_partials([o0, o0], [l0, l0]).any()          # nothing anywhere: zeros, no NaN


def test_large_logits_do_not_overflow():
    o = O.merge_partials(np.array([[[1.0]], [[3.0]]]), np.array([[5000.0], [5000.0 + math.log(3.0)]]))
    assert np.allclose(o, [[(1.0 + 9.0) / 4.0]], rtol=1e-14)
