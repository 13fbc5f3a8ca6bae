"""Pins of the oracle's sink tokens (Appendix E fixes a sink length in its settings): the first sink_len tokens stay
unquantized for good and take no part in scoring; everything after them behaves like a stream without a sink."""
import numpy as np

from oracle import mixkvq_oracle as O


def bf(x):
    return (np.asarray(x, np.float32).view(np.uint32) & 0xFFFF0000).view(np.float32)


def data(n, g, seed):
    rng = np.random.default_rng(seed)
    return bf(rng.normal(0, 1, (n, 128))), bf(rng.normal(0, 1, (n, 128))), bf(rng.normal(0, 2, (g, n, 128)))


def test_a_sequence_inside_the_sink_is_unquantized_attention():
    k, v, q = data(20, 3, 1)
    st = O.OracleStream(g=3, R=32, G=32, tau_bf16=0.5, sink_len=32)
    st.append_many(k, v, q)
    assert st.n_sink == 20 and st.r == 0 and not st.blocks and st.cnt == 0 and st.n_tokens == 20
    qd = bf(np.random.default_rng(2).normal(0, 1, (3, 128)))
    want = O.unquantized_attention(qd, k, v, 0.1)
    assert np.allclose(st.attention(qd, 0.1), want, rtol=0, atol=1e-6)


def test_after_the_sink_the_stream_is_a_stream_without_sink():
    n, g, sink = 32 + 3 * 64 + 11, 2, 32
    k, v, q = data(n, g, 3)
    a = O.OracleStream(g=g, R=64, G=32, tau_bf16=1.2, tau_u4=0.6, sink_len=sink)
    a.append_many(k, v, q)
    b = O.OracleStream(g=g, R=64, G=32, tau_bf16=1.2, tau_u4=0.6)
    b.append_many(k[sink:], v[sink:], q[:, sink:])
    assert a.n_sink == sink and np.array_equal(a.sinkK, k[:sink]) and np.array_equal(a.sinkV, v[:sink])
    assert len(a.blocks) == len(b.blocks) == 3 and a.r == b.r and a.cnt == b.cnt and np.array_equal(a.acc, b.acc)
    for x, y in zip(a.blocks, b.blocks):
        assert np.array_equal(x.tiers, y.tiers) and np.array_equal(x.kcodes, y.kcodes) and np.array_equal(x.vcodes, y.vcodes)
    pa, pb = O.pack_stream(a), O.pack_stream(b)
    for key in ("base", "table", "extras", "state", "resK", "resV"):
        assert pa[key] == pb[key]
    assert len(pa["sinkK"]) == sink * 256 and pb["sinkK"] == b""
    # attention: the sink rows are the first keys and values
    qd = bf(np.random.default_rng(4).normal(0, 1, (g, 128)))
    K = np.concatenate([k[:sink].astype(np.float64), b.keys()])
    V = np.concatenate([v[:sink].astype(np.float64), b.values()])
    assert np.allclose(a.attention(qd, 0.09), O.unquantized_attention(qd, K, V, 0.09), rtol=0, atol=1e-6)


def test_single_appends_equal_bulk_with_a_sink():
    k, v, q = data(32 + 64 + 5, 2, 9)
    a = O.OracleStream(g=2, R=32, G=32, tau_bf16=1.0, sink_len=32)
    a.append_many(k, v, q)
    b = O.OracleStream(g=2, R=32, G=32, tau_bf16=1.0, sink_len=32)
    for t in range(k.shape[0]):
        b.append(k[t], v[t], q[:, t])
    assert O.pack_stream(a) == O.pack_stream(b)
