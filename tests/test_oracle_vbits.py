"""Pins of the oracle's 4-bit values: Eq. 2 with 16 levels per token group, stored as two 2-bit planes."""
import numpy as np

from oracle import mixkvq_oracle as O


def bf(x):
    return (np.asarray(x, np.float32).view(np.uint32) & 0xFFFF0000).view(np.float32)


def stream(v_bits, G=32, seed=0, n=64 + 7):
    rng = np.random.default_rng(seed)
    st = O.OracleStream(g=2, R=64, G=G, tau_bf16=2.0, v_bits=v_bits)
    k, v, q = bf(rng.normal(0, 1, (n, 128))), bf(rng.normal(0, 3, (n, 128))), bf(rng.normal(0, 1, (2, n, 128)))
    st.append_many(k, v, q)
    return st, v


def test_four_bit_values_obey_the_half_scale_bound_and_use_sixteen_levels():
    for G in (32, 64):
        st, v = stream(4, G)
        blk = st.blocks[0]
        assert blk.vcodes.max() == 15 and blk.vcodes.min() == 0
        deq = st.values()[:64]
        s = np.repeat(blk.vs.astype(np.float64), G, axis=1)
        assert np.all(np.abs(deq - v[:64].astype(np.float64)) <= s / 2 * (1 + 1e-6))
        # group minimum -> code 0 (exact zero-point), group maximum -> code 15
        grp = v[:64].reshape(64, 128 // G, G)
        codes = blk.vcodes.reshape(64, 128 // G, G)
        assert np.all(codes[grp == grp.min(axis=2, keepdims=True)] == 0)
        assert np.all(codes[grp == grp.max(axis=2, keepdims=True)] == 15)


def test_four_bit_values_are_closer_than_two_bit_values():
    a, v = stream(2)
    b, _ = stream(4)
    ea = np.abs(a.values()[:64] - v[:64]).mean()
    eb = np.abs(b.values()[:64] - v[:64]).mean()
    assert eb < ea / 3
    assert np.array_equal(a.blocks[0].kcodes, b.blocks[0].kcodes)       # the keys do not depend on the value width


def test_two_planes_round_trip_and_block_size():
    for G in (32, 64):
        st, _ = stream(4, G)
        blk = st.blocks[0]
        buf = O.pack_base(blk, 64, G, 4)
        assert len(buf) == O.base_bytes(64, G, 4) == O.base_bytes(64, G) + 2 * 1024
        klow, ks, kz, vcodes, vs, vz = O.unpack_base(buf, 64, G, 4)
        assert np.array_equal(vcodes, blk.vcodes) and np.array_equal(vs, blk.vs) and np.array_equal(vz, blk.vz)
        # the low plane alone is what a 2-bit reader of the same bytes would see
        low = O.unpack_base(buf[:], 64, G, 4)[3] & 3
        assert np.array_equal(low, blk.vcodes & 3)
