"""Pins for the cache workflow (Section 4.2, Appendix D.1/D.2) and the byte layout."""
import json
import os

import numpy as np
import pytest

from conftest import to_bf16
from oracle import mixkvq_oracle as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))


def _tokens(rng, n, g):
    k = rng.standard_normal((n, O.D)); k[:, [3, 64, 65, 120]] *= 15
    v = rng.standard_normal((n, O.D))
    q = rng.standard_normal((g, n, O.D)) * rng.uniform(0.5, 4, (1, 1, O.D))
    return to_bf16(k), to_bf16(v), to_bf16(q)


def test_flush_cadence_matches_published_call_rate(rng):
    R = GOLD["call_rate"]["residual_len"]
    st = O.OracleStream(g=1, R=R, G=32)
    k, v, q = _tokens(rng, 32 * 40 + 1, 1)
    for i in range(k.shape[0]):
        st.append(k[i], v[i], q[:, i])
    rate = 100.0 * st.n_flushes / (k.shape[0] - 1)
    assert rate == pytest.approx(GOLD["call_rate"]["percent"], abs=0.006)   # 3.125 % printed as 3.13


def test_flush_is_lazy_newest_tokens_stay_full_precision(rng):
    st = O.OracleStream(g=2, R=64, G=32)
    k, v, q = _tokens(rng, 65, 2)
    for i in range(64):
        st.append(k[i], v[i], q[:, i])
    assert st.r == 64 and len(st.blocks) == 0          # full window, not flushed yet
    assert np.array_equal(st.keys(), k[:64].astype(np.float64))
    st.append(k[64], v[64], q[:, 64])
    assert st.r == 1 and len(st.blocks) == 1 and st.n_tokens == 65
    assert np.array_equal(st.keys()[-1], k[64].astype(np.float64))


@pytest.mark.parametrize("R,G", [(128, 32), (128, 128), (64, 32), (96, 32), (256, 64)])
def test_bulk_equals_streamed(rng, R, G):
    n = 2 * R + 37
    k, v, q = _tokens(rng, n, 3)
    a = O.OracleStream(g=3, R=R, G=G, tau_bf16=6.0, tau_u4=3.0)
    b = O.OracleStream(g=3, R=R, G=G, tau_bf16=6.0, tau_u4=3.0)
    a.append_many(k, v, q)
    for i in range(n):
        b.append(k[i], v[i], q[:, i])
    pa, pb = O.pack_stream(a), O.pack_stream(b)
    assert pa.keys() == pb.keys()
    for key in pa:
        assert pa[key] == pb[key], key
    assert len(a.blocks) == 2 and a.r == 37


def test_window_and_cumulative_importance(rng):
    k, v, q = _tokens(rng, 129, 2)
    w = O.OracleStream(g=2, importance_mode=0)
    c = O.OracleStream(g=2, importance_mode=1)
    w.append_many(k, v, q); c.append_many(k, v, q)
    assert w.cnt == 2 and c.cnt == 2 * 129
    assert np.array_equal(w.acc, np.abs(q[:, 128].astype(np.float64)).sum(0))
    assert np.allclose(c.acc, np.abs(q.astype(np.float64)).sum((0, 1)), rtol=1e-13)


def test_blocks_keep_their_tiers(rng):
    k, v, q = _tokens(rng, 257, 1)
    st = O.OracleStream(g=1, tau_bf16=5.0, tau_u4=2.5)
    st.append_many(k[:129], v[:129], q[:, :129])
    t0 = st.blocks[0].tiers.copy()
    q2 = q.copy(); q2[:, 129:, :] *= 8
    st.append_many(k[129:], v[129:], q2[:, 129:])
    assert np.array_equal(st.blocks[0].tiers, t0)
    assert (st.blocks[1].tiers == O.TIER_BF16).sum() > (t0 == O.TIER_BF16).sum()


# ---------------------------------------------------------------------------------------- layout
def _flushed(rng, R, G, tau16=6.0, tau4=3.0):
    k, v, q = _tokens(rng, R + 1, 2)
    st = O.OracleStream(g=2, R=R, G=G, tau_bf16=tau16, tau_u4=tau4)
    st.append_many(k, v, q)
    return st, k, v


@pytest.mark.parametrize("R,G", [(128, 32), (128, 64), (128, 128), (64, 32), (256, 128)])
def test_pack_roundtrip_and_sizes(rng, R, G):
    st, k, v = _flushed(rng, R, G, tau4=1.0)
    blk = st.blocks[0]
    n16, n4 = int((blk.tiers == 2).sum()), int((blk.tiers == 1).sum())
    assert n16 >= 3 and n4 >= 5
    base = O.pack_base(blk, R, G)
    assert len(base) == (R // G) * 512 + (R // 32) * (2048 + 128 * (128 // G))
    klow, ks, kz, vc, vs, vz = O.unpack_base(base, R, G)
    quant = blk.tiers != O.TIER_BF16
    assert np.array_equal(klow[:, quant], blk.kcodes[:, quant] & 3)
    assert not klow[:, ~quant].any() and not ks[:, ~quant].any() and not kz[:, ~quant].any()
    assert np.array_equal(ks[:, quant], blk.ks[:, quant]) and np.array_equal(kz[:, quant], blk.kz[:, quant])
    assert np.array_equal(vc, blk.vcodes) and np.array_equal(vs, blk.vs) and np.array_equal(vz, blk.vz)
    ex, a, b = O.pack_extras(blk, R, dense=True)                      # the 4-bit-base form of the high plane
    n16p, n4p = (n16 + 1) // 2, 2 * ((n4 + 1) // 2)
    assert (a, b) == (n16, n4) and O.dense_high_plane(-1.0) and not O.dense_high_plane(3.8)
    assert len(ex) == 16 * ((2 * n16p + n4p + 15) // 16) + (R // 32) * (128 * n16p + 1024)
    assert len(ex) % 16 == 0
    # dense high plane: code >> 2 of a UINT4 channel sits where the low plane keeps the channel's low bits
    hdr = 16 * ((2 * n16p + n4p + 15) // 16)
    words = np.frombuffer(ex[hdr:], "<u4")
    unit_words = (128 * n16p + 1024) // 4
    for (j, d) in [(0, 0), (33, 17), (R - 1, 127), (40, 64), (5, 99)]:
        u, jj = divmod(j, 32)
        off, bit = O._k_code_pos(jj, d)
        got = (int(words[u * unit_words + 32 * n16p + off // 4]) >> bit) & 3
        assert got == (blk.kcodes[j, d] >> 2 if blk.tiers[d] == O.TIER_U4 else 0)
    st2, _, _ = _flushed(rng, R, G, tau4=4.5)                         # few UINT4 channels: 16 bytes per channel pair
    blk2 = st2.blocks[0]
    m16, m4 = int((blk2.tiers == 2).sum()), int((blk2.tiers == 1).sum())
    assert m4 > 0
    assert len(O.pack_extras(blk2, R)[0]) == 16 * ((2 * ((m16 + 1) // 2) + 2 * ((m4 + 1) // 2) + 15) // 16) + (R // 32) * (
        128 * ((m16 + 1) // 2) + 8 * 2 * ((m4 + 1) // 2))


def test_extras_content_by_hand(rng):
    R, G = 128, 32
    st, k, v = _flushed(rng, R, G, tau4=4.5)
    blk = st.blocks[0]
    ex, n16, n4 = O.pack_extras(blk, R)
    assert 5 <= n4
    chan16 = [d for d in range(128) if blk.tiers[d] == 2]
    chan4 = [d for d in range(128) if blk.tiers[d] == 1]
    n16p, n4p = (n16 + 1) // 2, 2 * ((n4 + 1) // 2)
    assert list(ex[:n16]) == chan16 and list(ex[2 * n16p:2 * n16p + n4]) == chan4
    hdr = 16 * ((2 * n16p + n4p + 15) // 16)
    assert all(b in (0, 0xFF) for b in ex[2 * n16p + n4:hdr])
    unit = 128 * n16p + 8 * n4p
    words = np.frombuffer(ex[hdr:], "<u4")
    raw = O.bf16_to_u16(k[:R])
    for (j, i) in [(0, 0), (37, 1), (127, n16p - 1), (64, 0)]:
        u, jj = divmod(j, 32)
        w = int(words[(u * unit) // 4 + i * 32 + jj])
        assert (w & 0xFFFF) == raw[j, chan16[2 * i]]
        if 2 * i + 1 < n16:
            assert (w >> 16) == raw[j, chan16[2 * i + 1]]
        else:
            assert (w >> 16) == 0
    for (j, idx) in [(0, 0), (45, 1), (100, n4 - 1), (31, 2)]:
        u, jj = divmod(j, 32)
        i, e = divmod(idx, 2)
        mt, row = divmod(jj, 16); rh, r = divmod(row, 8)
        w = int(words[(u * unit + 128 * n16p) // 4 + i * 4 + (r % 4)])
        got = (w >> (16 * e + 8 * (r // 4) + 2 * (2 * mt + rh))) & 3
        assert got == blk.kcodes[j, chan4[idx]] >> 2
    # dequantizing both planes reproduces Eq. 3 for a UINT4 channel
    d = chan4[0]
    c = blk.kcodes[:, d].astype(np.float64)
    s = np.repeat(blk.ks[:, d].astype(np.float64), G); z = np.repeat(blk.kz[:, d].astype(np.float64), G)
    assert np.array_equal((blk.kcodes[:, d] & 3) * s + (blk.kcodes[:, d] >> 2) * (4 * s) + z, c * s + z)


def test_fragment_order_of_key_codes():
    # one 16-byte chunk per (lane, m-tile) holds registers a0..a3; field kt of each half = k-tile kt
    for jj in range(32):
        for d in range(128):
            off, bit = O._k_code_pos(jj, d)
            mt, lane, a = off // 512, (off % 512) // 16, (off % 16) // 4
            r, t = lane // 4, lane % 4
            rh, ch = a % 2, a // 2
            assert jj == mt * 16 + rh * 8 + r
            assert d == (bit % 16) // 2 * 16 + ch * 8 + 2 * t + bit // 16


@pytest.mark.parametrize("G", [32, 64, 128])
def test_tile_layout_roundtrip_and_content(rng, G):
    st, k, v = _flushed(rng, 128, G)
    blk = st.blocks[0]
    chan16 = [d for d in range(128) if blk.tiers[d] == 2]
    chan4 = [d for d in range(128) if blk.tiers[d] == 1]
    n16, n4 = len(chan16), len(chan4)
    assert n16 >= 3 and n4 >= 5
    base = O.pack_base_tile(blk, G)
    assert len(base) == (128 // G) * 512 + 8192 + 512 * (128 // G) == O.tile_base_bytes(G)
    klow, ks, kz, vc, vs, vz = O.unpack_base_tile(base, G)
    quant = blk.tiers != O.TIER_BF16
    assert np.array_equal(klow[:, quant], blk.kcodes[:, quant] & 3)
    assert not klow[:, ~quant].any() and not ks[:, ~quant].any() and not kz[:, ~quant].any()
    assert np.array_equal(ks[:, quant], blk.ks[:, quant]) and np.array_equal(kz[:, quant], blk.kz[:, quant])
    assert np.array_equal(vc, blk.vcodes) and np.array_equal(vs, blk.vs) and np.array_equal(vz, blk.vz)
    # by hand: token 77's key codes are the 32 bytes at {0, 2048} + 77*16 of the key plane, channel d in
    # word (d % 64) // 16 of half d // 64, field (d % 16) // 2 of 16-bit half d % 2
    kplane = np.frombuffer(base[(128 // G) * 512:(128 // G) * 512 + 4096], "<u2")
    for d in [0, 1, 17, 63, 64, 100, 127]:
        if quant[d]:
            half = kplane[((d // 64) * 2048 + 77 * 16 + ((d % 64) // 16) * 4) // 2 + d % 2]
            assert (int(half) >> (2 * ((d % 16) // 2))) & 3 == blk.kcodes[77, d] & 3
    vplane = np.frombuffer(base[(128 // G) * 512 + 4096:(128 // G) * 512 + 8192], "<u2")
    for t in [0, 15, 16, 64, 99, 127]:
        half = vplane[((t // 64) * 2048 + 5 * 16 + ((t % 64) // 16) * 4) // 2 + t % 2]
        assert (int(half) >> (2 * ((t % 16) // 2))) & 3 == blk.vcodes[t, 5]
    ex, a, b = O.pack_extras_tile(blk)
    n16p, n4w = (n16 + 1) // 2, (n4 + 15) // 16
    assert (a, b) == (n16, n4) and len(ex) == 16 * ((2 * n16p + 16 * n4w + 15) // 16) + 512 * (n16p + n4w)
    hdr = len(ex) - 512 * (n16p + n4w)
    assert list(ex[:n16]) == chan16 and list(ex[2 * n16p:2 * n16p + n4]) == chan4
    assert all(x in (0, 0xFF) for x in ex[2 * n16p + n4:hdr])
    words = np.frombuffer(ex[hdr:], "<u4")
    raw = O.bf16_to_u16(k[:128])
    for (j, i) in [(0, 0), (37, 1), (127, n16p - 1)]:
        w = int(words[i * 128 + j])
        assert (w & 0xFFFF) == raw[j, chan16[2 * i]]
        assert (w >> 16) == (raw[j, chan16[2 * i + 1]] if 2 * i + 1 < n16 else 0)
    for (j, idx) in [(0, 0), (45, 1), (100, n4 - 1)]:
        w = int(words[(n16p + idx // 16) * 128 + j])
        assert (w >> (16 * (idx % 2) + 2 * ((idx % 16) // 2))) & 3 == blk.kcodes[j, chan4[idx]] >> 2


def test_stream_regions(rng):
    k, v, q = _tokens(rng, 3 * 128 + 5, 2)
    st = O.OracleStream(g=2, tau_bf16=6.0, tau_u4=3.0)
    st.append_many(k, v, q)
    p = O.pack_stream(st, layout=O.LAYOUT_TILE)
    assert len(p["base"]) == 3 * 12288 and len(p["table"]) == 24
    off = 0
    for i, blk in enumerate(st.blocks):
        e = p["table"][8 * i:8 * i + 8]
        assert int.from_bytes(e[:4], "little") == off
        assert e[4] == (blk.tiers == 2).sum() and e[5] == (blk.tiers == 1).sum() and e[6:] == b"\0\0"
        off += len(O.pack_extras_tile(blk)[0]) // 16
    assert int.from_bytes(p["state"][1028:1032], "little") == off
    assert len(p["resK"]) == 5 * 256 and len(p["resV"]) == 5 * 256
    assert np.array_equal(np.frombuffer(p["resV"], "<u2").reshape(5, 128), O.bf16_to_u16(v[-5:]))


def test_fragment_layout_places_each_scale_group_before_its_first_unit():
    # G = 32: [meta 0][unit 0][meta 1][unit 1]...; G = 128: [meta 0][unit 0][unit 1][unit 2][unit 3]
    assert [O.frag_meta_off(kg, 32, 2560) for kg in range(4)] == [0, 3072, 6144, 9216]
    assert [O.frag_unit_off(u, 32, 2560) for u in range(4)] == [512, 3584, 6656, 9728]
    assert O.frag_meta_off(0, 128, 2176) == 0 and [O.frag_unit_off(u, 128, 2176) for u in range(4)] == [512, 2688, 4864, 7040]
    # R = 256, G = 64: a group covers two units
    assert [O.frag_meta_off(kg, 64, 2304) for kg in range(4)] == [0, 5120, 10240, 15360]
    assert [O.frag_unit_off(u, 64, 2304) for u in range(8)] == [512, 2816, 5632, 7936, 10752, 13056, 15872, 18176]
    for G, ub, U in ((32, 2560, 4), (64, 2304, 8), (128, 2176, 4)):
        spans = sorted([(O.frag_meta_off(kg, G, ub), 512) for kg in range(U * 32 // G)] + [(O.frag_unit_off(u, G, ub), ub) for u in range(U)])
        assert spans[0][0] == 0 and all(a + n == b for (a, n), (b, _) in zip(spans, spans[1:]))      # a partition of the block
        assert spans[-1][0] + spans[-1][1] == O.base_bytes(U * 32, G)
