"""Pins for the scoring rule of Section 4.2 and B_eff of Appendix C."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from conftest import to_bf16
from oracle import mixkvq_oracle as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))


def _window(rng, g=3, n=16):
    q = to_bf16(rng.standard_normal((g, n, O.D)) * rng.uniform(0.5, 4, (1, 1, O.D)))
    k = rng.standard_normal((n, O.D))
    k[:, [5, 17, 99]] *= 20
    return q, to_bf16(k)


def _exact_salience(q, k, bits):
    """Fractions: mean |q| over heads and tokens times (max - min)/(2^B - 1)."""
    g, n, D = q.shape
    out = []
    for d in range(D):
        I = sum(Fraction(abs(float(q[h, i, d]))) for i in range(n) for h in range(g)) / (g * n)
        S = (Fraction(float(k[:, d].max())) - Fraction(float(k[:, d].min()))) / ((1 << bits) - 1)
        out.append(I * S)
    return out


@pytest.mark.parametrize("bits", [2, 4])
def test_selected_set_equals_brute_force(rng, bits):
    q, k = _window(rng)
    acc, cnt = O.importance_from_queries(q)
    _, _, A = O.salience(acc, cnt, k, bits)
    exact = _exact_salience(q, k, bits)
    assert np.allclose(A, [float(a) for a in exact], rtol=1e-14, atol=0)
    srt = sorted(exact, reverse=True)
    for kbudget in (1, 3, 4, 10):
        # a threshold strictly between the k-th and (k+1)-th score selects exactly the top k
        tau = float((srt[kbudget - 1] + srt[kbudget]) / 2)
        tiers = O.assign_tiers(A, tau, -1.0)
        want = {d for d in range(O.D) if exact[d] > Fraction(float(np.float32(tau)))}
        assert set(np.flatnonzero(tiers == O.TIER_BF16)) == want
        assert want == set(np.argsort(-A)[:kbudget])


def test_three_tiers_and_strictness():
    A = np.array([0.0, 0.5, 1.0, 1.5, 2.0])
    t = O.assign_tiers(A, 1.5, 0.5)
    # A > tau_BF16 -> BF16; tau_U4 < A <= tau_BF16 -> UINT4; A <= tau_U4 -> UINT2 (equalities go down)
    assert list(t) == [O.TIER_U2, O.TIER_U2, O.TIER_U4, O.TIER_U4, O.TIER_BF16]


def test_tier_precedence_when_thresholds_cross(rng):
    # the paper's own R1-Qwen-14B pair has tau_BF16 < tau_INT4: the UINT4 tier is then empty
    t16, t4, _ = GOLD["thresholds"]["R1-Qwen-14B"]
    assert t16 < t4
    A = rng.uniform(0, 3, 1000)
    t = O.assign_tiers(A, t16, t4)
    assert not np.any(t == O.TIER_U4)
    assert np.array_equal(t == O.TIER_BF16, A > float(np.float32(t16)))


def test_monotone_in_thresholds(rng):
    q, k = _window(rng)
    acc, cnt = O.importance_from_queries(q)
    _, _, A = O.salience(acc, cnt, k, 2)
    prev16 = None
    for tau in np.linspace(0.1, 30, 40):
        sel = set(np.flatnonzero(O.assign_tiers(A, tau, 0.0) == O.TIER_BF16))
        if prev16 is not None:
            assert sel <= prev16
        prev16 = sel


def test_query_scaling_moves_only_that_channel(rng):
    q, k = _window(rng)
    acc, cnt = O.importance_from_queries(q)
    _, S0, A0 = O.salience(acc, cnt, k, 2)
    q2 = q.copy()
    q2[:, :, 7] *= -4.0
    acc2, _ = O.importance_from_queries(q2)
    _, S1, A1 = O.salience(acc2, cnt, k, 2)
    assert np.array_equal(S0, S1)
    assert A1[7] == 4.0 * A0[7]
    assert np.array_equal(np.delete(A0, 7), np.delete(A1, 7))


def test_error_only_variant_reduces_to_sensitivity(rng):
    # unit query magnitudes: I = 1 and the salience is the sensitivity alone (ablation 'error-only')
    q, k = _window(rng)
    q = np.sign(q) + (q == 0)
    acc, cnt = O.importance_from_queries(q.astype(np.float32))
    I, S, A = O.salience(acc, cnt, k, 2)
    assert np.all(I == 1.0) and np.array_equal(A, S)
    rngk = k.max(0).astype(np.float64) - k.min(0).astype(np.float64)
    assert np.array_equal(S, rngk / 3.0)


def test_gqa_aggregation_is_a_mean(rng):
    # repeating the heads of the group leaves the importance (a mean) unchanged
    q, k = _window(rng, g=2)
    a1, c1 = O.importance_from_queries(q)
    a2, c2 = O.importance_from_queries(np.concatenate([q, q], axis=0))
    assert c2 == 2 * c1
    assert np.allclose(a1 / c1, a2 / c2, rtol=1e-15)


def test_score_bits_is_a_constant_factor(rng):
    q, k = _window(rng)
    acc, cnt = O.importance_from_queries(q)
    _, S2, _ = O.salience(acc, cnt, k, 2)
    _, S4, _ = O.salience(acc, cnt, k, 4)
    assert np.allclose(S2 * 3, S4 * 15, rtol=1e-15)


def test_effective_bits_formula():
    bits = GOLD["tier_bits"]["bits"]
    assert bits == [16, 4, 2]
    assert O.effective_bits(4, 0, 124) == 2.4375
    assert O.effective_bits(3, 24, 101) == pytest.approx(2.703125)
    assert O.effective_bits(128, 0, 0) == 16 and O.effective_bits(0, 0, 128) == 2
    # the published effective bit-widths are reachable tier mixes of 128 channels
    for name, val in GOLD["thresholds"].items():
        if name == "cite":
            continue
        beff = val[2]
        best = min(abs(O.effective_bits(a, b, 128 - a - b) - beff) for a in range(20) for b in range(129 - a))
        assert best < 0.02


def test_memory_figures():
    m = GOLD["memory_example"]
    assert O.fp16_cache_bytes(m["n_layers"], m["n_kv_heads"], m["head_dim"], m["batch"], m["tokens"]) == m["bytes"] == 2 ** 39
    s = GOLD["memory_saving"]
    assert 1 - s["to_bits"] / s["from_bits"] == pytest.approx(s["saving_min"])


def test_error_only_mode_ranks_channels_by_sensitivity_alone(rng):
    # the ablation of Appendix E: A_d = S_d; the queries must not matter, the key ranges decide
    from conftest import to_bf16
    k = to_bf16(rng.standard_normal((129, O.D)) * rng.uniform(0.5, 6.0, (1, O.D)))
    v = to_bf16(rng.standard_normal((129, O.D)))
    outs = []
    for scale in (1.0, 7.0):
        q = to_bf16(rng.standard_normal((2, 129, O.D)) * scale)
        st = O.OracleStream(g=2, tau_bf16=5.0, tau_u4=3.0, importance_mode=2)
        st.append_many(k, v, q)
        outs.append(st.blocks[0])
    a, b = outs
    assert np.array_equal(a.tiers, b.tiers) and np.array_equal(a.A, b.A)
    S = (k[:128].max(0).astype(np.float64) - k[:128].min(0).astype(np.float64)) / 3.0
    assert np.array_equal(a.A, S)
    assert np.array_equal(a.tiers, np.where(S > 5.0, O.TIER_BF16, np.where(S > 3.0, O.TIER_U4, O.TIER_U2)))
    assert len(set(a.tiers.tolist())) == 3
