"""Pins of the oracle's fixed-budget tier rule: it is the threshold rule of Section 4.2 with thresholds placed between
consecutive saliences, it fills its quotas exactly, and equal saliences rank by channel index."""
import numpy as np

from oracle import mixkvq_oracle as O


def test_budget_rule_equals_threshold_rule_between_consecutive_saliences():
    rng = np.random.default_rng(3)
    for trial in range(20):
        A = rng.lognormal(0.0, 1.5, 128)                      # distinct with probability 1
        order = np.sort(A)[::-1]
        for k16, k4 in ((4, 0), (3, 24), (0, 7), (1, 127), (128, 0), (0, 0)):
            tiers = O.assign_tiers_by_budget(A, k16, k4) if k16 + k4 else O.assign_tiers(A, 1e30, 1e30)
            hi = 1e30 if k16 == 0 else (float(order[k16 - 1] + order[k16]) / 2 if k16 < 128 else float(order[-1]) / 2)
            n = k16 + k4
            lo = hi if k4 == 0 else (float(order[n - 1] + order[n]) / 2 if n < 128 else float(order[-1]) / 2)
            want = np.full(128, O.TIER_U2, np.uint8)
            want[A > lo] = O.TIER_U4
            want[A > hi] = O.TIER_BF16
            assert np.array_equal(tiers, want), (trial, k16, k4)
            assert int((tiers == O.TIER_BF16).sum()) == k16 and int((tiers == O.TIER_U4).sum()) == k4


def test_equal_saliences_rank_by_channel_index():
    A = np.array([2.0, 5.0, 2.0, 2.0, 0.5, 5.0])
    assert list(O.assign_tiers_by_budget(A, 1, 2)) == [O.TIER_U4, O.TIER_BF16, O.TIER_U2, O.TIER_U2, O.TIER_U2, O.TIER_U4]
    assert list(O.assign_tiers_by_budget(A, 3, 1)) == [O.TIER_BF16, O.TIER_BF16, O.TIER_U4, O.TIER_U2, O.TIER_U2, O.TIER_BF16]


def test_stream_with_budget_has_constant_tier_counts():
    rng = np.random.default_rng(5)
    st = O.OracleStream(g=2, R=32, G=32, budget_bf16=3, budget_u4=5)
    bf = lambda x: (np.asarray(x, np.float32).view(np.uint32) & 0xFFFF0000).view(np.float32)
    for _ in range(3 * 32 + 1):
        st.append(bf(rng.normal(0, 1, 128)), bf(rng.normal(0, 1, 128)), bf(rng.normal(0, 1, (2, 128))))
    assert len(st.blocks) == 3
    for blk in st.blocks:
        assert int((blk.tiers == O.TIER_BF16).sum()) == 3 and int((blk.tiers == O.TIER_U4).sum()) == 5
        top = np.argsort(-blk.A, kind="stable")[:3]
        assert set(np.flatnonzero(blk.tiers == O.TIER_BF16)) == set(top)
