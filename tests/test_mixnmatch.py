"""Layer-wise Mix'n'Match bookkeeping (Section 3.2 and the Appendix's four strategies): shapes the paper states."""
import pytest

from paper_2502_06786_b200 import mixnmatch as mnm


def test_hand_written_assignments():
    # 8 layers, two int8, four int4, two int2
    assert mnm.assign(2, 4, 2, "pyramid") == [2, 4, 4, 8, 8, 4, 4, 2]
    assert mnm.assign(2, 4, 2, "reverse_pyramid") == [8, 4, 4, 2, 2, 4, 4, 8]
    assert mnm.assign(2, 4, 2, "increasing") == [2, 2, 4, 4, 4, 4, 8, 8]
    assert mnm.assign(2, 4, 2, "decreasing") == [8, 8, 4, 4, 4, 4, 2, 2]
    # odd counts: the extra layer goes to the start
    assert mnm.assign(1, 3, 3, "pyramid") == [2, 2, 4, 4, 8, 4, 2]


@pytest.mark.parametrize("n8,n4,n2", [(8, 10, 8), (0, 26, 0), (5, 0, 21), (1, 1, 1), (42, 0, 0), (3, 7, 32)])
def test_shapes_the_paper_states(n8, n4, n2):
    n = n8 + n4 + n2
    for s in mnm.STRATEGIES:
        rs = mnm.assign(n8, n4, n2, s)
        assert len(rs) == n and rs.count(8) == n8 and rs.count(4) == n4 and rs.count(2) == n2
        assert mnm.effective_bits(rs) == pytest.approx((8 * n8 + 4 * n4 + 2 * n2) / n)
    p = mnm.assign(n8, n4, n2, "pyramid")
    peak = p.index(max(p))
    assert p[:peak + 1] == sorted(p[:peak + 1]) and p[peak:] == sorted(p[peak:], reverse=True)   # rises to the centre, then falls
    assert abs(p[:peak].count(2) - p[peak:].count(2)) <= 1                                    # both ends carry the low precision
    r = mnm.assign(n8, n4, n2, "reverse_pyramid")
    low = r.index(min(r))
    assert r[:low + 1] == sorted(r[:low + 1], reverse=True) and r[low:] == sorted(r[low:])
    assert mnm.assign(n8, n4, n2, "increasing") == sorted(p)
    assert mnm.assign(n8, n4, n2, "decreasing") == sorted(p, reverse=True)


def test_effective_bits_and_budget():
    assert mnm.effective_bits([2] * 10, overflow_fraction=0.05) == pytest.approx(2.05)     # the Errata's 2.05 bits
    assert mnm.effective_bits([8, 2], overflow_fraction=0.05) == pytest.approx(5.025)       # int8 layers have no extra bucket
    cands = mnm.counts_for_budget(26, 3.0)
    assert cands and all((8 * a + 4 * b + 2 * c) / 26 <= 3.0 and a + b + c == 26 for a, b, c in cands)
    best = cands[0]
    assert (8 * best[0] + 4 * best[1] + 2 * best[2]) / 26 == pytest.approx(3.0)            # 26 layers can hit 3 bits exactly
    with pytest.raises(ValueError):
        mnm.assign(1, 1, 1, "zigzag")
    with pytest.raises(ValueError):
        mnm.assign(-1, 1, 1)
