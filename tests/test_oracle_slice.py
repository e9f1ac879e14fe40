"""Pins for the oracle's slicing operator (Eq. 6, Eq. 8, Appendix A, Errata).

Nothing here calls the CUDA path.  The expected values are the paper's printed
examples (tests/golden), closed forms derived by hand from Eq. 6 / Eq. 8, and
invariants; a wrong rounding rule, clamp, shift or sign fails at least one.
"""
import os

import numpy as np
import pytest

from oracle import ref

ALL_Q = np.arange(256, dtype=np.uint8)


def S(q, r, ep=False):
    st, out = ref.slice_values(np.ascontiguousarray(q, dtype=np.uint8), r, ep)
    assert st == ref.OK
    return out.astype(np.int64)


def _rows(path):
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                yield line.split()


def test_paper_worked_examples(golden_dir):
    n = 0
    for q, r, ep, want in _rows(os.path.join(golden_dir, "slice_worked_examples.txt")):
        got = S(np.array([int(q)]), int(r), bool(int(ep)))[0]
        assert got == int(want), (q, r, ep, got, want)
        n += 1
    assert n == 4


def test_int2_level_set(golden_dir):
    levels = [int(v) for v in next(_rows(os.path.join(golden_dir, "int2_levels.txt")))]
    assert sorted(set(S(ALL_Q, 2).tolist())) == levels


def test_identity_at_full_width():
    # S(q, c) = q: nothing to round when r = c (both equations).
    assert np.array_equal(S(ALL_Q, 8), ALL_Q.astype(np.int64))
    assert np.array_equal(S(ALL_Q, 8, True), ALL_Q.astype(np.int64))


@pytest.mark.parametrize("r", range(1, 8))
def test_preimage_intervals_closed_form(r):
    # Inverting Eq. 6 by hand: round-half-up sends q to bucket k exactly when
    # k*2^sh - 2^(sh-1) <= q < k*2^sh + 2^(sh-1); the clamp folds bucket 2^r
    # into bucket 2^r - 1; Eq. 8 keeps it.
    sh = 8 - r
    h = 1 << (sh - 1)
    got = S(ALL_Q, r)
    got_ep = S(ALL_Q, r, True)
    for k in range(0, (1 << r) + 1):
        lo = max(0, (k << sh) - h)
        hi = min(255, (k << sh) + h - 1)
        if lo > hi:
            continue
        assert np.all(got_ep[lo:hi + 1] == (k << sh)), (r, k)
        kk = min(k, (1 << r) - 1)
        assert np.all(got[lo:hi + 1] == (kk << sh)), (r, k)


@pytest.mark.parametrize("r", range(1, 9))
def test_checksums_closed_form(r):
    # sum_q q = 32640.  Eq. 8 moves each full bucket's mass by +2^(sh-1) and the
    # two half buckets by -h(h-1)/2 and +h(h+1)/2 (h = 2^(sh-1)): total +2^(c-1),
    # so sum S_EP = 2^15.  The clamp removes 2^sh from each of the 2^(sh-1)
    # overflow codes: sum S = 2^15 - 2^(2 sh - 1).
    sh = 8 - r
    if sh == 0:
        assert S(ALL_Q, r).sum() == 32640 and S(ALL_Q, r, True).sum() == 32640
        return
    assert S(ALL_Q, r, True).sum() == 2 ** 15
    assert S(ALL_Q, r).sum() == 2 ** 15 - 2 ** (2 * sh - 1)
    assert {1: 24576, 2: 30720, 3: 32256, 4: 32640, 5: 32736, 6: 32760, 7: 32766}[r] == S(ALL_Q, r).sum()


def test_bucket_populations():
    # r = 2: 32 / 64 / 64 / 96 codes map to k = 0..3; r = 4: 8, then 16 each, then 24.
    k2 = S(ALL_Q, 2) >> 6
    assert np.bincount(k2, minlength=4).tolist() == [32, 64, 64, 96]
    k4 = S(ALL_Q, 4) >> 4
    assert np.bincount(k4, minlength=16).tolist() == [8] + [16] * 14 + [24]


@pytest.mark.parametrize("r", range(1, 9))
def test_invariants(r):
    sh = 8 - r
    s = S(ALL_Q, r)
    q = ALL_Q.astype(np.int64)
    assert np.all(s % (1 << sh) == 0)
    assert s.min() >= 0 and s.max() <= ((1 << r) - 1) << sh
    assert np.all(np.diff(s) >= 0)                       # monotone in q
    assert np.array_equal(S(s.astype(np.uint8), r), s)   # idempotent
    if sh:
        h = 1 << (sh - 1)
        unclamped = q < 256 - h
        assert np.all(np.abs(q - s)[unclamped] <= h)
        assert np.abs(q - s).max() == (1 << sh) - 1      # q = 255 under the clamp
        # rounding really is "add the (r+1)-th most significant bit" (Appendix A)
        bit = (q >> (sh - 1)) & 1
        trunc = q >> sh
        assert np.array_equal(np.minimum(trunc + bit, (1 << r) - 1) << sh, s)


@pytest.mark.parametrize("r", range(1, 8))
def test_extra_precision_properties(r):
    sh = 8 - r
    h = 1 << (sh - 1)
    q = ALL_Q.astype(np.int64)
    s, e = S(ALL_Q, r), S(ALL_Q, r, True)
    assert len(set(e.tolist())) == (1 << r) + 1          # Errata: 2^r + 1 possible values
    assert set((e - s).tolist()) == {0, 1 << sh}
    assert np.array_equal(e != s, q >= 256 - h)          # overflow <=> q >= 2^c - 2^(sh-1)
    assert (e != s).sum() == h
    assert np.abs(q - e).max() <= h                      # no clamp => never more than half a bucket off
    assert e.max() == 256


def test_tie_rule_is_half_up_and_where_half_even_would_differ():
    # The only codes at which round-half-even would change Eq. 6 are exact
    # ties q = (odd + 1/2) * 2^sh that half-up sends to an odd bucket:
    # r = 2: 32 and 160; r = 3: 16, 80, 144, 208.
    for r, want in [(2, [32, 160]), (3, [16, 80, 144, 208]), (4, list(range(8, 256, 32)))]:
        sh = 8 - r
        q = ALL_Q.astype(np.float64)
        half_even = np.clip(np.rint(q / (1 << sh)), 0, (1 << r) - 1).astype(np.int64) << sh
        diff = np.nonzero(half_even != S(ALL_Q, r))[0].tolist()
        assert diff == want, (r, diff)
    assert S(np.array([32]), 2)[0] == 64 and S(np.array([160]), 2)[0] == 192


def test_slices_come_from_the_full_code_not_from_another_slice():
    # Section 3.2: every precision is sliced from the largest bit-width.  Slicing
    # int4 first and then int2 rounds twice and disagrees on some codes,
    # e.g. q = 24: S(24, 2) = 0 but S(S(24, 4), 2) = S(32, 2) = 64.
    direct = S(ALL_Q, 2)
    twice = S(S(ALL_Q, 4).astype(np.uint8), 2)
    assert direct[24] == 0 and twice[24] == 64
    assert (direct != twice).sum() == 24


def test_bad_arguments():
    st, _ = ref.slice_values(ALL_Q, 0)
    assert st == ref.ERR_UNSUPPORTED
    st, _ = ref.slice_values(ALL_Q, 9)
    assert st == ref.ERR_UNSUPPORTED
    st, _ = ref.slice_values(ALL_Q, 4, c=4)
    assert st == ref.ERR_UNSUPPORTED
