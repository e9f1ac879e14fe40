"""Pins for the oracle's MinMax quantizer (Eq. 1) and plane packing.

Expected values are hand-worked rows whose fp32 arithmetic is exact, the
properties Eq. 1 forces (row minimum -> 0, maximum -> 2^c - 1, half-step
round-trip error), an fp64 re-evaluation, and hand-written byte patterns.
"""
import numpy as np
import pytest

from oracle import ref
from paper_2502_06786_b200 import synth


def bf16(vals):
    return synth.f32_to_bf16_bits(np.asarray(vals, dtype=np.float32))


def test_hand_row_alpha_one_zero_point_zero_pins_half_up():
    # Row contains 0 and 255 => alpha = 255/255 = 1, z = 0, q = round_half_up(w).
    # 0.5, 1.5, 2.5 are exact in bf16; half-even would give 0, 2, 2.
    w = [0.0, 255.0, 0.5, 1.5, 2.5, 3.25, 100.0, 126.5, 17.75, 0.25]
    st, q, a, z = ref.quantize(bf16([w]))
    assert st == ref.OK and a[0] == 1.0 and z[0] == 0.0
    assert q[0].tolist() == [0, 255, 1, 2, 3, 3, 100, 127, 18, 0]


def test_hand_row_signed_range():
    # Row spanning [-128, 127] => alpha = 1, z = 128, q = w + 128.
    w = np.array([[-128.0, 127.0, 0.0, -1.0, 1.0, 64.0, -64.5, 63.5]], np.float32)
    st, q, a, z = ref.quantize(bf16(w))
    assert st == ref.OK and a[0] == 1.0 and z[0] == 128.0
    assert q[0].tolist() == [0, 255, 128, 127, 129, 192, 64, 192]   # -64.5+128=63.5->64; 63.5+128=191.5->192


def test_hand_row_scaled():
    # Range 0..510 => alpha = 2, z = 0: w = 3 -> 1.5 -> 2, w = 1 -> 0.5 -> 1, w = 253 -> 126.5 -> 127.
    st, q, a, z = ref.quantize(bf16([[0.0, 510.0, 3.0, 1.0, 253.0, 4.0]]))
    assert st == ref.OK and a[0] == 2.0 and z[0] == 0.0
    assert q[0].tolist() == [0, 255, 2, 1, 127, 2]


def test_constant_row_and_same_sign_row():
    st, q, a, z = ref.quantize(bf16([[0.75] * 8, [2.0, 3.0, 2.5, 2.0, 3.0, 2.25, 2.75, 2.5]]))
    assert st == ref.OK
    assert a[0] == 1.0 and z[0] == -0.75 and np.all(q[0] == 0)     # alpha := 1, dequant = 0.75 exactly
    assert 1.0 * (0 - z[0]) == 0.75
    assert z[1] < 0                                                 # real-valued z outside [0, 255]
    assert q[1, 0] == 0 and q[1, 1] == 255


def test_nonfinite_is_reported():
    w = np.zeros((3, 16), np.float32); w[1, 5] = np.inf
    st, *_ = ref.quantize(bf16(w))
    assert st == ref.ERR_NONFINITE
    w[1, 5] = np.nan
    st, *_ = ref.quantize(bf16(w))
    assert st == ref.ERR_NONFINITE


@pytest.mark.parametrize("dist", ["normal", "student"])
def test_properties_on_random_weights(dist):
    N, K = 37, 1000
    W = (synth.normal_bf16((N, K), 0.02, 11) if dist == "normal"
         else synth.student_t_bf16((N, K), 3.0, 0.02, 12))
    st, q, a, z = ref.quantize(W)
    assert st == ref.OK
    w = synth.bf16_bits_to_f32(W).astype(np.float64)
    # Eq. 1: alpha = (max - min) / 255, z = -min / alpha
    np.testing.assert_allclose(a, (w.max(1) - w.min(1)) / 255.0, rtol=1e-6)
    np.testing.assert_allclose(z, -w.min(1) / a.astype(np.float64), rtol=1e-6)
    rows = np.arange(N)
    assert np.all(q[rows, w.argmin(1)] == 0) and np.all(q[rows, w.argmax(1)] == 255)
    # round trip: no clamp is active in pure min-max, so the error is half a step
    deq = a[:, None].astype(np.float64) * (q.astype(np.float64) - z[:, None])
    assert np.all(np.abs(w - deq) <= a[:, None] * (0.5 + 1e-3))
    # fp64 evaluation of Eq. 1 agrees except within rounding noise of a tie, and then by 1
    u = w / a[:, None].astype(np.float64) + z[:, None].astype(np.float64)
    q64 = np.clip(np.floor(u + 0.5), 0, 255)
    d = q.astype(np.int64) - q64.astype(np.int64)
    assert np.abs(d).max() <= 1
    near_tie = np.abs((u - np.floor(u)) - 0.5) < 1e-3
    assert np.all(near_tie[d != 0])
    assert (d != 0).mean() < 1e-3
    # sliced round trip: |w - alpha (S - z)| <= alpha (1/2 + 2^(sh-1)) where the clamp is inactive
    for r in (4, 2):
        sh = 8 - r
        _, S = ref.slice_values(q, r)
        deq_r = a[:, None].astype(np.float64) * (S.astype(np.float64) - z[:, None])
        ok = q < 256 - (1 << (sh - 1))
        assert np.all(np.abs(w - deq_r)[ok] <= a[:, None].repeat(K, 1)[ok] * (0.5 + (1 << (sh - 1)) + 1e-3))


def test_fp32_step_order_matches_numpy_float32():
    # Same single-precision steps evaluated by NumPy's IEEE float32 ops: guards
    # against the C build contracting into FMAs or using a reciprocal.
    W = synth.normal_bf16((16, 512), 0.02, 13)
    st, q, a, z = ref.quantize(W)
    w = synth.bf16_bits_to_f32(W)
    mn, mx = w.min(1), w.max(1)
    a32 = ((mx - mn) / np.float32(255.0)).astype(np.float32)
    z32 = ((-mn) / a32).astype(np.float32)
    u = (w / a32[:, None]).astype(np.float32) + z32[:, None]
    fl = np.floor(u)
    q32 = np.clip(fl + ((u - fl) >= np.float32(0.5)), 0, 255).astype(np.uint8)
    assert np.array_equal(a, a32) and np.array_equal(z, z32) and np.array_equal(q, q32)


# ------------------------------------------------------------------ packing

def test_pack_hand_patterns():
    # fields 0,1,2,3 repeated at r = 2 -> every byte 0b11100100 = 0xE4 (element 0 in the low bits)
    q = np.tile(np.array([0, 64, 128, 192], np.uint8), (2, 8))
    out = ref.slice_pack(q, 2)
    assert out["status"] == ref.OK and out["packed"].shape == (2, 8)
    assert np.all(out["packed"] == 0xE4)
    # fields 0..15 at r = 4 -> 0x10, 0x32, ..., 0xFE
    q = (np.arange(16, dtype=np.uint8) * 16)[None, :]
    out = ref.slice_pack(q, 4)
    assert out["packed"][0].tolist() == [0x10, 0x32, 0x54, 0x76, 0x98, 0xBA, 0xDC, 0xFE]
    # r = 8: the plane is the code tensor
    q = synth.uniform_codes((3, 40), 5)
    assert np.array_equal(ref.slice_pack(q, 8)["packed"], q)


@pytest.mark.parametrize("r", [8, 4, 2])
def test_pack_roundtrip_and_size(r):
    N, K = 9, 264
    q = synth.uniform_codes((N, K), 21)
    out = ref.slice_pack(q, r)
    assert out["packed"].shape == (N, K * r // 8)
    st, fields = ref.unpack(out["packed"], K, r)
    _, S = ref.slice_values(q, r)
    assert st == ref.OK
    assert np.array_equal(fields.astype(np.int64) << (8 - r), S.astype(np.int64))
    assert np.array_equal(out["sliced"].astype(np.int64), S.astype(np.int64))


def test_pack_shape_errors():
    q = synth.uniform_codes((2, 7), 3)
    assert ref.slice_pack(q, 4)["status"] == ref.ERR_SHAPE
    assert ref.slice_pack(q, 2)["status"] == ref.ERR_SHAPE
    assert ref.slice_pack(q, 3, want_packed=False)["status"] == ref.OK   # any 1 <= r <= 8 unpacked
    assert ref.slice_pack(q, 0, want_packed=False)["status"] == ref.ERR_UNSUPPORTED


@pytest.mark.parametrize("r", [4, 2])
def test_extra_precision_lists(r):
    N, K = 13, 512
    q = synth.uniform_codes((N, K), 31)
    q[4, :] = 0                      # a row with no overflow
    q[7, :] = 255                    # a row that overflows everywhere
    std = ref.slice_pack(q, r)
    ep = ref.slice_pack(q, r, extra_precision=True)
    assert ep["status"] == ref.OK
    assert np.array_equal(ep["packed"], std["packed"])        # base plane identical to the standard plane
    thr = 256 - (1 << (8 - r - 1))
    rp, col = ep["ovf_row_ptr"], ep["ovf_col"]
    assert rp[0] == 0 and rp[N] == ep["ovf_count"] == int((q >= thr).sum()) == col.size
    for n in range(N):
        want = np.nonzero(q[n] >= thr)[0]
        got = col[rp[n]:rp[n + 1]]
        assert np.array_equal(got, want)
        assert np.all(np.diff(got.astype(np.int64)) > 0)
    assert rp[5] - rp[4] == 0 and rp[8] - rp[7] == K
    # capacity too small: count still reported
    small = ref.slice_pack(q, r, extra_precision=True, ovf_capacity=10)
    assert small["status"] == ref.ERR_CAPACITY and small["ovf_count"] == ep["ovf_count"]


def test_avg_bits_accounting(golden_dir):
    # Errata: one extra bit per weight in the extra bucket.  On uniform codes the
    # overflow fraction is 2^(sh-1)/256 = 2^-(r+1): 2.125 bits at r = 2, 4.03125 at r = 4.
    q = synth.uniform_codes((64, 4096), 41)
    for r in (2, 4):
        ep = ref.slice_pack(q, r, extra_precision=True)
        avg = r + ep["ovf_count"] / q.size
        assert abs(avg - (r + 2.0 ** -(r + 1))) < 2e-3
    # r = c: no overflow possible (Table 7 lists exactly 8 bits for int8)
    assert ref.slice_pack(q, 8, extra_precision=True)["ovf_count"] == 0
    # a code histogram with 5 % of its mass in the top bucket reproduces Table 7's ~2.05 bits
    qs = synth.skewed_codes((64, 4096), 0.05, 224, 42)
    ep = ref.slice_pack(qs, 2, extra_precision=True)
    avg = 2 + ep["ovf_count"] / qs.size
    with open(golden_dir + "/avg_bits_table7.txt") as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    paper = [float(v) for v in rows[0][1:]]
    assert rows[0][0] == "2" and min(paper) - 5e-3 < avg < max(paper) + 5e-3
