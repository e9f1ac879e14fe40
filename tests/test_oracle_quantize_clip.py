"""Pins for the oracle's Eq. 3 (MinMax quantisation with OmniQuant's clipping scales gamma, beta).

None of the expected values below comes from the code under test: a worked row whose arithmetic is exact, the
reduction to Eq. 1, and properties that follow from the definition (the code is the nearest grid point of the CLIPPED
weight), checked in float64.
"""
import numpy as np

from oracle import ref
from paper_2502_06786_b200 import synth


def _bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_gamma_beta_one_is_eq1():
    W = synth.normal_bf16((37, 512), 0.02, 4242)
    st1, q1, a1, z1 = ref.quantize(W)
    ones = np.ones(37, np.float32)
    for g, b in ((None, None), (ones, None), (None, ones), (ones, ones)):
        st3, q3, a3, z3 = ref.quantize_clip(W, g, b)
        assert st1 == st3 == ref.OK
        assert np.array_equal(q1, q3) and np.array_equal(a1, a3) and np.array_equal(z1, z3)


def test_worked_row_with_exact_arithmetic():
    # w_i = i / 64, i = -128 .. 127 (exact in bf16), gamma = beta = 1/2:
    #   gamma max = 127/128, beta min = -1, alpha = (255/128) / 255 = 1/128, z = 1 / (1/128) = 128,
    #   w/alpha + z = 2 i + 128: an integer, so no rounding anywhere, and the clamp cuts at i <= -64 and i >= 64.
    i = np.arange(-128, 128)
    W = _bits(i / 64.0)[None, :]
    half = np.full(1, 0.5, np.float32)
    st, q, a, z = ref.quantize_clip(W, half, half)
    assert st == ref.OK
    assert a[0] == np.float32(1 / 128) and z[0] == np.float32(128)
    want = np.where(i <= -64, 0, np.where(i >= 64, 255, 2 * i + 128))
    assert q[0].tolist() == want.tolist()
    # beta alone widens or narrows only the lower end: gamma = 1, beta = 1/2 -> alpha = (127/64 + 1) / 255, z = 1 / alpha
    st, q, a, z = ref.quantize_clip(W, None, half)
    alpha = np.float32(np.float32(127 / 64 + 1) / np.float32(255))
    assert a[0] == alpha and z[0] == np.float32(np.float32(1) / alpha)
    assert q[0, -1] == 255 and q[0, 0] == 0 and q[0, 64] == 0 and q[0, 65] == 1        # w = -1 is the new minimum


def test_codes_are_nearest_grid_point_of_the_clipped_weight():
    rng = np.random.default_rng(5)
    N, K = 64, 1024
    W = synth.student_t_bf16((N, K), 3.0, 0.02, 99)
    gamma = rng.uniform(0.3, 1.0, N).astype(np.float32)
    beta = rng.uniform(0.3, 1.0, N).astype(np.float32)
    W[7] = _bits(np.abs(synth.bf16_bits_to_f32(W[7])) + 0.5)     # a same-sign row: beta min > 0, z < 0
    gamma[7], beta[7] = 1.0, 0.5                                  # (keeps gamma max above beta min)
    st, q, a, z = ref.quantize_clip(W, gamma, beta)
    assert st == ref.OK
    w = synth.bf16_bits_to_f32(W).astype(np.float64)
    hi = gamma.astype(np.float64) * w.max(1)
    lo = beta.astype(np.float64) * w.min(1)
    assert np.allclose(a, (hi - lo) / 255.0, rtol=1e-5) and np.allclose(z, -lo / a.astype(np.float64), rtol=1e-5)   # a few fp32 roundings
    deq = a[:, None].astype(np.float64) * (q.astype(np.float64) - z[:, None].astype(np.float64))
    grid_lo = a.astype(np.float64) * (0 - z.astype(np.float64))
    grid_hi = a.astype(np.float64) * (255 - z.astype(np.float64))
    clipped = np.clip(w, grid_lo[:, None], grid_hi[:, None])
    assert np.all(np.abs(deq - clipped) <= 0.5001 * a[:, None] + 1e-7)
    # the clamp really is active, at both ends, and the codes are monotone in the weight
    assert (q == 255).mean() > 1e-3 and (q == 0).mean() > 1e-3
    order = np.argsort(w[3], kind="stable")
    assert np.all(np.diff(q[3][order].astype(int)) >= 0)
    # swapping gamma and beta is a different quantiser
    st, q_sw, a_sw, z_sw = ref.quantize_clip(W, beta, gamma)
    assert not np.array_equal(a, a_sw)


def test_degenerate_and_nonfinite():
    W = synth.normal_bf16((3, 64), 0.02, 1)
    g = np.array([1.0, 0.0, 1.0], np.float32)
    b = np.array([1.0, 0.0, 1.0], np.float32)
    st, q, a, z = ref.quantize_clip(W, g, b)              # row 1: range 0 -> alpha = 1, z = 0, codes round(w) clamped
    assert st == ref.OK and a[1] == 1.0 and z[1] == 0.0 and not q[1].any()
    g[2] = np.inf
    st, _, _, _ = ref.quantize_clip(W, g, b)
    assert st == ref.ERR_NONFINITE
