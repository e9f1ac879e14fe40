"""Pins for the oracle's dequantised matmuls (the forward F(S(Q(W, c), r), x) of Eq. 7).

The oracle's triple loop is checked against NumPy's fp64 matmul over
explicitly dequantised weights (the textbook form at r = 8 and at every r),
against basis / ones vectors, an all-integer case with a hand-countable
result, linearity, and the extra-precision difference formula.
"""
import numpy as np
import pytest

from oracle import ref
from paper_2502_06786_b200 import synth


def _setup(N=23, K=256, B=3, seed=7, dist="normal"):
    W = synth.normal_bf16((N, K), 0.02, seed) if dist == "normal" else synth.student_t_bf16((N, K), 3.0, 0.02, seed)
    st, q, a, z = ref.quantize(W)
    assert st == ref.OK
    x = synth.normal_bf16((B, K), 1.0, seed + 1)
    return W, q, a, z, x


def _dequant(S, a, z):
    return a.astype(np.float64)[:, None] * (S.astype(np.float64) - z.astype(np.float64)[:, None])


@pytest.mark.parametrize("r", [8, 4, 2])
def test_gemv_is_textbook_dequantised_matmul(r):
    W, q, a, z, x = _setup()
    K = q.shape[1]
    sp = ref.slice_pack(q, r)
    st, y = ref.gemv(sp["packed"], K, r, a, z, x)
    assert st == ref.OK
    _, S = ref.slice_values(q, r)
    want = synth.bf16_bits_to_f32(x).astype(np.float64) @ _dequant(S, a, z).T
    np.testing.assert_allclose(y, want, rtol=1e-12, atol=1e-12)
    if r == 8:
        # r = c: the layer is the plain int8 weight-only linear layer x . (alpha (q - z))^T
        want8 = synth.bf16_bits_to_f32(x).astype(np.float64) @ _dequant(q, a, z).T
        np.testing.assert_allclose(y, want8, rtol=1e-12, atol=1e-12)


def test_basis_and_ones_vectors():
    W, q, a, z, _ = _setup(N=11, K=64)
    K = 64
    sp = ref.slice_pack(q, 4)
    _, S = ref.slice_values(q, 4)
    D = _dequant(S, a, z)
    e = np.zeros((2, K), np.float32); e[0, 17] = 1.0; e[1, :] = 1.0
    st, y = ref.gemv(sp["packed"], K, 4, a, z, synth.f32_to_bf16_bits(e))
    np.testing.assert_allclose(y[0], D[:, 17], rtol=1e-13)       # x = e_j picks column j of the dequantised weights
    np.testing.assert_allclose(y[1], D.sum(1), rtol=1e-12, atol=1e-12)


def test_exact_integer_case_by_hand():
    # alpha = 1, z = 0, fields and x small integers: y is an integer computed with Python ints.
    N, K = 5, 32
    rng = np.random.default_rng(3)
    q = rng.integers(0, 256, (N, K), dtype=np.uint8)
    xi = rng.integers(-4, 5, (2, K))
    a = np.ones(N, np.float32); z = np.zeros(N, np.float32)
    for r in (8, 4, 2):
        sh = 8 - r
        sp = ref.slice_pack(q, r)
        st, y = ref.gemv(sp["packed"], K, r, a, z, synth.f32_to_bf16_bits(xi.astype(np.float32)))
        for b in range(2):
            for n in range(N):
                acc = 0
                for k in range(K):
                    kk = int(q[n, k]) if sh == 0 else min((int(q[n, k]) + (1 << (sh - 1))) >> sh, (1 << r) - 1)
                    acc += int(xi[b, k]) * (kk << sh)
                assert y[b, n] == float(acc)


def test_zero_point_and_scale_enter_as_alpha_times_S_minus_z():
    # One weight, one activation: y = x * alpha * (S - z).  A sign slip in z or a
    # misplaced alpha changes this number.
    q = np.array([[200, 8]], np.uint8)
    a = np.array([0.5], np.float32); z = np.array([3.0], np.float32)
    x = synth.f32_to_bf16_bits(np.array([[2.0, 1.0]], np.float32))
    sp = ref.slice_pack(q, 4)                     # S(200,4) = 13*16 = 208 ; S(8,4) = 1*16 = 16
    st, y = ref.gemv(sp["packed"], 2, 4, a, z, x)
    assert y[0, 0] == 2.0 * 0.5 * (208 - 3.0) + 1.0 * 0.5 * (16 - 3.0)


def test_linearity_in_x():
    W, q, a, z, x = _setup(B=2)
    K = q.shape[1]
    sp = ref.slice_pack(q, 2)
    xf = synth.bf16_bits_to_f32(x)
    comb = synth.f32_to_bf16_bits((2.0 * xf[0] - 0.5 * xf[1])[None, :])   # exact scalings; sum re-rounded to bf16
    combf = synth.bf16_bits_to_f32(comb).astype(np.float64)
    _, y = ref.gemv(sp["packed"], K, 2, a, z, x)
    _, yc = ref.gemv(sp["packed"], K, 2, a, z, comb)
    _, S = ref.slice_values(q, 2)
    np.testing.assert_allclose(yc[0], combf[0] @ _dequant(S, a, z).T, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("r", [4, 2])
def test_extra_precision_difference_formula(r):
    # Eq. 8 minus Eq. 6: y_EP - y = alpha_n 2^sh sum_{j in ovf(n)} x_j
    N, K, B = 9, 128, 2
    q = synth.skewed_codes((N, K), 0.1, 224, 19)
    a = (np.abs(synth.bf16_bits_to_f32(synth.normal_bf16((N,), 1.0, 20))) + 0.1).astype(np.float32)
    z = synth.bf16_bits_to_f32(synth.normal_bf16((N,), 50.0, 21)).astype(np.float32)
    x = synth.normal_bf16((B, K), 1.0, 22)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    ep = ref.slice_pack(q, r, extra_precision=True)
    _, y0 = ref.gemv(ep["packed"], K, r, a, z, x)
    _, y1 = ref.gemv(ep["packed"], K, r, a, z, x, ep["ovf_row_ptr"], ep["ovf_col"])
    thr = 256 - (1 << (8 - r - 1))
    want = (xf @ (q >= thr).astype(np.float64).T) * a.astype(np.float64)[None, :] * (1 << (8 - r))
    np.testing.assert_allclose(y1 - y0, want, rtol=1e-9, atol=1e-9)
    # and equals the dense definition with Eq. 8 values
    _, S_ep = ref.slice_values(q, r, True)
    np.testing.assert_allclose(y1, xf @ _dequant(S_ep, a, z).T, rtol=1e-12, atol=1e-10)


def test_gemm_multi_consistency():
    W, q, a, z, X = _setup(N=17, K=128, B=6)
    K = 128
    st, Ys, a2, z2 = ref.gemm_multi(ref.SRC_BF16, W, K, X)
    assert st == ref.OK and np.array_equal(a, a2) and np.array_equal(z, z2)
    st, Yc, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, X, alpha=a, zero=z)
    for i, r in enumerate((8, 4, 2)):
        sp = ref.slice_pack(q, r)
        _, y = ref.gemv(sp["packed"], K, r, a, z, X)                 # three independent single-precision calls
        assert np.array_equal(Ys[i], y) and np.array_equal(Yc[i], y)
        st, Yp, _, _ = ref.gemm_multi(ref.SRC_PACKED, sp["packed"], K, X, rs=(r,), alpha=a, zero=z)
        assert st == ref.OK and np.array_equal(Yp[0], y)
    # quantisation error shrinks with r: the r = 8 forward is closest to the bf16 forward
    full = synth.bf16_bits_to_f32(X).astype(np.float64) @ synth.bf16_bits_to_f32(W).astype(np.float64).T
    errs = [np.abs(Y - full).mean() for Y in Ys]
    assert errs[0] < errs[1] < errs[2]
    # extra precision through the dense entry point
    ep = ref.slice_pack(q, 2, extra_precision=True)
    st, Ye, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, X, rs=(2,), alpha=a, zero=z, extra_precision=True)
    _, ye = ref.gemv(ep["packed"], K, 2, a, z, X, ep["ovf_row_ptr"], ep["ovf_col"])
    assert np.array_equal(Ye[0], ye)
