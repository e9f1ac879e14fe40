"""Pins for the oracle's multi-precision reconstruction loss (Eq. 7 with the L2 loss of Eq. 5 on one linear layer)."""
import numpy as np

from oracle import ref
from paper_2502_06786_b200 import synth


def _bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_hand_value_one_weight():
    # q = 200, alpha = 1/2, z = 10, x = 1:  Y_8 = (200 - 10)/2 = 95;  S(200, 4) = 13 * 16 = 208 -> 99;  S(200, 2) = 3 * 64 -> 91.
    # Target 100: squared errors 25, 1, 81; lambda = (1, 2, 3) -> 25 + 2 + 243 = 270.
    q = np.array([[200]], np.uint8)
    st, L, total, _, _ = ref.gemm_multi_loss(ref.SRC_CODES8, q, 1, _bits([[1.0]]), np.array([[100.0]], np.float32), (1.0, 2.0, 3.0),
                                             alpha=np.array([0.5], np.float32), zero=np.array([10.0], np.float32))
    assert st == ref.OK and L == [25.0, 1.0, 81.0] and total == 270.0


def test_integer_case_against_python_ints():
    # alpha = 1, z = 0, small integer activations: every output is an exact integer.  With the int8 forward as the
    # target, L_8 = 0 and L_r = || X (q - S(q, r))^T ||^2, recomputed here with integer matmuls from Eq. 6 typed out.
    rng = np.random.default_rng(3)
    N, K, M = 24, 64, 10
    q = rng.integers(0, 256, (N, K)).astype(np.uint8)
    x = rng.integers(-4, 5, (M, K))
    one, zer = np.ones(N, np.float32), np.zeros(N, np.float32)
    y8 = x @ q.astype(np.int64).T
    st, L, total, _, _ = ref.gemm_multi_loss(ref.SRC_CODES8, q, K, _bits(x.astype(np.float32)), y8.astype(np.float32), (0.5, 1.0, 2.0),
                                             alpha=one, zero=zer)
    assert st == ref.OK and L[0] == 0.0
    want = []
    for r in (4, 2):
        sh = 8 - r
        S = np.minimum((q.astype(np.int64) + (1 << (sh - 1))) >> sh, (1 << r) - 1) << sh
        d = x @ (q.astype(np.int64) - S).T
        want.append(int((d * d).sum()))
    assert L[1] == float(want[0]) and L[2] == float(want[1])
    assert total == 1.0 * want[0] + 2.0 * want[1]
    assert L[2] > L[1] > 0                                            # coarser slices reconstruct worse


def test_weights_are_linear_and_target_shift_is_quadratic():
    W = synth.normal_bf16((16, 128), 0.02, 77)
    X = synth.normal_bf16((9, 128), 1.0, 78)
    st, Ys, a, z = ref.gemm_multi(ref.SRC_BF16, W, 128, X)
    Yt = Ys[0].astype(np.float32)
    st, L, total, _, _ = ref.gemm_multi_loss(ref.SRC_BF16, W, 128, X, Yt, (1.0, 1.0, 1.0))
    st, L2, total2, _, _ = ref.gemm_multi_loss(ref.SRC_BF16, W, 128, X, Yt, (3.0, 0.0, 0.5))
    assert L == L2 and np.isclose(total, sum(L)) and np.isclose(total2, 3.0 * L[0] + 0.5 * L[2])
    assert L[0] < 1e-9 * L[2]                                         # the target is the int8 forward itself (up to its fp32 rounding)
    # adding a constant d to every target entry adds M N d^2 - 2 d sum(Yt - Y_r) to L_r
    d = 0.25
    st, L3, _, _, _ = ref.gemm_multi_loss(ref.SRC_BF16, W, 128, X, Yt + np.float32(d), (1.0, 1.0, 1.0))
    for r in range(3):
        resid = float((Yt.astype(np.float64) - Ys[r]).sum())
        assert np.isclose(L3[r], L[r] + Yt.size * d * d + 2 * d * resid, rtol=1e-5)      # Yt + d rounds in fp32


def test_co_distillation_hand_values():
    # the one-weight case again: Y_8 = 95, Y_4 = 99, Y_2 = 91, target 100.
    q = np.array([[200]], np.uint8)
    args = (ref.SRC_CODES8, q, 1, _bits([[1.0]]), np.array([[100.0]], np.float32), (1.0, 1.0, 1.0))
    kw = dict(alpha=np.array([0.5], np.float32), zero=np.array([10.0], np.float32))
    st, L, total, _, _ = ref.gemm_multi_loss(*args, teacher=(-1, 0, 0), **kw)          # int8 teaches int4 and int2
    assert L == [25.0, 16.0, 16.0] and total == 57.0
    st, L, total, _, _ = ref.gemm_multi_loss(*args, teacher=(-1, -1, 1), **kw)         # int4 teaches int2: (99 - 91)^2
    assert L == [25.0, 1.0, 64.0]
    both = ref.TEACHER_AND_TARGET
    st, L, total, _, _ = ref.gemm_multi_loss(*args, teacher=(-1, -1, both + 0), **kw)  # target and int8 teacher, equal weights
    assert L == [25.0, 1.0, 81.0 + 16.0]
