"""GPU parity of the multi-precision dense forward (Eq. 7's F(S(Q(W, c), r), x) for every r in R) against the oracle.

Tolerance: max|dY| <= 1e-2 * rms(Y_oracle) per output (tensor-core path); alpha / zero produced by the fused
MinMax quantisation must equal the oracle's as fp32 values; the all-integer case must be exact.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2502_06786_b200 import binding as mq
from paper_2502_06786_b200 import synth
from tests.util import bf16_dev, dev, host, rms, status_word

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _check(Ys, Yr, tol=TOL):
    for yg, yr in zip(Ys, Yr):
        err = np.abs(host(yg) - yr).max()
        assert err <= tol * rms(yr), (err, rms(yr))


@pytest.mark.parametrize("M,N,K", [(200, 264, 256), (128, 128, 64), (1, 8, 64), (384, 512, 1024), (130, 1000, 192)])
def test_codes_source_all_precisions(M, N, K):
    W = synth.normal_bf16((N, K), 0.02, 40 + M)
    st, q, a, z = ref.quantize(W)
    X = synth.normal_bf16((M, K), 1.0, 41 + M)
    status = status_word()
    Ys, _, _ = mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), rs=(8, 4, 2), alpha=dev(a), zero=dev(z), dev_status=status)
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, X, alpha=a, zero=z)
    assert st == ref.OK
    _check(Ys, Yr)
    assert int(host(status)[0]) == mq.OK


def test_bf16_source_quantizes_on_the_fly():
    M, N, K = 160, 392, 512
    W = synth.student_t_bf16((N, K), 3.0, 0.02, 50)
    X = synth.normal_bf16((M, K), 1.0, 51)
    Ys, a, z = mq.gemm_multi(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X))
    st, Yr, ar, zr = ref.gemm_multi(ref.SRC_BF16, W, K, X)
    assert np.array_equal(host(a), ar) and np.array_equal(host(z), zr)
    _check(Ys, Yr)
    # interpolated precisions (r = 6, 3) and a single output
    Ys, _, _ = mq.gemm_multi(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X), rs=(6, 3))
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_BF16, W, K, X, rs=(6, 3))
    _check(Ys, Yr)


@pytest.mark.parametrize("r,ep", [(4, False), (2, False), (2, True), (4, True), (8, False)])
def test_packed_source(r, ep):
    M, N, K = 96, 136, 256
    q = synth.skewed_codes((N, K), 0.05, 224, 60 + r)
    a = (np.abs(synth.bf16_bits_to_f32(synth.normal_bf16((N,), 0.01, 61))) + 1e-3).astype(np.float32)
    z = synth.bf16_bits_to_f32(synth.normal_bf16((N,), 40.0, 62)).astype(np.float32) + 128
    X = synth.normal_bf16((M, K), 1.0, 63)
    sp = ref.slice_pack(q, r, extra_precision=ep)
    rp, col = (sp["ovf_row_ptr"], sp["ovf_col"]) if (ep and r < 8) else (None, None)
    Ys, _, _ = mq.gemm_multi(mq.SRC_PACKED, dev(sp["packed"]), K, bf16_dev(X), rs=(r,), alpha=dev(a), zero=dev(z),
                             extra_precision=ep, ovf_row_ptr=dev(rp) if rp is not None else None,
                             ovf_col=dev(col if col.size else np.zeros(1, np.uint16)) if rp is not None else None)
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_PACKED, sp["packed"], K, X, rs=(r,), alpha=a, zero=z, extra_precision=ep,
                                  ovf_row_ptr=rp, ovf_col=col)
    assert st == ref.OK
    _check(Ys, Yr)
    # the same result from the codes with Eq. 8 applied on the fly
    Yc, _, _ = mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), rs=(r,), alpha=dev(a), zero=dev(z), extra_precision=ep)
    assert torch.equal(Yc[0], Ys[0])


@pytest.mark.parametrize("M,N,K", [(130, 128, 128), (130, 256, 192), (257, 392, 256), (64, 1000, 128), (300, 2056, 64), (33, 136, 64)])
@pytest.mark.parametrize("r,ep", [(4, False), (2, True)])
def test_single_precision_uses_256_channel_tiles(M, N, K, r, ep):
    # one plane only: the CTA takes 256 channels (two adjacent tiles, one N = 256 MMA); ragged N in either half
    W = synth.normal_bf16((N, K), 0.02, 70 + N)
    st, q, a, z = ref.quantize(W)
    if ep:
        q = synth.skewed_codes((N, K), 0.05, 224, 71 + N)
    X = synth.normal_bf16((M, K), 1.0, 72 + M)
    Ys, _, _ = mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), rs=(r,), alpha=dev(a), zero=dev(z), extra_precision=ep)
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, X, rs=(r,), alpha=a, zero=z, extra_precision=ep)
    assert st == ref.OK
    _check(Ys, Yr)


@pytest.mark.parametrize("M,N,K,rs", [(200, 264, 256, (8, 4, 2)), (130, 1000, 192, (8, 4, 2)), (64, 136, 128, (4,)),
                                      (300, 520, 64, (2,)), (1, 8, 64, (8, 2)), (257, 392, 320, (6, 3))])
def test_loss_matches_the_definition(M, N, K, rs):
    # Eq. 7 with the L2 loss of Eq. 5: squared error of every precision against a target, in the GEMM's epilogue
    W = synth.normal_bf16((N, K), 0.02, 80 + M)
    X = synth.normal_bf16((M, K), 1.0, 81 + M)
    Wf = synth.bf16_bits_to_f32(W).astype(np.float64)
    Xf = synth.bf16_bits_to_f32(X).astype(np.float64)
    Yt = (Xf @ Wf.T).astype(np.float32)                      # the unquantised layer's output
    lam = tuple(0.5 + 0.75 * i for i in range(len(rs)))
    st, L_ref, total_ref, a_ref, z_ref = ref.gemm_multi_loss(ref.SRC_BF16, W, K, X, Yt, lam, rs=rs)
    assert st == ref.OK
    status = status_word()
    loss, a, z = mq.gemm_multi_loss(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X), dev(Yt), lam, rs=rs, dev_status=status)
    got = host(loss)
    assert np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref)
    assert np.allclose(got[:-1], L_ref, rtol=2e-3) and np.isclose(got[-1], total_ref, rtol=2e-3), (got, L_ref)
    assert int(host(status)[0]) == mq.OK
    # reproducible bit for bit, and the forward's outputs give the same numbers when differenced on the host
    loss2, _, _ = mq.gemm_multi_loss(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X), dev(Yt), lam, rs=rs)
    assert np.array_equal(host(loss2), got)
    Ys, _, _ = mq.gemm_multi(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X), rs=rs)
    for i, y in enumerate(Ys):
        want = float(((Yt.astype(np.float64) - host(y).astype(np.float64)) ** 2).sum())
        assert np.isclose(got[i], want, rtol=1e-4)


@pytest.mark.parametrize("teacher", [(-1, 0, 0), (-1, -1, 1), (-1, 0, 256), (-1, 256, 257)])
def test_loss_with_co_distillation_targets(teacher):
    M, N, K = 200, 264, 256
    W = synth.normal_bf16((N, K), 0.02, 90)
    X = synth.normal_bf16((M, K), 1.0, 91)
    Yt = (synth.bf16_bits_to_f32(X).astype(np.float64) @ synth.bf16_bits_to_f32(W).astype(np.float64).T).astype(np.float32)
    lam = (1.0, 0.5, 2.0)
    st, L_ref, total_ref, _, _ = ref.gemm_multi_loss(ref.SRC_BF16, W, K, X, Yt, lam, teacher=teacher)
    loss, _, _ = mq.gemm_multi_loss(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X), dev(Yt), lam, teacher=teacher)
    got = host(loss)
    assert np.allclose(got[:-1], L_ref, rtol=2e-3) and np.isclose(got[-1], total_ref, rtol=2e-3), (got, L_ref)
    with pytest.raises(mq.MatqError):
        mq.gemm_multi_loss(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X), dev(Yt), lam, teacher=(-1, 1, 0))   # a precision cannot teach itself


def test_loss_is_zero_against_its_own_int8_forward_in_the_integer_case():
    rng = np.random.default_rng(9)
    N, K, M = 136, 128, 70
    q = rng.integers(0, 256, (N, K)).astype(np.uint8)
    x = rng.integers(-3, 4, (M, K)).astype(np.float32)
    one, zer = np.ones(N, np.float32), np.zeros(N, np.float32)
    y8 = (x.astype(np.int64) @ q.astype(np.int64).T).astype(np.float32)
    loss, _, _ = mq.gemm_multi_loss(mq.SRC_CODES8, dev(q), K, bf16_dev(synth.f32_to_bf16_bits(x)), dev(y8), (1.0, 1.0, 1.0),
                                    alpha=dev(one), zero=dev(zer))
    st, L_ref, total_ref, _, _ = ref.gemm_multi_loss(ref.SRC_CODES8, q, K, synth.f32_to_bf16_bits(x), y8, (1.0, 1.0, 1.0), alpha=one, zero=zer)
    got = host(loss)
    assert got[0] == 0.0 and L_ref[0] == 0.0
    assert np.allclose(got[1:3], L_ref[1:], rtol=1e-5)


def test_exact_integer_case_and_independence_of_outputs():
    # alpha = 1, z = 0, integer activations: every partial sum is an exact fp32 integer
    M, N, K = 128, 128, 512
    q = synth.uniform_codes((N, K), 70)
    X = synth.small_int_bf16((M, K), -4, 4, 71)
    a = np.ones(N, np.float32); z = np.zeros(N, np.float32)
    Ys, _, _ = mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), alpha=dev(a), zero=dev(z))
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, X, alpha=a, zero=z)
    for yg, yr in zip(Ys, Yr):
        assert np.array_equal(host(yg).astype(np.float64), yr)
    # each precision alone gives the same bits as in the fused call
    for i, r in enumerate((8, 4, 2)):
        Y1, _, _ = mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), rs=(r,), alpha=dev(a), zero=dev(z))
        assert torch.equal(Y1[0], Ys[i])


def test_matches_decode_gemv_and_full_path():
    # quantize -> slice_pack -> gemv on M rows one batch at a time == the dense forward
    M, N, K = 8, 256, 512
    W = synth.normal_bf16((N, K), 0.02, 80)
    X = synth.normal_bf16((M, K), 1.0, 81)
    Ys, a, z = mq.gemm_multi(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X))
    q, a2, z2 = mq.quantize(bf16_dev(W))
    assert torch.equal(a, a2) and torch.equal(z, z2)
    for i, r in enumerate((8, 4, 2)):
        sp = mq.slice_pack(q, r)
        y = mq.gemv(sp["packed"], K, r, a, z, bf16_dev(X))
        assert np.abs(host(y) - host(Ys[i])).max() <= 1e-3 * rms(host(y))


def test_a_wait_that_runs_out_is_a_status_not_a_hang():
    # matq_gemm_multi_test_stall: the tensor-core kernel issues none of its copies, so the MMA warp's wait for its first
    # stage and the epilogue's wait for the accumulators run out (bounded in clock cycles).  The kernel must return,
    # report MATQ_ERR_TIMEOUT, store nothing and free its tensor memory; the same context must then serve the same call.
    M, N, K = 200, 264, 256
    W = synth.normal_bf16((N, K), 0.02, 90)
    st, q, a, z = ref.quantize(W)
    X = synth.normal_bf16((M, K), 1.0, 91)
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, X, alpha=a, zero=z)
    status = status_word()
    Ys = [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    assert mq.gemm_multi_test_stall(True) == 0
    try:
        mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), rs=(8, 4, 2), alpha=dev(a), zero=dev(z), Ys=Ys, dev_status=status)
        torch.cuda.synchronize()
    finally:
        assert mq.gemm_multi_test_stall(False) == 1
    assert int(host(status)[0]) == mq.ERR_TIMEOUT
    for y in Ys:
        assert bool(torch.isnan(y).all())               # nothing was stored
    # tensor memory was given back (a CTA that kept its columns would block the next one on its SM)
    status.zero_()
    for _ in range(3):
        Ys2, _, _ = mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), rs=(8, 4, 2), alpha=dev(a), zero=dev(z), dev_status=status)
        _check(Ys2, Yr)
    assert int(host(status)[0]) == mq.OK


def test_argument_errors_and_empty():
    lib = mq._lib
    fake = C.c_void_p(0x1000)
    rs3 = (C.c_int * 3)(8, 4, 2)
    ys = (C.c_void_p * 3)(0x1000, 0x1000, 0x1000)

    def call(src=mq.SRC_CODES8, N=128, K=128, c=8, M=128, ldx=128, rs=rs3, n_r=3, ldy=128, ws=fake, wsb=1 << 30):
        return lib.matq_gemm_multi(src, fake, N, K, c, fake, fake, 0, None, None, fake, M, ldx, rs, n_r, ys, ldy, ws, wsb, None, None)
    assert call(n_r=4) == mq.ERR_INVALID_ARG and call(n_r=0) == mq.ERR_INVALID_ARG
    assert call(src=7) == mq.ERR_INVALID_ARG
    assert call(c=4) == mq.ERR_UNSUPPORTED
    assert call(rs=(C.c_int * 3)(8, 8, 2)) == mq.ERR_INVALID_ARG          # precisions must be distinct
    assert call(rs=(C.c_int * 3)(9, 4, 2)) == mq.ERR_UNSUPPORTED
    assert call(K=100, ldx=104) == mq.ERR_SHAPE and call(N=132, ldy=132) == mq.ERR_SHAPE
    assert call(src=mq.SRC_PACKED, n_r=3) == mq.ERR_INVALID_ARG            # one plane, one precision
    assert call(wsb=16) == mq.ERR_WORKSPACE and call(ws=None) == mq.ERR_WORKSPACE
    assert call(M=0) == mq.OK
    assert mq.gemm_multi_workspace_bytes(mq.SRC_BF16, 128, 128, 128, 3) >= 128 * 128 * (1 + 6) + 512


def _check_rows(Ys_dev, Yr, rows, tol=TOL):
    """Rows `rows` of every device output against the oracle's outputs for exactly those rows of X."""
    idx = torch.as_tensor(rows, device="cuda")
    for yg, yr in zip(Ys_dev, Yr):
        got = host(yg.index_select(0, idx))
        err = np.abs(got - yr).max()
        assert err <= tol * rms(yr), (err, rms(yr))


def test_benchmark_shape_bf16_source_three_precisions():
    # The co-training forward at its benchmark size (W 14336 x 4096, 4096 tokens: 32 x 112 output tiles, 64 K blocks per
    # tile), in the configuration the benchmark times.  The oracle cannot do 1.4e12 flop in test time, so it computes a
    # block of 128 consecutive token rows and 64 seeded random token rows (full K, all channels, all three precisions).
    N, K, M = 14336, 4096, 4096
    W = synth.normal_bf16((N, K), 0.02, synth.seed_for(4, 0))
    X = synth.normal_bf16((M, K), 1.0, synth.seed_for(4, 500))
    Ys, a, z = mq.gemm_multi(mq.SRC_BF16, bf16_dev(W), K, bf16_dev(X))
    rng = np.random.default_rng(4096)
    block = list(range(1920, 2048))                      # straddles nothing special: one whole token tile ...
    block2 = list(range(4000, 4096))                     # ... and the end of the last one
    scattered = sorted(rng.choice(M, size=64, replace=False).tolist())
    for rows in (block, block2 + scattered):
        st, Yr, ar, zr = ref.gemm_multi(ref.SRC_BF16, W, K, np.ascontiguousarray(X[rows]))
        assert st == ref.OK
        assert np.array_equal(host(a), ar) and np.array_equal(host(z), zr)
        _check_rows(Ys, Yr, rows)


def test_benchmark_shape_prefill_from_extra_precision_plane():
    # configs[4] prefill: an extra-precision int2 plane with 5 % of the codes in the extra bucket, 14336 x 3584, 2048 tokens
    N, K, M = 14336, 3584, 2048
    q = synth.skewed_codes((N, K), 0.05, 224, synth.seed_for(5, 0))
    sp = ref.slice_pack(q, 2, extra_precision=True, want_unpacked=False)
    X = synth.normal_bf16((M, K), 1.0, synth.seed_for(5, 500))
    a = np.full(N, 1e-3, np.float32); z = np.full(N, 128.0, np.float32)
    Ys, _, _ = mq.gemm_multi(mq.SRC_PACKED, dev(sp["packed"]), K, bf16_dev(X), rs=(2,), alpha=dev(a), zero=dev(z), extra_precision=True,
                             ovf_row_ptr=dev(sp["ovf_row_ptr"]), ovf_col=dev(sp["ovf_col"]))
    rng = np.random.default_rng(2048)
    rows = list(range(1024, 1152)) + sorted(rng.choice(M, size=64, replace=False).tolist())
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_PACKED, sp["packed"], K, np.ascontiguousarray(X[rows]), rs=(2,), alpha=a, zero=z,
                                  extra_precision=True, ovf_row_ptr=sp["ovf_row_ptr"], ovf_col=sp["ovf_col"])
    assert st == ref.OK
    _check_rows(Ys, Yr, rows)
