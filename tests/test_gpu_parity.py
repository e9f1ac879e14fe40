"""GPU parity: every CUDA entry point against the CPU oracle on the same seeded inputs.

Integer outputs (codes, slices, packed bytes, overflow lists) must match bit
for bit; alpha and z must be equal as fp32 values; y must satisfy
max|dy| <= 1e-3 * rms(y_oracle) on the fp32 FMA path.
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2502_06786_b200 import binding as mq
from paper_2502_06786_b200 import synth
from tests.util import bf16_dev, dev, host, rms, status_word

pytestmark = pytest.mark.gpu

TOL_FMA = 1e-3      # max|dy| / rms(y) on the fp32 FMA path
TOL_TENSOR = 1e-2   # ... on the tensor-core path (bf16 x bf16 -> fp32 MMA with the 128-offset trick)
# Integer tensor path (B = 1): the weights side and the sums are exact; an activation is rounded to an absolute
# 2^-24 of its column's largest at worst, and the fp32 epilogue cancels alpha*2^sh*sum(x k) against alpha*z*sum(x)
# (about 2^6 above the result at 2^-24 each; more when one activation dominates sum(x)).  Both stay below 1e-4 of rms(y).
TOL_INT8 = 1e-4


# ------------------------------------------------------------------ quantize

@pytest.mark.parametrize("N,K,dist", [(1, 16, "normal"), (37, 1024, "normal"), (300, 2304, "normal"),
                                      (64, 4096, "student"), (5, 14336, "normal"), (19, 1000, "normal"),
                                      (7, 24, "student"), (3, 65536, "normal")])
def test_quantize_bit_exact(N, K, dist):
    W = synth.normal_bf16((N, K), 0.02, 100 + N) if dist == "normal" else synth.student_t_bf16((N, K), 3.0, 0.02, 200 + N)
    st, q_ref, a_ref, z_ref = ref.quantize(W)
    assert st == ref.OK
    status = status_word()
    q, a, z = mq.quantize(bf16_dev(W), dev_status=status)
    assert np.array_equal(host(q), q_ref)
    assert np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref)
    assert int(host(status)[0]) == mq.OK


def test_quantize_special_rows_and_strided_input():
    K = 256
    W = synth.normal_bf16((6, K), 0.02, 7)
    Wf = synth.bf16_bits_to_f32(W).copy()
    Wf[1, :] = 0.375                      # constant row: alpha = 1, z = -0.375, codes 0
    Wf[2, :] = np.abs(Wf[2, :]) + 1.0     # same-sign row: z < 0
    Wf[3, :] = 0.0                        # all-zero row
    Wf[4, :8] = [0.0, 255.0, 0.5, 1.5, 2.5, 126.5, 3.25, 17.75]   # alpha = 1 ties round up
    Wf[4, 8:] = 1.0
    W = synth.f32_to_bf16_bits(Wf)
    st, q_ref, a_ref, z_ref = ref.quantize(W)
    q, a, z = mq.quantize(bf16_dev(W))
    assert np.array_equal(host(q), q_ref) and np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref)
    assert host(q)[4, :8].tolist() == [0, 255, 1, 2, 3, 127, 3, 18]
    # row stride larger than K (a view into a wider matrix), and alpha / z only
    wide = torch.zeros((6, K + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = bf16_dev(W)
    q2, a2, z2 = mq.quantize(wide[:, :K])
    assert np.array_equal(host(q2), q_ref) and np.array_equal(host(a2), a_ref)
    q3, a3, z3 = mq.quantize(bf16_dev(W), want_codes=False)
    assert q3 is None and np.array_equal(host(a3), a_ref) and np.array_equal(host(z3), z_ref)


def test_quantize_bit_exact_over_many_scales_and_offsets():
    # Rows with very different ranges and offsets: zero-centred, same-sign (z far outside [0, 255], up to the point where
    # the kernel must leave its fast path), tiny and huge scales, and many exact ties (weights on a coarse grid).
    rng = np.random.default_rng(123)
    N, K = 4096, 512
    base = synth.bf16_bits_to_f32(synth.normal_bf16((N, K), 1.0, 314)).astype(np.float64)
    scale = 10.0 ** rng.uniform(-6, 4, size=(N, 1))
    offset = np.where(rng.random((N, 1)) < 0.5, 0.0, 10.0 ** rng.uniform(-2, 7, size=(N, 1))) * scale
    Wf = base * scale + offset
    Wf[::7] = np.round(base[::7] * 8) / 8                 # coarse grid: u lands on exact halves often
    Wf[::11] = np.round(base[::11] * 2) * 0.5 + 1000.0
    W = synth.f32_to_bf16_bits(Wf.astype(np.float32))
    st, q_ref, a_ref, z_ref = ref.quantize(W)
    assert st == ref.OK
    q, a, z = mq.quantize(bf16_dev(W))
    assert np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref)
    assert np.array_equal(host(q), q_ref)
    assert np.abs(z_ref).max() > 2 ** 21                   # some rows did take the pinned path


def test_quantize_bit_exact_on_every_bf16_numerator():
    # The register kernel replaces the IEEE division by FMA corrections; this walks EVERY bf16 value between a row's
    # extremes (8192 consecutive bit patterns per sign) for 256 different scales, alphas with all-ones and near-all-ones
    # significands among them, so a quotient that is one ulp off anywhere would move a code.
    rng = np.random.default_rng(7)
    N, K = 256, 16384
    W = np.empty((N, K), dtype=np.uint16)
    for n in range(N):
        top = int(rng.integers(0x2000, 0x5f00))                 # largest magnitude's bit pattern (about 1e-19 .. 1e19)
        mags = np.arange(top - K // 2 + 1, top + 1, dtype=np.uint16)
        W[n, : K // 2] = mags
        W[n, K // 2:] = mags | 0x8000
        if n % 4 == 1:
            W[n, K // 2:] = mags[rng.integers(0, K // 2, K // 2)]   # same-sign row: another alpha, large z
    st, q_ref, a_ref, z_ref = ref.quantize(W)
    assert st == ref.OK
    q, a, z = mq.quantize(bf16_dev(W))
    assert np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref)
    assert np.array_equal(host(q), q_ref)


@pytest.mark.parametrize("N,K,dist", [(9216, 2304, "normal"), (300, 9216, "student"), (64, 4096, "student"), (33, 16384, "normal"),
                                      (19, 1000, "normal"), (7, 72, "student"), (2304, 9216, "normal"), (6, 77, "normal"), (9, 32768, "student")])
def test_quantize_clip_bit_exact(N, K, dist):
    # Eq. 3: per-channel clipping scales; every kernel variant (register, shared-memory and scalar paths) against the oracle
    W = synth.normal_bf16((N, K), 0.02, 900 + N) if dist == "normal" else synth.student_t_bf16((N, K), 3.0, 0.02, 950 + N)
    rng = np.random.default_rng(N + K)
    gamma = rng.uniform(0.4, 1.0, N).astype(np.float32)
    beta = rng.uniform(0.4, 1.0, N).astype(np.float32)
    gamma[::5] = 1.0
    beta[1::7] = 1.0
    if N > 4:
        gamma[2], beta[2] = 0.0, 0.0                     # degenerate range: alpha = 1
        gamma[3], beta[3] = 1.5, 1.25                    # scales above 1 widen the range
    st, q_ref, a_ref, z_ref = ref.quantize_clip(W, gamma, beta)
    assert st == ref.OK
    status = status_word()
    q, a, z = mq.quantize(bf16_dev(W), gamma=dev(gamma), beta=dev(beta), dev_status=status)
    assert np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref)
    assert np.array_equal(host(q), q_ref)
    assert int(host(status)[0]) == mq.OK
    assert (q_ref == 255).any() and (q_ref == 0).any()
    # only one of the two scales
    st, q_ref, a_ref, z_ref = ref.quantize_clip(W, None, beta)
    q, a, z = mq.quantize(bf16_dev(W), beta=dev(beta))
    assert np.array_equal(host(q), q_ref) and np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref)


def test_quantize_clip_on_every_bf16_numerator_and_nonfinite_scale():
    rng = np.random.default_rng(11)
    N, K = 64, 16384
    W = np.empty((N, K), dtype=np.uint16)
    for n in range(N):
        top = int(rng.integers(0x3000, 0x4f00))
        mags = np.arange(top - K // 2 + 1, top + 1, dtype=np.uint16)
        W[n, : K // 2] = mags
        W[n, K // 2:] = mags | 0x8000
    gamma = rng.uniform(0.05, 1.0, N).astype(np.float32)
    beta = rng.uniform(0.05, 1.0, N).astype(np.float32)
    st, q_ref, a_ref, z_ref = ref.quantize_clip(W, gamma, beta)
    q, a, z = mq.quantize(bf16_dev(W), gamma=dev(gamma), beta=dev(beta))
    assert np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref) and np.array_equal(host(q), q_ref)
    gamma[5] = np.nan
    status = status_word()
    mq.quantize(bf16_dev(W), gamma=dev(gamma), beta=dev(beta), dev_status=status)
    assert int(host(status)[0]) == mq.ERR_NONFINITE


def test_quantize_reports_nonfinite_without_trapping():
    Wf = synth.bf16_bits_to_f32(synth.normal_bf16((4, 128), 0.02, 9)).copy()
    Wf[2, 77] = np.inf
    status = status_word()
    mq.quantize(bf16_dev(synth.f32_to_bf16_bits(Wf)), dev_status=status)
    assert int(host(status)[0]) == mq.ERR_NONFINITE
    Wf[2, 77] = np.nan
    status = status_word()
    mq.quantize(bf16_dev(synth.f32_to_bf16_bits(Wf)), dev_status=status)
    assert int(host(status)[0]) == mq.ERR_NONFINITE
    # the context is still usable
    q, a, z = mq.quantize(bf16_dev(synth.normal_bf16((4, 128), 0.02, 9)))
    assert host(q).shape == (4, 128)


# ---------------------------------------------------------------- slice/pack

@pytest.mark.parametrize("r", range(1, 9))
def test_slice_all_256_codes_every_r(r):
    q = np.tile(np.arange(256, dtype=np.uint8), (3, 1))
    out = mq.slice_pack(dev(q), r, want_packed=False, want_unpacked=True)
    _, S = ref.slice_values(q, r)
    assert np.array_equal(host(out["sliced"]).astype(np.uint16), S)


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("N,K", [(1, 16), (33, 2304), (129, 4096), (7, 1000), (5, 24), (0, 64)])
def test_pack_bit_exact(r, N, K):
    q = synth.uniform_codes((N, K), 300 + N + r)
    out = mq.slice_pack(dev(q), r, want_unpacked=True)
    want = ref.slice_pack(q, r)
    assert want["status"] == ref.OK
    assert np.array_equal(host(out["packed"]), want["packed"])
    assert np.array_equal(host(out["sliced"]), want["sliced"])


@pytest.mark.parametrize("r", [4, 2])
@pytest.mark.parametrize("N,K,p", [(64, 2304, 0.05), (1500, 512, 0.125), (9, 1000, 0.3), (40, 4096, 0.0), (33, 16384, 0.05),
                                   (17, 9216, 0.5), (12, 32768, 0.02), (10, 16, 0.3), (9216, 2304, 0.005), (4099, 256, 0.1)])
def test_extra_precision_lists_bit_exact(r, N, K, p):
    q = synth.skewed_codes((N, K), p, 224, 400 + N) if p > 0 else synth.uniform_codes((N, K), 1) // 2
    if N > 8:
        q[3, :] = 255     # a full row
        q[5, :] = 0       # an empty row
    status = status_word()
    out = mq.slice_pack(dev(q), r, extra_precision=True, dev_status=status)
    want = ref.slice_pack(q, r, extra_precision=True)
    cnt = int(host(out["ovf_count"])[0])
    assert cnt == want["ovf_count"]
    assert np.array_equal(host(out["packed"]), want["packed"])
    assert np.array_equal(host(out["ovf_row_ptr"]), want["ovf_row_ptr"])
    assert np.array_equal(host(out["ovf_col"])[:cnt], want["ovf_col"])
    assert int(host(status)[0]) == mq.OK
    # standard plane == E.P. base plane
    std = mq.slice_pack(dev(q), r)
    assert torch.equal(std["packed"], out["packed"])


@pytest.mark.parametrize("ep", [True, False])
@pytest.mark.parametrize("N,K,p", [(64, 2304, 0.05), (1500, 512, 0.125), (9, 1000, 0.3), (40, 4096, 0.0), (33, 16384, 0.05),
                                   (12, 32768, 0.02), (10, 16, 0.3), (9216, 2304, 0.005), (4099, 256, 0.1), (7, 20, 0.2)])
def test_slice_pack_nested_bit_exact(N, K, p, ep):
    # the int4 and the int2 plane (+ Eq. 8 lists) from one read of the codes: the bits of the two single calls and of
    # the oracle; shapes the one-pass kernel takes, and shapes that fall back to two calls (K % 16 != 0, K > 16384)
    q = synth.skewed_codes((N, K), p, 224, 900 + N) if p > 0 else synth.uniform_codes((N, K), 1) // 2
    if N > 8:
        q[3, :] = 255
        q[5, :] = 0
    status = status_word()
    out = mq.slice_pack_nested(dev(q), extra_precision=ep, dev_status=status)
    want4 = ref.slice_pack(q, 4)
    want2 = ref.slice_pack(q, 2, extra_precision=ep)
    assert np.array_equal(host(out["packed4"]), want4["packed"])
    assert np.array_equal(host(out["packed2"]), want2["packed"])
    if ep:
        cnt = int(host(out["ovf_count"])[0])
        assert cnt == want2["ovf_count"]
        assert np.array_equal(host(out["ovf_row_ptr"]), want2["ovf_row_ptr"])
        assert np.array_equal(host(out["ovf_col"])[:cnt], want2["ovf_col"])
    assert int(host(status)[0]) == mq.OK


def test_slice_pack_nested_argument_errors():
    q = dev(synth.uniform_codes((8, 64), 3))
    p4 = torch.empty((8, 32), dtype=torch.uint8, device="cuda")
    st = mq._lib.matq_slice_pack_nested(q.data_ptr(), 8, 64, 8, p4.data_ptr(), None, 0, None, None, 0, None, None, None)
    assert st == mq.ERR_INVALID_ARG
    out = mq.slice_pack_nested(dev(synth.uniform_codes((8, 6), 3)), raise_on_error=False)
    assert out["status"] == mq.ERR_SHAPE


def test_extra_precision_capacity_error_is_a_status():
    q = synth.skewed_codes((32, 512), 0.2, 224, 77)
    want = ref.slice_pack(q, 2, extra_precision=True)
    status = status_word()
    out = mq.slice_pack(dev(q), 2, extra_precision=True, ovf_capacity=16, dev_status=status)
    assert int(host(out["ovf_count"])[0]) == want["ovf_count"] > 16
    assert int(host(status)[0]) == mq.ERR_CAPACITY
    assert np.array_equal(host(out["ovf_row_ptr"]), want["ovf_row_ptr"])
    # r = c: no overflow, count forced to 0
    cnt = torch.full((1,), 5, dtype=torch.int64, device="cuda")
    mq.slice_pack(dev(q), 8, extra_precision=True, ovf_count=cnt)
    assert int(host(cnt)[0]) == 0


@pytest.mark.parametrize("nested", [False, True])
def test_a_look_back_that_runs_out_is_a_status_not_a_hang(nested):
    # matq_slice_pack_test_stall: the first tile of the one-pass kernel never publishes its overflow count, so the
    # look-back of every later tile meets "nothing yet" until its (shortened) limit or the mark of a tile that gave up.
    # The call must return, report MATQ_ERR_TIMEOUT and still write the planes; the next call must be bit-exact.
    N, K = 9216, 2304
    q = synth.skewed_codes((N, K), 0.005, 224, 1234)
    want2 = ref.slice_pack(q, 2, extra_precision=True)
    qd = dev(q)
    status = status_word()
    call = (lambda: mq.slice_pack_nested(qd, extra_precision=True, dev_status=status)) if nested else \
           (lambda: mq.slice_pack(qd, 2, extra_precision=True, dev_status=status))
    assert mq.slice_pack_test_stall(True) == 0
    try:
        out = call()
        torch.cuda.synchronize()
    finally:
        assert mq.slice_pack_test_stall(False) == 1
    assert int(host(status)[0]) == mq.ERR_TIMEOUT
    assert np.array_equal(host(out["packed2" if nested else "packed"]), want2["packed"])      # the planes do not wait for anything
    if nested:
        assert np.array_equal(host(out["packed4"]), ref.slice_pack(q, 4)["packed"])
    status.zero_()
    out = call()
    cnt = int(host(out["ovf_count"])[0])
    assert cnt == want2["ovf_count"]
    assert np.array_equal(host(out["ovf_row_ptr"]), want2["ovf_row_ptr"])
    assert np.array_equal(host(out["ovf_col"])[:cnt], want2["ovf_col"])
    assert int(host(status)[0]) == mq.OK


# ---------------------------------------------------------------------- gemv

def _gemv_case(N, K, B, r, seed, ep=False, flags=0):
    W = synth.normal_bf16((N, K), 0.02, seed)
    st, q, a, z = ref.quantize(W)
    if ep:
        q = synth.skewed_codes((N, K), 0.05, 224, seed + 5)
    x = synth.normal_bf16((B, K), 1.0, seed + 1)
    sp = ref.slice_pack(q, r, extra_precision=ep)
    rp = sp["ovf_row_ptr"] if ep else None
    col = sp["ovf_col"] if ep else None
    st, y_ref = ref.gemv(sp["packed"], K, r, a, z, x, rp, col)
    assert st == ref.OK
    y = mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x),
                ovf_row_ptr=dev(rp) if ep else None,
                ovf_col=dev(col if col.size else np.zeros(1, np.uint16)) if ep else None, flags=flags)
    return host(y), y_ref


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("N,K,B", [(1024, 1024, 1), (300, 2304, 1), (130, 9216, 8), (77, 3584, 4), (3, 128, 16),
                                   (257, 14336, 3), (64, 256, 5)])
def test_gemv_cuda_core_within_tolerance(r, N, K, B):
    y, y_ref = _gemv_case(N, K, B, r, 500 + N + r, flags=mq.GEMV_CUDA_CORE)
    assert np.abs(y - y_ref).max() <= TOL_FMA * rms(y_ref)


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("N,K,B", [(1024, 1024, 1), (300, 2304, 1), (130, 9216, 8), (77, 3584, 4), (3, 128, 16),
                                   (257, 14336, 3), (64, 256, 5), (2304, 9216, 8), (500, 2432, 11), (129, 384, 2)])
def test_gemv_tensor_within_tolerance(r, N, K, B):
    y, y_ref = _gemv_case(N, K, B, r, 500 + N + r, flags=mq.GEMV_TENSOR)
    assert np.abs(y - y_ref).max() <= TOL_TENSOR * rms(y_ref)


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("N,K", [(1024, 1024), (300, 2304), (130, 9216), (77, 3584), (3, 128), (257, 14336), (64, 256),
                                 (2304, 9216), (500, 2432), (129, 384), (9216, 2304), (128, 128), (40000, 128),
                                 (5000, 256), (33, 32768), (20000, 384)])
def test_gemv_int8_tensor_within_tolerance(r, N, K):
    # u8 x u8 -> s32 MMAs; every K split (1 .. 32 warps), one and two m-tiles, several staging passes (K = 32768)
    y, y_ref = _gemv_case(N, K, 1, r, 500 + N + r, flags=mq.GEMV_TENSOR_INT8)
    assert np.abs(y - y_ref).max() <= TOL_INT8 * rms(y_ref)


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("kind", ["zero", "outlier", "large", "small", "one_hot"])
def test_gemv_int8_tensor_activation_ranges(r, kind):
    # The integer path scales the activations by a power of two taken from their largest magnitude: vectors that
    # are all zero, that hold one element 2^12 times the rest, that are scaled by 2^40 or 2^-40, or that are a unit vector.
    N, K, B = 200, 1024, 1
    W = synth.normal_bf16((N, K), 0.02, 4100 + r)
    _, q, a, z = ref.quantize(W)
    xf = synth.bf16_bits_to_f32(synth.normal_bf16((B, K), 1.0, 4200 + r)).copy()
    if kind == "zero":
        xf[0, :] = 0.0
    elif kind == "outlier":
        xf[:, 17] *= 4096.0
    elif kind == "large":
        xf *= 2.0 ** 40
    elif kind == "small":
        xf *= 2.0 ** -40
    else:
        xf[:] = 0.0
        xf[0, K - 1] = -3.0
    x = synth.f32_to_bf16_bits(xf)
    sp = ref.slice_pack(q, r)
    _, y_ref = ref.gemv(sp["packed"], K, r, a, z, x)
    y = host(mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x), flags=mq.GEMV_TENSOR_INT8))
    for b in range(B):
        assert np.abs(y[b] - y_ref[b]).max() <= TOL_INT8 * max(rms(y_ref[b]), 1e-300), (kind, b)


@pytest.mark.parametrize("r", [8, 4, 2])
def test_gemv_int8_tensor_exact_integer_case(r):
    # alpha = 1, z = 0, small integer x: the scaled activations are exact integers, the sums are integer sums.
    N, K, B = 70, 512, 1
    q = synth.uniform_codes((N, K), 720 + r)
    x = synth.small_int_bf16((B, K), -4, 4, 721)
    a = np.ones(N, np.float32); z = np.zeros(N, np.float32)
    sp = ref.slice_pack(q, r)
    _, y_ref = ref.gemv(sp["packed"], K, r, a, z, x)
    y = mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x), flags=mq.GEMV_TENSOR_INT8)
    assert np.array_equal(host(y).astype(np.float64), y_ref)


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("N,K,B", [(1024, 1024, 1), (300, 2304, 1), (130, 9216, 8), (77, 3584, 4), (3, 128, 16),
                                   (257, 14336, 3), (64, 256, 5), (2304, 9216, 8), (500, 2432, 11), (129, 384, 2),
                                   (9216, 2304, 1), (128, 128, 1)])
def test_gemv_tcgen05_within_tolerance(r, N, K, B):
    # default path: tcgen05.mma with the unpacked weights as the TMEM A operand
    y, y_ref = _gemv_case(N, K, B, r, 500 + N + r, flags=mq.GEMV_TCGEN05)
    assert np.abs(y - y_ref).max() <= TOL_TENSOR * rms(y_ref)


@pytest.mark.parametrize("r", [4, 2])
@pytest.mark.parametrize("N,K,B,ep", [(9216, 2304, 1, False), (9216, 2304, 8, False), (2304, 9216, 1, True), (14336, 3584, 1, False),
                                      (14336, 3584, 8, True), (4096, 3584, 2, False), (2048, 3584, 1, True), (3584, 14336, 8, False),
                                      (9216, 2304, 1, True), (36864, 256, 3, False), (75008, 128, 1, False), (151680, 128, 2, True)])
def test_gemv_default_dispatch_at_benchmark_shapes(r, N, K, B, ep):
    # The library's own choice of warp tile, K split and CTA size (and the programmatic-dependent-launch flag the benchmark
    # passes) on the layer shapes of the Gemma-2-2B / 9B workloads, every output checked against the oracle.
    y, y_ref = _gemv_case(N, K, B, r, 700 + r, ep=ep, flags=mq.GEMV_AUTO | mq.GEMV_PDL)
    assert np.abs(y - y_ref).max() <= TOL_TENSOR * rms(y_ref)


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("N,K,B,ep", [(5001, 4096, 8, True), (5000, 4096, 16, False), (4801, 8192, 4, False),
                                      (3000, 4096, 12, True), (3584, 14336, 8, True), (2500, 8192, 5, False)])
def test_gemv_batches_on_long_rows_split_k_over_a_cluster(r, N, K, B, ep):
    # B >= 4 on long rows: clusters of 4 CTAs split K and the first CTA sums the partial results through distributed
    # shared memory.  Every cluster variant (one / two m-tiles, 8 / 16 warps, one / two n-tiles), ragged N, overflow lists.
    ep = ep and r < 8
    y, y_ref = _gemv_case(N, K, B, r, 880 + r + B, ep=ep, flags=mq.GEMV_AUTO | mq.GEMV_PDL)
    assert np.abs(y - y_ref).max() <= TOL_TENSOR * rms(y_ref)


@pytest.mark.parametrize("r", [8, 2])
def test_gemv_default_dispatch_rows_too_long_for_integer_sums(r):
    # K = 65536 is beyond what the integer path's 32-bit sums allow; the library's own choice must still be right.
    y, y_ref = _gemv_case(20, 65536, 1, r, 770 + r, flags=mq.GEMV_AUTO)
    assert np.abs(y - y_ref).max() <= TOL_TENSOR * rms(y_ref)
    y, y_ref = _gemv_case(20, 65536, 1, r, 770 + r, flags=mq.GEMV_TENSOR_INT8)
    assert np.abs(y - y_ref).max() <= TOL_TENSOR * rms(y_ref)


def test_gemv_default_dispatch_on_random_shapes():
    # Ragged N, every batch size class, short and long rows, with and without overflow lists: the split heuristic has
    # many branches (SK = 1 .. 32, one or two m-tiles, 8 / 16 / 32 warps) and each must give the oracle's result.
    rng = np.random.default_rng(2024)
    for case in range(36):
        N = int(rng.choice([1, 7, 16, 33, 100, 257, 600, 1500, 4100, 5000, 9500]))
        K = 128 * int(rng.choice([1, 2, 3, 5, 8, 19, 36, 72]))
        B = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 16]))
        r = int(rng.choice([8, 4, 2]))
        ep = bool(rng.integers(0, 2)) and r < 8
        y, y_ref = _gemv_case(N, K, B, r, 3000 + case, ep=ep, flags=mq.GEMV_AUTO | (mq.GEMV_PDL if case % 2 else 0))
        assert y.shape == y_ref.shape
        assert np.abs(y - y_ref).max() <= TOL_TENSOR * rms(y_ref), (N, K, B, r, ep)


@pytest.mark.parametrize("flags,tol", [(mq.GEMV_CUDA_CORE, TOL_FMA), (mq.GEMV_TENSOR, TOL_TENSOR), (mq.GEMV_TCGEN05, TOL_TENSOR),
                                       (mq.GEMV_AUTO, TOL_TENSOR), (mq.GEMV_TENSOR_INT8, TOL_TENSOR)])
@pytest.mark.parametrize("r", [4, 2])
@pytest.mark.parametrize("B", [1, 8])
def test_gemv_extra_precision(r, B, flags, tol):
    # (the integer path takes B = 1; with B = 8 its flag runs the bf16 kernel)
    y, y_ref = _gemv_case(130, 2304, B, r, 600 + r, ep=True, flags=flags)
    assert np.abs(y - y_ref).max() <= tol * rms(y_ref)


@pytest.mark.parametrize("flags", [mq.GEMV_CUDA_CORE, mq.GEMV_TENSOR, mq.GEMV_TCGEN05])
@pytest.mark.parametrize("r", [8, 4, 2])
def test_gemv_exact_integer_case(r, flags):
    # alpha = 1, z = 0, integer x: every partial sum is an exact fp32 integer, so the result must be exact.
    N, K, B = 70, 512, 4
    q = synth.uniform_codes((N, K), 700 + r)
    x = synth.small_int_bf16((B, K), -4, 4, 701)
    a = np.ones(N, np.float32); z = np.zeros(N, np.float32)
    sp = ref.slice_pack(q, r)
    _, y_ref = ref.gemv(sp["packed"], K, r, a, z, x)
    y = mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x), flags=flags)
    assert np.array_equal(host(y).astype(np.float64), y_ref)


def test_gemv_strided_x_and_y():
    N, K, B, r = 50, 256, 3, 4
    q = synth.uniform_codes((N, K), 800)
    a = np.full(N, 0.01, np.float32); z = np.full(N, 100.0, np.float32)
    x = synth.normal_bf16((B, K), 1.0, 801)
    sp = ref.slice_pack(q, r)
    _, y_ref = ref.gemv(sp["packed"], K, r, a, z, x)
    xw = torch.zeros((B, K + 8), dtype=torch.bfloat16, device="cuda"); xw[:, :K] = bf16_dev(x)
    yw = torch.full((B, N + 5), -1.0, dtype=torch.float32, device="cuda")
    mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), xw[:, :K], y=yw[:, :N])
    assert np.abs(host(yw)[:, :N] - y_ref).max() <= TOL_TENSOR * rms(y_ref)
    assert np.all(host(yw)[:, N:] == -1.0)


@pytest.mark.parametrize("r", [7, 6, 5, 3, 1])
def test_interpolated_precisions_decode_from_an_unpacked_slice(r):
    # Section 5.1 serves precisions that were not trained (int6, int3, ...) by slicing the same int8 codes.  For decode the
    # slice S(q, r) of Eq. 6, one byte per weight, IS an 8-bit plane: y = sum_k x alpha (S - z) is the r = 8 GEMV on it.
    # Checked against the oracle's dequantised product at that r (a different oracle routine than its GEMV).
    N, K = 520, 2304
    W = synth.normal_bf16((N, K), 0.02, 950 + r)
    st, q, a, z = ref.quantize(W)
    sl = mq.slice_pack(dev(q), r, want_packed=False, want_unpacked=True)["sliced"]
    st, S = ref.slice_values(q, r)
    assert st == ref.OK and np.array_equal(host(sl), S.astype(np.uint8))
    for B, tol in ((1, TOL_INT8), (4, TOL_TENSOR)):
        x = synth.normal_bf16((B, K), 1.0, 960 + r + B)
        st, Yr, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, x, rs=(r,), alpha=a, zero=z)
        assert st == ref.OK
        y = mq.gemv(sl, K, 8, dev(a), dev(z), bf16_dev(x))
        assert np.abs(host(y).reshape(B, N) - Yr[0]).max() <= tol * rms(Yr[0])
        yg = torch.empty((B, N), dtype=torch.float32, device="cuda")
        ad, zd, xd = dev(a), dev(z), bf16_dev(x)
        mq.gemv_grouped(mq.gemv_group([dict(packed=sl, K=K, r=8, alpha=ad, zero=zd, x=xd, y=yg)]))
        assert np.abs(host(yg) - Yr[0]).max() <= TOL_INT8 * rms(Yr[0])


def test_full_path_quantize_slice_pack_gemv():
    # bf16 weights -> codes -> plane -> y, everything on the GPU, against the oracle end to end.
    N, K, B = 260, 2304, 2
    W = synth.normal_bf16((N, K), 0.02, 900)
    x = synth.normal_bf16((B, K), 1.0, 901)
    q, a, z = mq.quantize(bf16_dev(W))
    st, q_ref, a_ref, z_ref = ref.quantize(W)
    for r in (8, 4, 2):
        sp = mq.slice_pack(q, r)
        y = mq.gemv(sp["packed"], K, r, a, z, bf16_dev(x))
        spr = ref.slice_pack(q_ref, r)
        _, y_ref = ref.gemv(spr["packed"], K, r, a_ref, z_ref, x)
        assert np.array_equal(host(sp["packed"]), spr["packed"])
        assert np.abs(host(y) - y_ref).max() <= TOL_TENSOR * rms(y_ref)
