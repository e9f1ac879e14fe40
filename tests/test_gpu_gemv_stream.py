"""GPU parity of the persistent decode GEMV (MATQ_GEMV_STREAM) and of matq_gemv_grouped against the CPU oracle.

The integer path's tolerance applies: exact integer sums, activations rounded to an absolute 2^-24 of the largest
at worst, fp32 epilogue: max|dy| <= 1e-4 * rms(y_oracle).
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2502_06786_b200 import binding as mq
from paper_2502_06786_b200 import synth
from tests.util import bf16_dev, dev, host, rms, status_word

pytestmark = pytest.mark.gpu

TOL_INT8 = 1e-4


def _problem(N, K, r, seed, ep=False, x=None):
    """Host side of one problem: oracle inputs and the oracle's y."""
    W = synth.normal_bf16((N, K), 0.02, seed)
    _, q, a, z = ref.quantize(W)
    if ep:
        q = synth.skewed_codes((N, K), 0.05, 224, seed + 5)
    if x is None:
        x = synth.normal_bf16((1, K), 1.0, seed + 1)
    sp = ref.slice_pack(q, r, extra_precision=ep)
    rp = sp["ovf_row_ptr"] if ep else None
    col = sp["ovf_col"] if ep else None
    st, y_ref = ref.gemv(sp["packed"], K, r, a, z, x, rp, col)
    assert st == ref.OK
    return dict(N=N, K=K, r=r, packed=sp["packed"], a=a, z=z, x=x, rp=rp, col=col, y_ref=y_ref[0])


def _to_device(p, x_dev=None):
    d = dict(packed=dev(p["packed"]), K=p["K"], r=p["r"], alpha=dev(p["a"]), zero=dev(p["z"]),
             x=bf16_dev(p["x"]).reshape(-1) if x_dev is None else x_dev,
             y=torch.full((p["N"],), float("nan"), dtype=torch.float32, device="cuda"))
    if p["rp"] is not None:
        d["ovf_row_ptr"] = dev(p["rp"])
        d["ovf_col"] = dev(p["col"] if p["col"].size else np.zeros(1, np.uint16))
    return d


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("N,K", [(1024, 1024), (300, 2304), (130, 9216), (77, 3584), (3, 128), (257, 14336), (64, 256),
                                 (2304, 9216), (500, 2432), (129, 384), (9216, 2304), (128, 128), (40000, 128),
                                 (5000, 256), (33, 16384), (33, 32768), (20000, 384), (14336, 3584), (1, 640), (17, 896),
                                 (37900, 3584)])
def test_stream_single_problem(r, N, K):
    # every stage shape: 1, 2 and 4 tiles per row block, one and several K panels, half-full last chunks (r = 2,
    # K % 256 == 128), fewer tiles than SMs and many tiles per SM, the last tile ragged; 37900 x 3584: rows in several
    # K panels with at least as many pairs of tiles per CTA as warps (two tiles per pass at r = 2, sums kept across panels)
    p = _problem(N, K, r, 500 + N + r)
    status = status_word()
    y = mq.gemv(dev(p["packed"]), K, r, dev(p["a"]), dev(p["z"]), bf16_dev(p["x"]), flags=mq.GEMV_STREAM | mq.GEMV_PDL,
                dev_status=status)
    assert np.abs(host(y)[0] - p["y_ref"]).max() <= TOL_INT8 * rms(p["y_ref"])
    assert int(host(status)[0]) == mq.OK


@pytest.mark.parametrize("r", [4, 2])
@pytest.mark.parametrize("N,K", [(9216, 2304), (2304, 9216), (300, 2432), (2048, 3584), (70, 128), (4800, 3584), (37900, 3584)])
def test_stream_extra_precision(r, N, K):
    # 4800 x 3584: pairs of tiles whose K panels are spread over warps; 37900 x 3584: pairs kept by one warp across panels
    p = _problem(N, K, r, 900 + r, ep=True)
    d = _to_device(p)
    y = mq.gemv(d["packed"], K, r, d["alpha"], d["zero"], d["x"].reshape(1, -1), ovf_row_ptr=d["ovf_row_ptr"],
                ovf_col=d["ovf_col"], flags=mq.GEMV_STREAM)
    assert np.abs(host(y)[0] - p["y_ref"]).max() <= TOL_INT8 * rms(p["y_ref"])


@pytest.mark.parametrize("r", [4, 2])
def test_stream_extra_precision_full_and_empty_rows(r):
    # rows whose every code is in the extra bucket (a list as long as the row), rows with none, a ragged last tile
    N, K = 77, 2304
    q = synth.skewed_codes((N, K), 0.05, 224, 4321 + r)
    q[3, :] = 255
    q[16:19, :] = 250
    q[40, :] = 0
    q[76, ::2] = 255
    W = synth.normal_bf16((N, K), 0.02, 99)
    _, _, a, z = ref.quantize(W)
    x = synth.normal_bf16((1, K), 1.0, 98)
    sp = ref.slice_pack(q, r, extra_precision=True)
    _, y_ref = ref.gemv(sp["packed"], K, r, a, z, x, sp["ovf_row_ptr"], sp["ovf_col"])
    y = mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x), ovf_row_ptr=dev(sp["ovf_row_ptr"]), ovf_col=dev(sp["ovf_col"]),
                flags=mq.GEMV_STREAM)
    assert np.abs(host(y)[0] - y_ref[0]).max() <= TOL_INT8 * rms(y_ref[0])


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("kind", ["zero", "outlier", "large", "small", "one_hot"])
def test_stream_activation_ranges(r, kind):
    N, K = 200, 1024
    W = synth.normal_bf16((N, K), 0.02, 4100 + r)
    _, q, a, z = ref.quantize(W)
    xf = synth.bf16_bits_to_f32(synth.normal_bf16((1, K), 1.0, 4200 + r)).copy()
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
    y = host(mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x), flags=mq.GEMV_STREAM))
    assert np.abs(y[0] - y_ref[0]).max() <= TOL_INT8 * max(rms(y_ref[0]), 1e-300), kind


@pytest.mark.parametrize("r", [8, 4, 2])
def test_stream_exact_integer_case(r):
    # alpha = 1, z = 0, small integer x: every sum is an exact integer, so the result must equal the oracle's exactly
    N, K = 70, 512
    q = synth.uniform_codes((N, K), 720 + r)
    x = synth.small_int_bf16((1, K), -4, 4, 721)
    a = np.ones(N, np.float32); z = np.zeros(N, np.float32)
    sp = ref.slice_pack(q, r)
    _, y_ref = ref.gemv(sp["packed"], K, r, a, z, x)
    y = mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x), flags=mq.GEMV_STREAM)
    assert np.array_equal(host(y).astype(np.float64), y_ref)


def test_grouped_mixed_list():
    # one launch: q, k, v-like projections sharing x, gate/up sharing another x, a long-row matrix, mixed r
    # (a Mix'n'Match layer list), two problems with extra-precision lists, an empty problem in the middle
    xa = synth.normal_bf16((1, 2304), 1.0, 31)
    xb = synth.normal_bf16((1, 3584), 1.0, 32)
    hosts = [_problem(2048, 2304, 4, 1, x=xa), _problem(1024, 2304, 2, 2, x=xa), _problem(1000, 2304, 8, 3, x=xa),
             _problem(4000, 3584, 2, 4, x=xb), _problem(4001, 3584, 4, 5, x=xb, ep=True),
             _problem(300, 9216, 4, 6), _problem(515, 14336, 2, 7, ep=True), _problem(33, 128, 8, 8)]
    xa_d, xb_d = bf16_dev(xa).reshape(-1), bf16_dev(xb).reshape(-1)
    devs = [_to_device(p, xa_d if p["x"] is xa else xb_d if p["x"] is xb else None) for p in hosts]
    empty = dict(devs[0])
    empty["packed"] = devs[0]["packed"][:0]
    empty["y"] = devs[0]["y"][:0]
    order = devs[:3] + [empty] + devs[3:]
    status = status_word()
    mq.gemv_grouped(order, flags=mq.GEMV_PDL, dev_status=status)
    for p, d in zip(hosts, devs):
        assert np.abs(host(d["y"]) - p["y_ref"]).max() <= TOL_INT8 * rms(p["y_ref"]), (p["N"], p["K"], p["r"])
    assert int(host(status)[0]) == mq.OK


def test_grouped_long_list_and_equality_with_single_calls():
    # more problems than the small descriptor table holds; every output must equal, bit for bit, what matq_gemv's
    # persistent path gives for the problem alone (integer sums do not depend on how the list is cut)
    # (the long rows change the number of multiplying warps of the launch: the fp32 sum of x must not depend on it)
    shapes = [(300 + 37 * i, 128 * (1 + i % 9), (8, 4, 2)[i % 3]) for i in range(21)] + [(130, 9216, 4), (77, 14336, 2)]
    hosts = [_problem(N, K, r, 50 + i) for i, (N, K, r) in enumerate(shapes)]
    devs = [_to_device(p) for p in hosts]
    mq.gemv_grouped(devs)
    for p, d in zip(hosts, devs):
        y = host(d["y"])
        assert np.abs(y - p["y_ref"]).max() <= TOL_INT8 * rms(p["y_ref"])
        alone = mq.gemv(d["packed"], p["K"], p["r"], d["alpha"], d["zero"], d["x"].reshape(1, -1), flags=mq.GEMV_STREAM)
        assert np.array_equal(host(alone)[0], y)


def test_grouped_argument_errors():
    p = _to_device(_problem(64, 256, 4, 77))
    assert mq.gemv_grouped([], raise_on_error=False) == mq.OK
    bad = dict(p); bad["r"] = 3
    assert mq.gemv_grouped([bad], raise_on_error=False) == mq.ERR_UNSUPPORTED
    g = mq.gemv_group([p])
    g[0].K = 200
    assert mq.gemv_grouped(g, raise_on_error=False) == mq.ERR_SHAPE
    g = mq.gemv_group([p])
    g[0].x = g[0].x + 2
    assert mq.gemv_grouped(g, raise_on_error=False) == mq.ERR_ALIGNMENT
    g = mq.gemv_group([p])
    g[0].ovf_row_ptr = g[0].alpha
    assert mq.gemv_grouped(g, raise_on_error=False) == mq.ERR_INVALID_ARG
    assert mq.gemv_grouped(mq.gemv_group([p]), flags=7, raise_on_error=False) == mq.ERR_INVALID_ARG


def test_a_wait_that_runs_out_is_a_status_not_a_hang():
    # MATQ_GEMV_TEST_STALL: the producer of the persistent kernel issues no copies, so the multiplying warps' waits for
    # their stages run out.  The kernel must return, report MATQ_ERR_TIMEOUT, leave y alone, and the same context
    # (same stream) must then serve the same list correctly.
    hosts = [_problem(2048, 2304, 4, 11), _problem(300, 9216, 2, 12), _problem(515, 3584, 8, 13, ep=False)]
    devs = [_to_device(p) for p in hosts]
    status = status_word()
    st = mq.gemv_grouped(devs, flags=mq.GEMV_TEST_STALL, dev_status=status, raise_on_error=False)
    assert st == mq.OK                                    # the launch itself is fine: the error depends on the device
    assert int(host(status)[0]) == mq.ERR_TIMEOUT
    for d in devs:
        assert bool(torch.isnan(d["y"]).all())          # nothing was stored
    status.zero_()
    mq.gemv_grouped(devs, dev_status=status)
    for p, d in zip(hosts, devs):
        assert np.abs(host(d["y"]) - p["y_ref"]).max() <= TOL_INT8 * rms(p["y_ref"])
    assert int(host(status)[0]) == mq.OK
