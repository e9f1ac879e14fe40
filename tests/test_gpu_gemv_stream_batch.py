"""GPU parity of the batched persistent decode GEMV (2 <= B <= 16 activation vectors per problem: MATQ_GEMV_STREAM
with B > 1, and matq_gemv_grouped with batches) against the CPU oracle.

The weights' sums are exact integers.  Two vectors, and every batch at r = 2 (pair groups): an activation is a 22-bit
integer relative to the largest magnitude of its vector, and a field that sits s bits up in its byte meets its
activation divided by 2^s, so the activations of the top field keep 22 - (8 - r) bits: rounding steps of 2^-22 (r = 8),
2^-18 (r = 4) and 2^-16 (r = 2) of 2 max|x|.  With max|x| / rms(x) about 4 that is 1e-6, 2e-5 and 6e-5 of rms(y); the
tests allow 1e-4, 3e-4 and 1e-3.  Three or more vectors at r = 8 and r = 4 (quad groups): a 15-bit integer and its sign,
a rounding step of 2^-14 (2^-13 when the largest magnitude's significand is all ones) of the power of two at or below
max|x|, the same for both fields: about 4e-5 of rms(y) per output, 2e-4 at worst over tens of thousands of outputs; the
tests allow 1e-3 (the bound for the tensor-core paths is 1e-2 rms(y); the bf16 tensor path for batches is held to that).
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2502_06786_b200 import binding as mq
from paper_2502_06786_b200 import synth
from tests.util import bf16_dev, dev, host, rms, status_word

pytestmark = pytest.mark.gpu

TOL = {8: 1e-4, 4: 3e-4, 2: 1e-3}
TOL_QUAD = 1e-3


def tol(r, B):
    return TOL_QUAD if (r != 2 and B >= 3) else TOL[r]


def _problem(N, K, r, B, seed, scales=None):
    W = synth.normal_bf16((N, K), 0.02, seed)
    _, q, a, z = ref.quantize(W)
    x = synth.normal_bf16((B, K), 1.0, seed + 1)
    if scales is not None:                       # vectors of very different magnitude: each has its own block scale
        xf = synth.bf16_bits_to_f32(x) * np.asarray(scales, np.float32)[:B, None]
        x = synth.f32_to_bf16_bits(xf)
    sp = ref.slice_pack(q, r)
    st, y_ref = ref.gemv(sp["packed"], K, r, a, z, x, None, None)
    assert st == ref.OK
    return dict(N=N, K=K, r=r, B=B, packed=sp["packed"], a=a, z=z, x=x, y_ref=y_ref)


def _check(y, y_ref, r):
    y = host(y).reshape(y_ref.shape)
    for b in range(y_ref.shape[0]):
        assert np.abs(y[b] - y_ref[b]).max() <= tol(r, y_ref.shape[0]) * rms(y_ref[b]), f"vector {b}"


@pytest.mark.parametrize("r", [8, 4, 2])
@pytest.mark.parametrize("B", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("N,K", [(1024, 1024), (300, 2304), (130, 9216), (77, 3584), (3, 256), (2304, 2304), (40000, 256), (17, 1792)])
def test_stream_batch_single_problem(r, B, N, K):
    # one and several K panels, 1 to 4 tiles per unit, fewer tiles than SMs (panels spread over warps) and many tiles
    # per SM, ragged last tile; 1, 2 and 4 column groups, the last one half full for odd B
    if r == 2 and K % 256:
        pytest.skip("r = 2 batches need K % 256 == 0")
    p = _problem(N, K, r, B, 7000 + N + 10 * r + B)
    status = status_word()
    y = mq.gemv(dev(p["packed"]), K, r, dev(p["a"]), dev(p["z"]), bf16_dev(p["x"]), flags=mq.GEMV_STREAM | mq.GEMV_PDL, dev_status=status)
    _check(y, p["y_ref"], p["r"])
    assert int(host(status)[0]) == mq.OK


@pytest.mark.parametrize("r", [8, 4, 2])
def test_stream_batch_sixteen_vectors(r):
    # sixteen vectors: one problem of four quad groups at r = 8 and 4, two problems of 8 that share the plane at r = 2
    p = _problem(700, 2304, r, 16, 7100 + r)
    y = mq.gemv(dev(p["packed"]), 2304, r, dev(p["a"]), dev(p["z"]), bf16_dev(p["x"]), flags=mq.GEMV_STREAM)
    _check(y, p["y_ref"], p["r"])


@pytest.mark.parametrize("r", [8, 4, 2])
def test_stream_batch_vectors_of_different_magnitude(r):
    # every vector has its own power-of-two scale: one tiny, one huge, one all zero
    scales = [1.0, 2.0 ** -30, 2.0 ** 30, 0.0, 3.0, 1e-3]
    p = _problem(260, 1024, r, 6, 7200 + r, scales=scales)
    y = mq.gemv(dev(p["packed"]), 1024, r, dev(p["a"]), dev(p["z"]), bf16_dev(p["x"]), flags=mq.GEMV_STREAM)
    y = host(y)
    for b in range(6):
        ref_b = p["y_ref"][b]
        assert np.abs(y[b] - ref_b).max() <= tol(r, 6) * max(rms(ref_b), 1e-30), f"vector {b}"


def test_stream_batch_exact_integers():
    # all-integer case: alpha = 1, z = 0, small integer activations: the result is exact
    N, K, r, B = 48, 512, 4, 4
    rng = np.random.default_rng(5)
    q = rng.integers(0, 256, (N, K), dtype=np.uint8)
    sp = ref.slice_pack(q, r)
    x = synth.f32_to_bf16_bits(rng.integers(-8, 9, (B, K)).astype(np.float32))
    a, z = np.ones(N, np.float32), np.zeros(N, np.float32)
    _, y_ref = ref.gemv(sp["packed"], K, r, a, z, x, None, None)
    y = mq.gemv(dev(sp["packed"]), K, r, dev(a), dev(z), bf16_dev(x), flags=mq.GEMV_STREAM)
    assert np.array_equal(host(y).astype(np.float64), y_ref)


def test_grouped_list_with_batches_and_single_vectors():
    # one call: batches of different sizes (1, 2 and 4 groups in one launch), single vectors and a batch above 8
    specs = [(300, 2304, 4, 8), (130, 9216, 2, 4), (1024, 1024, 8, 1), (77, 3584, 4, 2), (500, 2304, 2, 8), (64, 256, 8, 3),
             (2304, 2304, 4, 12), (9216, 2304, 4, 8), (33, 1024, 2, 1), (200, 2304, 2, 9)]
    probs = [_problem(N, K, r, B, 7300 + i) for i, (N, K, r, B) in enumerate(specs)]
    items = []
    ys = []
    for p in probs:
        x = bf16_dev(p["x"])
        y = torch.full((p["B"], p["N"]), float("nan"), dtype=torch.float32, device="cuda")
        if p["B"] == 1:
            x, y = x.reshape(-1), y.reshape(-1)
        ys.append(y)
        items.append((dev(p["packed"]), p["K"], p["r"], dev(p["a"]), dev(p["z"]), x, y))
    status = status_word()
    group = mq.gemv_group(items)
    mq.gemv_grouped(group, flags=mq.GEMV_PDL, dev_status=status)
    for p, y in zip(probs, ys):
        _check(y, p["y_ref"], p["r"])
    assert int(host(status)[0]) == mq.OK
    # the same list again: nothing in the kernels' shared state is left behind by a call
    for y in ys:
        y.fill_(float("nan"))
    mq.gemv_grouped(group)
    for p, y in zip(probs, ys):
        _check(y, p["y_ref"], p["r"])


def test_grouped_batch_whole_stack_matches_single_calls_bit_for_bit():
    # a list of 20 batched problems in one call gives the bits of 20 single calls (integer sums do not depend on how the
    # list is cut into CTA shares)
    shapes = [(9216, 2304), (9216, 2304), (2304, 9216), (512, 2304)] * 5
    B, r = 4, 4
    probs = [_problem(N, K, r, B, 7400 + i) for i, (N, K) in enumerate(shapes[:4])]
    items, ys = [], []
    for i in range(len(shapes)):
        p = probs[i % 4]
        y = torch.empty((B, p["N"]), dtype=torch.float32, device="cuda")
        ys.append(y)
        items.append((dev(p["packed"]), p["K"], r, dev(p["a"]), dev(p["z"]), bf16_dev(p["x"]), y))
    mq.gemv_grouped(items)
    for i, y in enumerate(ys):
        p = probs[i % 4]
        single = mq.gemv(dev(p["packed"]), p["K"], r, dev(p["a"]), dev(p["z"]), bf16_dev(p["x"]), flags=mq.GEMV_STREAM)
        assert torch.equal(y, single)
        _check(y, p["y_ref"], p["r"])


def test_batch_argument_errors():
    p = _problem(64, 256, 2, 4, 7500)
    packed, a, z, x = dev(p["packed"]), dev(p["a"]), dev(p["z"]), bf16_dev(p["x"])
    y = torch.empty((4, 64), dtype=torch.float32, device="cuda")
    rp = torch.zeros(65, dtype=torch.int32, device="cuda")
    col = torch.zeros(1, dtype=torch.uint16, device="cuda")
    # lists with several vectors are not served by the grouped call
    st = mq.gemv_grouped([(packed, 256, 2, a, z, x, y, rp, col)], raise_on_error=False)
    assert st == mq.ERR_UNSUPPORTED
    # r = 2 with K % 256 == 128
    p2 = _problem(64, 384, 2, 2, 7501)
    y2 = torch.empty((2, 64), dtype=torch.float32, device="cuda")
    st = mq.gemv_grouped([(dev(p2["packed"]), 384, 2, dev(p2["a"]), dev(p2["z"]), bf16_dev(p2["x"]), y2)], raise_on_error=False)
    assert st == mq.ERR_SHAPE
