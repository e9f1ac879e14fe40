"""Randomised shapes for every entry point: each kernel family picks among several variants by shape (register /
shared-memory / scalar quantisers, one-pass or three-kernel extra-precision lists, 128- or 256-channel GEMM tiles),
and every variant must reproduce the oracle.  Seeds are fixed, so a failure names its case."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2502_06786_b200 import binding as mq
from paper_2502_06786_b200 import synth
from tests.util import bf16_dev, dev, host, rms, status_word

pytestmark = pytest.mark.gpu


def test_quantize_random_shapes():
    rng = np.random.default_rng(31)
    for case in range(30):
        N = int(rng.choice([1, 3, 8, 33, 129, 700]))
        K = int(rng.choice([8, 24, 72, 77, 256, 1000, 2304, 2312, 4104, 9216, 16384, 16392, 20000]))
        W = synth.student_t_bf16((N, K), 3.0, 0.02, 5000 + case)
        clip = case % 3 == 0
        g = rng.uniform(0.3, 1.2, N).astype(np.float32) if clip else None
        b = rng.uniform(0.3, 1.2, N).astype(np.float32) if clip else None
        st, q_ref, a_ref, z_ref = ref.quantize_clip(W, g, b) if clip else ref.quantize(W)
        assert st == ref.OK
        if case % 4 == 1:                                   # a view into a wider matrix (row stride > K, still 16-byte rows)
            wide = torch.zeros((N, K + 40), dtype=torch.bfloat16, device="cuda")
            wide[:, :K] = bf16_dev(W)
            Wd = wide[:, :K]
        else:
            Wd = bf16_dev(W)
        q, a, z = mq.quantize(Wd, gamma=dev(g) if clip else None, beta=dev(b) if clip else None)
        assert np.array_equal(host(a), a_ref) and np.array_equal(host(z), z_ref), (case, N, K)
        assert np.array_equal(host(q), q_ref), (case, N, K)


def test_slice_pack_random_shapes():
    rng = np.random.default_rng(32)
    for case in range(40):
        N = int(rng.choice([1, 5, 8, 9, 63, 64, 65, 300, 2000]))
        K = int(rng.choice([8, 16, 24, 48, 256, 1000, 2304, 4112, 16384, 16400]))
        r = int(rng.choice([8, 4, 2]))
        ep = bool(rng.integers(0, 2))
        p = float(rng.choice([0.0, 0.01, 0.2, 1.0]))
        q = synth.skewed_codes((N, K), p, 224, 6000 + case) if 0 < p < 1 else \
            (np.full((N, K), 255, np.uint8) if p == 1.0 else synth.uniform_codes((N, K), 6000 + case) // 2)
        want = ref.slice_pack(q, r, extra_precision=ep)
        status = status_word()
        out = mq.slice_pack(dev(q), r, extra_precision=ep, want_unpacked=True, dev_status=status)
        assert np.array_equal(host(out["packed"]), want["packed"]), (case, N, K, r, ep)
        assert np.array_equal(host(out["sliced"]), want["sliced"]), (case, N, K, r, ep)
        if ep and r < 8:
            cnt = int(host(out["ovf_count"])[0])
            assert cnt == want["ovf_count"], (case, N, K, r)
            assert np.array_equal(host(out["ovf_row_ptr"]), want["ovf_row_ptr"]), (case, N, K, r)
            assert np.array_equal(host(out["ovf_col"])[:cnt], want["ovf_col"]), (case, N, K, r)
        assert int(host(status)[0]) == mq.OK


def test_gemm_multi_random_shapes():
    rng = np.random.default_rng(33)
    for case in range(16):
        M = int(rng.choice([1, 17, 128, 130, 300]))
        N = 8 * int(rng.choice([1, 16, 17, 32, 33, 48, 100]))
        K = 64 * int(rng.choice([1, 2, 5, 16]))
        rs = [(8, 4, 2), (4,), (2,), (6, 3), (8, 2)][int(rng.integers(0, 5))]
        ep = bool(rng.integers(0, 2))
        W = synth.normal_bf16((N, K), 0.02, 7000 + case)
        st, q, a, z = ref.quantize(W)
        if ep:
            q = synth.skewed_codes((N, K), 0.05, 224, 7100 + case)
        X = synth.normal_bf16((M, K), 1.0, 7200 + case)
        Ys, _, _ = mq.gemm_multi(mq.SRC_CODES8, dev(q), K, bf16_dev(X), rs=rs, alpha=dev(a), zero=dev(z), extra_precision=ep)
        st, Yr, _, _ = ref.gemm_multi(ref.SRC_CODES8, q, K, X, rs=rs, alpha=a, zero=z, extra_precision=ep)
        assert st == ref.OK
        for y, yr in zip(Ys, Yr):
            assert np.abs(host(y) - yr).max() <= 1e-2 * rms(yr), (case, M, N, K, rs, ep)
