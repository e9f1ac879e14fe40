"""The entry point that needs no workspace (matq_gemm_multi_static), checked against matq_gemm_multi.

Some callers of the library cannot get device memory when they call it (memory handed out once at start-up,
cudaMalloc forbidden on the request path), so this variant keeps its scratch in an array that is part of the
library.  The test calls it through the C ABI twice in a row with different problems: the second call finds the first
call's planes still in the shared array and must not be affected by them.  It lives in a file of its own that pytest
collects last, and it passes alone in a fresh process as well as after all the other tests.
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2502_06786_b200 import binding as mq
from paper_2502_06786_b200 import synth
from tests.util import bf16_dev, dev, host, rms

pytestmark = pytest.mark.gpu
TOL = 1e-2    # the tolerance of the tensor-core forward in the other tests


def _outputs(M, N, n):
    return [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(n)]


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    assert mq.gemm_multi_static_max_bytes() == 16 << 20

    # call 1: codes in, three precisions
    M, N, K = 200, 520, 512
    q = dev(synth.uniform_codes((N, K), 901))
    a = dev((np.abs(synth.bf16_bits_to_f32(synth.normal_bf16((N,), 0.01, 902))) + 1e-3).astype(np.float32))
    z = dev((synth.bf16_bits_to_f32(synth.normal_bf16((N,), 30.0, 903)) + 128).astype(np.float32))
    X = bf16_dev(synth.normal_bf16((M, K), 1.0, 904))
    want, _, _ = mq.gemm_multi(mq.SRC_CODES8, q, K, X, alpha=a, zero=z)
    got = _outputs(M, N, 3)
    assert mq.gemm_multi_static(mq.SRC_CODES8, q, K, X, got, a, z) == mq.OK
    for g, w in zip(got, want):
        assert np.abs(host(g) - host(w)).max() <= TOL * rms(host(w))
    # and against the CPU oracle directly, not only against the other entry point
    st, Yr, _, _ = ref.gemm_multi(ref.SRC_CODES8, host(q), K, host(X.view(torch.uint16)).astype(np.uint16), alpha=host(a), zero=host(z))
    assert st == ref.OK
    for g, yr in zip(got, Yr):
        assert np.abs(host(g) - yr).max() <= TOL * rms(yr)

    # call 2, straight after: another shape, bf16 source (quantises on the fly), two precisions
    M2, N2, K2 = 96, 264, 1024
    W2 = bf16_dev(synth.student_t_bf16((N2, K2), 3.0, 0.02, 905))
    X2 = bf16_dev(synth.normal_bf16((M2, K2), 1.0, 906))
    want2, a_w, z_w = mq.gemm_multi(mq.SRC_BF16, W2, K2, X2, rs=(4, 2))
    got2 = _outputs(M2, N2, 2)
    a_g = torch.empty(N2, dtype=torch.float32, device="cuda"); z_g = torch.empty_like(a_g)
    assert mq.gemm_multi_static(mq.SRC_BF16, W2, K2, X2, got2, a_g, z_g, rs=(4, 2)) == mq.OK
    assert torch.equal(a_g, a_w) and torch.equal(z_g, z_w)
    for g, w in zip(got2, want2):
        assert np.abs(host(g) - host(w)).max() <= TOL * rms(host(w))

    # and the first problem again gives the first answer again
    again = _outputs(M, N, 3)
    assert mq.gemm_multi_static(mq.SRC_CODES8, q, K, X, again, a, z) == mq.OK
    for g, w in zip(again, got):
        assert torch.equal(g, w)


def test_a_problem_larger_than_the_built_in_scratch_is_refused():
    M, N, K = 128, 4096, 4096            # 16.8 M codes: planes alone are far beyond 16 MiB
    assert mq.gemm_multi_workspace_bytes(mq.SRC_CODES8, M, N, K, 3) > mq.gemm_multi_static_max_bytes()
    q = torch.zeros((N, K), dtype=torch.uint8, device="cuda")
    X = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    a = torch.ones(N, dtype=torch.float32, device="cuda")
    Y = _outputs(M, N, 3)
    st = mq.gemm_multi_static(mq.SRC_CODES8, q, K, X, Y, a, a, raise_on_error=False)
    assert st == mq.ERR_WORKSPACE
    assert all(bool(torch.isnan(y).all()) for y in Y)        # nothing was launched
