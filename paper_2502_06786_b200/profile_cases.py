"""Small, self-contained invocations of each kernel for profilers (ncu wants short runs with few launches).

    python -m paper_2502_06786_b200.profile_cases quantize|slice4|slice2ep|gemv4|gemv2|gemv2b8|gemv4t|gemv2t|stream8|stream4|stream2|group4|group2|batch4|batch8|gemm

(gemv4 / gemv2: the library's own choice at B = 1, the integer tensor kernel; a trailing t: the bf16 tensor kernel.)

Every case touches a few hundred MB of distinct buffers (more than the L2 holds) and launches each kernel 16-24 times.
"""
from __future__ import annotations

import sys

import torch

from . import binding as mq
from . import synth


def _planes(n, N, K, r):
    return [torch.randint(0, 256, (N, K * r // 8), dtype=torch.uint8, device="cuda") for _ in range(n)]


def main(which: str) -> None:
    N, K = 9216, 2304                       # a Gemma-2-2B gate / up matrix
    n = 12
    if which == "quantize":
        Ws = [torch.randn(N, K, device="cuda").mul_(0.02).to(torch.bfloat16) for _ in range(n)]
        outs = [(torch.empty(N, K, dtype=torch.uint8, device="cuda"), torch.empty(N, device="cuda"), torch.empty(N, device="cuda")) for _ in range(n)]
        for _ in range(2):
            for W, (q, a, z) in zip(Ws, outs):
                mq.quantize(W, q=q, alpha=a, zero=z)
    elif which in ("slice4", "slice2ep"):
        qs = [torch.from_numpy(synth.skewed_codes((N, K), 0.005, 224, 10 + i)).cuda() for i in range(n)]
        for _ in range(2):
            for q in qs:
                if which == "slice4":
                    mq.slice_pack(q, 4)
                else:
                    mq.slice_pack(q, 2, extra_precision=True, ovf_capacity=N * K // 16)
    elif which in ("gemv4", "gemv2", "gemv2b8", "gemv4t", "gemv2t"):
        r = 4 if which.startswith("gemv4") else 2
        flags = mq.GEMV_TENSOR if which.endswith("t") else mq.GEMV_AUTO
        B = 8 if which.endswith("b8") else 1
        n = 24
        P = _planes(n, N, K, r)
        X = [torch.randn(B, K, device="cuda").to(torch.bfloat16) for _ in range(n)]
        Y = [torch.empty(B, N, device="cuda") for _ in range(n)]
        a = torch.ones(N, device="cuda")
        for _ in range(2):
            for i in range(n):
                mq.gemv(P[i], K, r, a, a, X[i], y=Y[i], flags=flags)
    elif which in ("stream8", "stream4", "stream2"):
        # the persistent kernel on a plane large enough for its steady state: 65536 x 2304, one problem per launch
        r = int(which[-1])
        N3 = 65536
        P = _planes(4, N3, K, r)
        X = [torch.randn(1, K, device="cuda").to(torch.bfloat16) for _ in range(4)]
        Y = [torch.empty(1, N3, device="cuda") for _ in range(4)]
        a = torch.ones(N3, device="cuda")
        for _ in range(2):
            for i in range(4):
                mq.gemv(P[i], K, r, a, a, X[i], y=Y[i], flags=mq.GEMV_STREAM)
    elif which in ("group4", "group2"):
        # twelve matrices of the Gemma-2-2B MLP stack (4 layers) in one matq_gemv_grouped call
        r = int(which[-1])
        shapes = [(9216, 2304), (9216, 2304), (2304, 9216)] * 4
        P = [torch.randint(0, 256, (n_, k_ * r // 8), dtype=torch.uint8, device="cuda") for n_, k_ in shapes]
        X = [torch.randn(k_, device="cuda").to(torch.bfloat16) for n_, k_ in shapes]
        Y = [torch.empty(n_, device="cuda") for n_, k_ in shapes]
        a = torch.ones(9216, device="cuda")
        g = mq.gemv_group([(P[i], shapes[i][1], r, a[:shapes[i][0]], a[:shapes[i][0]], X[i], Y[i]) for i in range(len(shapes))])
        for _ in range(3):
            mq.gemv_grouped(g)
    elif which in ("batch4", "batch8"):
        # twelve matrices of the Gemma-2-2B MLP stack at r = 4 with 4 or 8 activation vectors each, one matq_gemv_grouped call
        B = int(which[-1])
        shapes = [(9216, 2304), (9216, 2304), (2304, 9216)] * 4
        P = [torch.randint(0, 256, (n_, k_ // 2), dtype=torch.uint8, device="cuda") for n_, k_ in shapes]
        X = [torch.randn(B, k_, device="cuda").to(torch.bfloat16) for n_, k_ in shapes]
        Y = [torch.empty(B, n_, device="cuda") for n_, k_ in shapes]
        a = torch.ones(9216, device="cuda")
        g = mq.gemv_group([(P[i], shapes[i][1], 4, a[:shapes[i][0]], a[:shapes[i][0]], X[i], Y[i]) for i in range(len(shapes))])
        for _ in range(3):
            mq.gemv_grouped(g)
    elif which == "gemm":
        N2, K2, M2 = 14336, 4096, 1024      # the Mistral-7B matrix with a quarter of the tokens
        q = torch.randint(0, 256, (N2, K2), dtype=torch.uint8, device="cuda")
        X = torch.randn(M2, K2, device="cuda").to(torch.bfloat16)
        a = torch.full((N2,), 1e-3, device="cuda")
        Ys = [torch.empty(M2, N2, device="cuda") for _ in range(3)]
        ws = torch.empty(mq.gemm_multi_workspace_bytes(mq.SRC_CODES8, M2, N2, K2, 3), dtype=torch.uint8, device="cuda")
        for _ in range(3):
            mq.gemm_multi(mq.SRC_CODES8, q, K2, X, alpha=a, zero=a, Ys=Ys, workspace=ws)
    else:
        raise SystemExit(__doc__)
    torch.cuda.synchronize()
    print("ok", which)


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else "")
