"""The N > 1 path on CPU: two gloo ranks shard a layer by output channel, run the path on their rows (with the
oracle standing in for the kernels) and all-gather y; the result must equal the unsharded computation exactly."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_06786_b200 import shard


def test_row_ranges_partition_the_rows():
    for N in (0, 1, 16, 100, 2304, 9216, 14337):
        for world in (1, 2, 3, 8):
            rs = [shard.row_range(N, world, r) for r in range(world)]
            assert rs[0][0] == 0 and rs[-1][1] == N
            for (l0, h0), (l1, h1) in zip(rs, rs[1:]):
                assert h0 == l1 and l0 <= h0
            assert all((h - l) % 16 == 0 for l, h in rs[:-1] if h < N)
            sizes = [h - l for l, h in rs]
            assert max(sizes) - min(sizes) <= 16 + 15


def _worker(rank, world, port, N, K, B, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import ref
        from paper_2502_06786_b200 import synth
        W = synth.normal_bf16((N, K), 0.02, 77)
        x = synth.normal_bf16((B, K), 1.0, 78)
        lo, hi = shard.row_range(N, world, rank)
        Wl = np.ascontiguousarray(W[lo:hi])
        st, q, a, z = ref.quantize(Wl)
        sp = ref.slice_pack(q, 2, extra_precision=True)
        st, y = ref.gemv(sp["packed"], K, 2, a, z, x, sp["ovf_row_ptr"], sp["ovf_col"])
        full = shard.all_gather_rows(torch.from_numpy(y), N)
        np.save(os.path.join(out_dir, f"y{rank}.npy"), full.numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_two_ranks_reproduce_the_unsharded_layer(tmp_path):
    from oracle import ref
    from paper_2502_06786_b200 import synth
    N, K, B, world = 200, 256, 3, 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(world, port, N, K, B, str(tmp_path)), nprocs=world, join=True)
    W = synth.normal_bf16((N, K), 0.02, 77)
    x = synth.normal_bf16((B, K), 1.0, 78)
    st, q, a, z = ref.quantize(W)
    sp = ref.slice_pack(q, 2, extra_precision=True)
    st, y = ref.gemv(sp["packed"], K, 2, a, z, x, sp["ovf_row_ptr"], sp["ovf_col"])
    for r in range(world):
        got = np.load(tmp_path / f"y{r}.npy")
        assert np.array_equal(got, y)
