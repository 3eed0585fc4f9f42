"""World-size-2 check (gloo, CPU) of the data-parallel sharding used by bench.py --gpus N: each rank takes its
block of batch rows, computes its share of the weight-side sums (here with the CPU oracle), the ranks all-reduce,
and the result must equal the unsharded computation exactly (integer sums)."""
import os
import tempfile

import numpy as np
import pytest

import oracle
from paper_2501_09849_b200 import inputs, sharding


def test_row_range_partitions_exactly():
    for n in (0, 1, 7, 64, 50176):
        for world in (1, 2, 3, 8):
            blocks = [sharding.row_range(n, r, world) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == n
            assert all(blocks[i][1] == blocks[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in blocks]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.row_range(4, 2, 2)


def _worker(rank, world, init_file, out_dir):
    import torch
    import torch.distributed as dist
    dist.init_process_group("gloo", init_method=f"file://{init_file}", rank=rank, world_size=world)
    M, K, N = 301, 48, 24
    A = inputs.uniform_indices((M, K), 0, 15, seed=1)
    G = inputs.uniform_indices((M, N), -127, 127, seed=2)
    x = inputs.relu_normal((M, 40), seed=3)
    r0, r1 = sharding.row_range(M, rank, world)
    dW = torch.from_numpy(oracle.gemm_dw(A[r0:r1], G[r0:r1]))                      # int64 partial sums
    _, h = oracle.hard(x[r0:r1], np.float32(0.25), 0, 15)
    hist = torch.from_numpy(h.view(np.int64).copy())
    g = inputs.normal((M, 40), 1.0, seed=4)
    part = oracle.backward(x[r0:r1], g[r0:r1], np.float32(0.25), 0, 15, np.float32(50.0), 5)
    scal = torch.tensor([part["grad_q"], part["grad_alpha"]], dtype=torch.float64)
    sharding.exchange(dist, world, dW, hist, scal, None)
    if rank == 0:
        np.save(os.path.join(out_dir, "dW.npy"), dW.numpy())
        np.save(os.path.join(out_dir, "hist.npy"), hist.numpy())
        np.save(os.path.join(out_dir, "scal.npy"), scal.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_sums():
    import torch.multiprocessing as mp
    with tempfile.TemporaryDirectory() as d:
        init_file = os.path.join(d, "rendezvous")
        mp.spawn(_worker, args=(2, init_file, d), nprocs=2, join=True)
        dW = np.load(os.path.join(d, "dW.npy"))
        hist = np.load(os.path.join(d, "hist.npy"))
        scal = np.load(os.path.join(d, "scal.npy"))
    M, K, N = 301, 48, 24
    A = inputs.uniform_indices((M, K), 0, 15, seed=1)
    G = inputs.uniform_indices((M, N), -127, 127, seed=2)
    x = inputs.relu_normal((M, 40), seed=3)
    g = inputs.normal((M, 40), 1.0, seed=4)
    assert np.array_equal(dW, oracle.gemm_dw(A, G))
    _, h = oracle.hard(x, np.float32(0.25), 0, 15)
    assert np.array_equal(hist.view(np.uint64), h)
    full = oracle.backward(x, g, np.float32(0.25), 0, 15, np.float32(50.0), 5)
    assert scal[0] == pytest.approx(full["grad_q"], rel=1e-12, abs=1e-12 * full["abs_q"])
    assert scal[1] == pytest.approx(full["grad_alpha"], rel=1e-12, abs=1e-12 * full["abs_alpha"])
