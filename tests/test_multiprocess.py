"""World-size-2 check (gloo, CPU) of the data-parallel exchange used by bench.py --gpus N: each rank takes its block
of batch rows and goes through the exchange points of a layer step in their order - activation histogram before the
entropy, integer weight-gradient accumulators before the conversion to float, the activation quantizer's two scalars
at the end - with the CPU oracle standing in for the kernels; the result must equal the unsharded step (bit for bit
for everything but the two fp64 sums)."""
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
    """One rank of a data-parallel step, with the oracle standing in for the kernels: the tensors that cross ranks,
    their types and the points of the step at which they cross are those of CdlLayerStep.run(exchange=...)."""
    import torch
    import torch.distributed as dist
    dist.init_process_group("gloo", init_method=f"file://{init_file}", rank=rank, world_size=world)
    f32 = np.float32
    A, G, x, g, q_s, q_g = _step_inputs()
    r0, r1 = sharding.row_range(M_ROWS, rank, world)
    ex = sharding.StepExchange(dist, world)
    # 1. activation histogram: summed before the entropy, so that H(x) and prob_x are those of the whole batch
    _, h = oracle.hard(x[r0:r1], q_s, 0, 15)
    hist = ex.histogram(torch.from_numpy(h.view(np.int64).copy()))
    H, prob, _ = oracle.entropy(hist.numpy().view(np.uint64))
    # 2. weight-gradient accumulators: summed as integers, converted once
    bits = sharding.acc_bits_for(M_ROWS, 15, 127)
    acc = oracle.gemm_dw(A[r0:r1], G[r0:r1])
    assert np.abs(acc).max() < 2 ** 31
    acc_t = torch.from_numpy(acc.astype(np.int32 if bits == 32 else np.int64))
    ex.accumulators(acc_t)
    dW = acc_t.numpy().astype(f32) * (q_g * q_s)
    with pytest.raises(TypeError):
        ex.accumulators(torch.from_numpy(dW))                    # float dW must never be what crosses ranks
    # 3. the activation quantizer's backward pass with the global level probabilities; its two scalars are summed
    part = oracle.backward(x[r0:r1], g[r0:r1], q_s, 0, 15, f32(50.0), 5, f32(0.01), prob.astype(f32).astype(np.float64))
    scal = torch.tensor([part["grad_q"], part["grad_alpha"]], dtype=torch.float64)
    ex.batch_scalars(scal)
    assert [c[0] for c in ex.calls] == ["histogram", "accumulators", "batch_scalars"]
    assert [c[1] for c in ex.calls] == ["int64", "int32", "float64"]
    np.save(os.path.join(out_dir, f"gx{rank}.npy"), part["grad_x"])
    if rank == 0:
        np.save(os.path.join(out_dir, "dW.npy"), dW)
        np.save(os.path.join(out_dir, "hist.npy"), hist.numpy())
        np.save(os.path.join(out_dir, "scal.npy"), scal.numpy())
        np.save(os.path.join(out_dir, "H.npy"), np.array([H]))
    dist.barrier()
    dist.destroy_process_group()


M_ROWS, K_COLS, N_COLS = 301, 48, 24


def _step_inputs():
    f32 = np.float32
    A = inputs.uniform_indices((M_ROWS, K_COLS), 0, 15, seed=1)
    G = inputs.uniform_indices((M_ROWS, N_COLS), -127, 127, seed=2)
    x = inputs.relu_normal((M_ROWS, 40), seed=3)
    g = inputs.normal((M_ROWS, 40), 1.0, seed=4)
    return A, G, x, g, f32(0.25), f32(1e-3)


def test_two_ranks_reproduce_the_unsharded_step():
    import torch.multiprocessing as mp
    f32 = np.float32
    with tempfile.TemporaryDirectory() as d:
        init_file = os.path.join(d, "rendezvous")
        mp.spawn(_worker, args=(2, init_file, d), nprocs=2, join=True)
        dW, hist, scal, H = (np.load(os.path.join(d, n + ".npy")) for n in ("dW", "hist", "scal", "H"))
        gx = np.concatenate([np.load(os.path.join(d, f"gx{r}.npy")) for r in range(2)])
    A, G, x, g, q_s, q_g = _step_inputs()
    _, h = oracle.hard(x, q_s, 0, 15)
    assert np.array_equal(hist.view(np.uint64), h)
    refH, prob, _ = oracle.entropy(h)
    assert H[0] == refH                                     # the entropy of the summed histogram, not a sum of entropies
    assert np.array_equal(dW, oracle.gemm_dw(A, G).astype(f32) * (q_g * q_s))        # bit for bit
    full = oracle.backward(x, g, q_s, 0, 15, f32(50.0), 5, f32(0.01), prob.astype(f32).astype(np.float64))
    assert np.array_equal(gx, full["grad_x"])               # every rank differentiated through the global probabilities
    assert scal[0] == pytest.approx(full["grad_q"], rel=1e-12, abs=1e-12 * full["abs_q"])
    assert scal[1] == pytest.approx(full["grad_alpha"], rel=1e-12, abs=1e-12 * full["abs_alpha"])


def test_accumulator_width_for_the_all_reduce():
    assert sharding.acc_bits_for(50176 * 8, 15, 127) == 32
    assert sharding.acc_bits_for(1127288, 15, 127) == 32 and sharding.acc_bits_for(1127289, 15, 127) == 64
