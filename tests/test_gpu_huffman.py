"""GPU parity of cdl_huffman_lengths against the oracle's textbook construction: the coded size is unique and must
match exactly; the individual lengths may differ where equal weights were paired differently, so they are checked
for being a valid optimal prefix code (used levels only, Kraft sum exactly one, same total)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
import paper_2501_09849_b200 as cdl
from paper_2501_09849_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    cdl.load_library()
    return torch


def run(torch, h):
    h = np.asarray(h, dtype=np.uint64)
    hd = torch.from_numpy(h.view(np.int64).copy()).cuda()
    lengths = torch.full((h.size,), 77, dtype=torch.uint8, device="cuda")
    total = torch.zeros(1, dtype=torch.int64, device="cuda")
    avg = torch.zeros(1, dtype=torch.float64, device="cuda")
    cdl.cdl_huffman_lengths(hd, h.size, lengths, total, avg)
    torch.cuda.synchronize()
    return lengths.cpu().numpy().astype(np.int64), int(total.item()), float(avg.item())


def check(torch, h):
    h = np.asarray(h, dtype=np.uint64)
    lengths, total, avg = run(torch, h)
    ref_len, ref_total = oracle.huffman_lengths(h)
    assert total == ref_total
    assert total == int(sum(int(c) * int(l) for c, l in zip(h, lengths)))
    assert all((l > 0) == (c > 0) for l, c in zip(lengths, h))
    used = int((h > 0).sum())
    if used >= 2:
        assert sum(Fraction(1, 2 ** int(l)) for l in lengths if l > 0) == 1
    elif used == 1:
        assert lengths[h > 0][0] == 1
    n = int(h.sum())
    assert avg == (total / n if n else 0.0)
    return lengths, ref_len


def test_worked_example_and_closed_forms(torch):
    lengths, _ = check(torch, [45, 13, 12, 16, 9, 5])
    assert list(lengths) == [1, 3, 3, 3, 4, 4]
    lengths, _ = check(torch, [8, 4, 2, 1, 1])
    assert list(lengths) == [1, 2, 3, 4, 4]
    for b in (1, 3, 8):
        lengths, _ = check(torch, [5] * (1 << b))
        assert set(lengths) == {b}


def test_degenerate_and_extreme_histograms(torch):
    check(torch, [0])
    check(torch, [7])
    check(torch, [0, 0, 0, 0])
    check(torch, [0, 9, 0])
    check(torch, [3, 0, 5])
    check(torch, [1] + [0] * 254 + [1])
    check(torch, [2 ** 40 + k for k in range(256)])                 # counts beyond 32 bits
    fib = [1, 1]
    while len(fib) < 60:
        fib.append(fib[-1] + fib[-2])
    lengths, _ = check(torch, fib)                                   # the deepest possible tree for its size
    assert max(lengths) == 59


@pytest.mark.parametrize("seed", range(8))
def test_random_histograms_with_ties_and_gaps(torch, seed):
    rng = np.random.default_rng(seed)
    nlev = int(rng.integers(1, 257))
    h = rng.integers(0, 50 if seed % 2 else 10 ** 9, nlev) * (rng.random(nlev) < 0.7)
    check(torch, h)


def test_histogram_of_a_quantized_tensor(torch):
    x = inputs.normal((1 << 20,), 1.0, seed=5)
    xd = torch.from_numpy(x).cuda()
    P = cdl.QuantParams(0.25, -15, 15)
    hist = torch.zeros(31, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_hard(xd, x.size, P, None, hist)
    H = torch.zeros(1, dtype=torch.float64, device="cuda")
    cdl.cdl_index_entropy(hist, 31, H)
    avg = torch.zeros(1, dtype=torch.float64, device="cuda")
    cdl.cdl_huffman_lengths(hist, 31, None, None, avg)
    torch.cuda.synchronize()
    _, ref_total = oracle.huffman_lengths(hist.cpu().numpy())
    assert avg.item() == ref_total / x.size
    assert H.item() <= avg.item() < H.item() + 1.0                  # the rate the entropy constraint stands for
