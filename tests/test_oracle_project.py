"""Pins for the oracle's mask-only projection (appendix, "Mask-only Projection"): brute force, closed forms, the
equivalence the paper relies on (rows of the all-token projection), linearity, index handling.  CPU only."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O


def test_brute_force_loops():
    rng = np.random.default_rng(0)
    h = rng.standard_normal((7, 5)); w = rng.standard_normal((4, 5))
    pos = [6, 0, 3]
    got = O.mask_project(h, pos, w)
    assert got.shape == (3, 4) and got.dtype == np.float64
    for m, p in enumerate(pos):
        for v in range(4):
            acc = 0.0
            for k in range(5):
                acc += h[p][k] * w[v][k]
            assert abs(got[m, v] - acc) < 1e-14


def test_closed_forms():
    rng = np.random.default_rng(1)
    h = rng.standard_normal((6, 8))
    pos = np.array([5, 2, 2, 0])
    # identity embedding: the logits are the selected hidden rows themselves, in the order of `positions`
    assert np.array_equal(O.mask_project(h, pos, np.eye(8)), h[pos])
    # a vocabulary row of ones sums the hidden row; a one-hot row picks one feature; a zero row gives zero
    w = np.zeros((3, 8)); w[0] = 1.0; w[1, 3] = 1.0
    got = O.mask_project(h, pos, w)
    assert np.allclose(got[:, 0], h[pos].sum(1), atol=1e-14) and np.array_equal(got[:, 1], h[pos, 3]) and not got[:, 2].any()
    # w is [vocab, width]: a non-square case tells a transposed operand apart
    w2 = np.arange(16.0).reshape(2, 8)
    assert np.allclose(O.mask_project(h, [1], w2)[0], [h[1] @ w2[0], h[1] @ w2[1]], atol=1e-13)


def test_equals_rows_of_the_all_token_projection_and_is_linear():
    g = torch.Generator().manual_seed(2)
    h = torch.randn(33, 24, generator=g, dtype=torch.float64)
    w = torch.randn(50, 24, generator=g, dtype=torch.float64)
    pos = torch.randperm(33, generator=g)[:9]
    full = torch.nn.functional.linear(h, w).numpy()                 # all-token projection, library routine
    got = O.mask_project(h, pos.numpy(), w)
    assert np.abs(got - full[pos.numpy()]).max() < 1e-12
    h2 = torch.randn(33, 24, generator=g, dtype=torch.float64)
    lin = O.mask_project(2.0 * h - 3.0 * h2, pos.numpy(), w)
    assert np.abs(lin - (2.0 * got - 3.0 * O.mask_project(h2, pos.numpy(), w))).max() < 1e-11
    # bf16 inputs are widened exactly
    hb, wb = h.to(torch.bfloat16), w.to(torch.bfloat16)
    assert np.abs(O.mask_project(hb, pos.numpy(), wb) - torch.nn.functional.linear(hb.double(), wb.double()).numpy()[pos.numpy()]).max() < 1e-12


def test_empty_and_bad_positions():
    h = np.ones((4, 3)); w = np.ones((2, 3))
    assert O.mask_project(h, [], w).shape == (0, 2)
    for bad in ([4], [-1]):
        with pytest.raises(IndexError):
            O.mask_project(h, bad, w)
