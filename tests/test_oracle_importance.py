"""Pins for the oracle's layer-importance score (Eq. 8): closed forms, invariances, a library cosine.  CPU only."""
import math

import numpy as np
import torch

from oracle import maskkv_oracle as O


def test_closed_forms():
    rng = np.random.default_rng(0)
    h = rng.standard_normal((17, 12))
    assert abs(O.layer_importance(h, h)) < 1e-14                       # identical states: cosine 1 everywhere
    assert abs(O.layer_importance(h, -h) - 2.0) < 1e-14                # opposite: cosine -1
    assert abs(O.layer_importance(h, 3.7 * h)) < 1e-14                 # scale of the output does not matter
    e = np.zeros((4, 6)); f = np.zeros((4, 6))
    e[:, 0] = 1; f[:, 1] = 1
    assert abs(O.layer_importance(e, f) - 1.0) < 1e-15                 # orthogonal rows: cosine 0
    # one row rotated by a known angle, the others untouched: I = (1 - cos(theta)) / n
    g = np.tile(np.array([[1.0, 0.0]]), (5, 1)); g2 = g.copy()
    th = 0.3
    g2[2] = [math.cos(th), math.sin(th)]
    assert abs(O.layer_importance(g, g2) - (1 - math.cos(th)) / 5) < 1e-15


def test_matches_library_cosine_and_is_row_permutation_invariant():
    g = torch.Generator().manual_seed(1)
    a = torch.randn(40, 33, generator=g, dtype=torch.float64)
    b = a + 0.5 * torch.randn(40, 33, generator=g, dtype=torch.float64)
    ref = 1.0 - torch.nn.functional.cosine_similarity(a, b, dim=1).mean().item()
    assert abs(O.layer_importance(a, b) - ref) < 1e-13
    perm = torch.randperm(40, generator=g)
    assert abs(O.layer_importance(a[perm], b[perm]) - ref) < 1e-13
    assert abs(O.layer_importance(b, a) - ref) < 1e-13                 # symmetric in its arguments


def test_zero_rows_count_as_cosine_zero_and_bf16_is_widened_exactly():
    a = np.array([[1.0, 2.0], [0.0, 0.0], [3.0, 0.0]]); b = np.array([[1.0, 2.0], [5.0, 1.0], [0.0, 0.0]])
    assert abs(O.layer_importance(a, b) - (1 - 1 / 3)) < 1e-15
    g = torch.Generator().manual_seed(2)
    x = torch.randn(9, 16, generator=g).bfloat16(); y = torch.randn(9, 16, generator=g).bfloat16()
    assert O.layer_importance(x, y) == O.layer_importance(x.double().numpy(), y.double().numpy())
