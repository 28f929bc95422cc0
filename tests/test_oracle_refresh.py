"""Pins for the oracle's response-token refresh rule (appendix: cos(V_t, V_{t-1}) < delta, union with the periodic
refresh): closed forms, a library cosine, invariances.  CPU only."""
import math

import numpy as np
import torch

from oracle import maskkv_oracle as O


def test_closed_forms_and_strict_inequality():
    rng = np.random.default_rng(0)
    v = rng.standard_normal((9, 16))
    cos, ref, idx = O.refresh_set(v, v, 0.999)
    assert np.allclose(cos, 1.0, atol=1e-15) and not ref.any() and idx.size == 0      # unchanged features: nothing to refresh
    cos, ref, idx = O.refresh_set(v, -v, -0.5)
    assert np.allclose(cos, -1.0, atol=1e-15) and ref.all() and np.array_equal(idx, np.arange(9))
    # rows rotated by known angles against a threshold cos(0.2): exactly the rows turned further than 0.2 rad
    th = np.array([0.0, 0.1, 0.2, 0.3, 1.0, math.pi / 2, 3.0])
    a = np.tile(np.array([[2.0, 0.0]]), (th.size, 1))
    b = np.stack([0.5 * np.cos(th), 0.5 * np.sin(th)], axis=1)                         # lengths do not matter
    cos, ref, idx = O.refresh_set(a, b, math.cos(0.25))
    assert np.allclose(cos, np.cos(th), atol=1e-15)
    assert np.array_equal(idx, np.array([3, 4, 5, 6], dtype=np.int32))
    # the inequality is strict: a row exactly at the threshold stays cached
    e = np.array([[1.0, 0.0], [1.0, 0.0]]); f = np.array([[0.0, 1.0], [1.0, 0.0]])
    _, ref, _ = O.refresh_set(e, f, 0.0)
    assert not ref.any()
    _, ref, _ = O.refresh_set(e, f, 1e-12)
    assert ref.tolist() == [True, False]


def test_periodic_refresh_takes_every_row():
    rng = np.random.default_rng(1)
    v = rng.standard_normal((5, 8))
    for step, t_r, want_all in ((0, 4, True), (8, 4, True), (7, 4, False), (3, 0, False), (3, None, False)):
        _, ref, idx = O.refresh_set(v, v, 0.5, step, t_r)
        assert ref.all() == want_all and idx.size == (5 if want_all else 0)


def test_matches_library_cosine_symmetry_and_zero_rows():
    g = torch.Generator().manual_seed(2)
    a = torch.randn(64, 40, generator=g, dtype=torch.float64)
    b = a + torch.randn(64, 40, generator=g, dtype=torch.float64) * torch.linspace(0, 2, 64, dtype=torch.float64)[:, None]
    lib = torch.nn.functional.cosine_similarity(a, b, dim=1).numpy()
    cos, ref, idx = O.refresh_set(a, b, 0.7)
    assert np.abs(cos - lib).max() < 1e-13
    assert np.array_equal(ref, lib < 0.7) and np.array_equal(idx, np.nonzero(lib < 0.7)[0])
    cos2, ref2, _ = O.refresh_set(b, 5.0 * a, 0.7)                                     # symmetric, scale-free
    assert np.abs(cos2 - cos).max() < 1e-13 and np.array_equal(ref2, ref)
    z = np.zeros((2, 4)); w = np.ones((2, 4))
    cos, ref, _ = O.refresh_set(z, w, 0.1)
    assert cos.tolist() == [0.0, 0.0] and ref.all()                                    # zero row: cosine 0
    # bf16 inputs are widened exactly
    ab, bb = a.to(torch.bfloat16), b.to(torch.bfloat16)
    cos3, _, _ = O.refresh_set(ab, bb, 0.7)
    assert np.abs(cos3 - torch.nn.functional.cosine_similarity(ab.double(), bb.double(), dim=1).numpy()).max() < 1e-13
