"""Pins for the oracle's scoring step (Eq. 6-7 and the sums of Eq. 14): brute force on tiny inputs,
a library softmax, closed forms and invariants.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O


def _rand(rng, *shape):
    return rng.standard_normal(shape)


def brute_force_score(q, kp, km, scale):
    """Scalar loops only (math.exp), one request: returns I [H_kv][N], Sp [H_kv], Sm [H_kv]."""
    M, H, d = q.shape
    N, Hkv, _ = kp.shape
    g = H // Hkv
    imp = [[0.0] * N for _ in range(Hkv)]
    sp = [0.0] * Hkv
    sm = [0.0] * Hkv
    for h in range(H):
        hk = h // g
        for i in range(M):
            logits = []
            for j in range(N + M):
                krow = kp[j, hk] if j < N else km[j - N, hk]
                acc = 0.0
                for c in range(d):
                    acc += q[i, h, c] * krow[c]
                logits.append(acc * scale)
            den = sum(math.exp(x) for x in logits)          # no max subtraction: tiny logits
            for j in range(N + M):
                a = math.exp(logits[j]) / den
                if j < N:
                    imp[hk][j] += a
                    sp[hk] += a
                else:
                    sm[hk] += a
    return np.array(imp), np.array(sp), np.array(sm)


@pytest.mark.parametrize("H,Hkv", [(2, 2), (4, 2), (3, 1)])
def test_score_matches_scalar_brute_force(H, Hkv):
    rng = np.random.default_rng(1)
    M, N, d = 3, 7, 4
    q, kp, km = _rand(rng, M, H, d), _rand(rng, N, Hkv, d), _rand(rng, M, Hkv, d)
    s, mp, mm = O.score(q, kp, km, [0, N], [0, M], scale=0.5)
    bi, bp, bm = brute_force_score(q, kp, km, 0.5)
    np.testing.assert_allclose(s, bi, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(mp[0], bp, rtol=1e-12)
    np.testing.assert_allclose(mm[0], bm, rtol=1e-12)


def test_score_matches_library_softmax():
    """Special case (one request, MHA) reduces to torch.softmax(QK^T*scale)[:, :N].sum(0) in fp64."""
    g = torch.Generator().manual_seed(7)
    M, N, H, d = 16, 50, 3, 8
    q = torch.randn(M, H, d, generator=g, dtype=torch.float64)
    kp = torch.randn(N, H, d, generator=g, dtype=torch.float64)
    km = torch.randn(M, H, d, generator=g, dtype=torch.float64)
    s, mp, mm = O.score(q, kp, km, [0, N], [0, M])
    for h in range(H):
        kf = torch.cat([kp[:, h], km[:, h]], 0)
        a = torch.softmax(q[:, h] @ kf.T / math.sqrt(d), dim=-1)
        np.testing.assert_allclose(s[h], a[:, :N].sum(0).numpy(), rtol=1e-12)
        np.testing.assert_allclose(mp[0, h], a[:, :N].sum().item(), rtol=1e-12)
        np.testing.assert_allclose(mm[0, h], a[:, N:].sum().item(), rtol=1e-12)


def test_attention_rows_sum_to_one_and_mass_identity():
    rng = np.random.default_rng(2)
    M, N, H, Hkv, d = 12, 40, 6, 2, 16
    q, kp, km = 3 * _rand(rng, M, H, d), 3 * _rand(rng, N, Hkv, d), 3 * _rand(rng, M, Hkv, d)
    a, _ = O.attention_weights(q[:, 0], np.concatenate([kp[:, 0], km[:, 0]]), 0.25)
    assert np.abs(a.sum(1) - 1).max() < 1e-12
    assert (a > 0).all()
    s, mp, mm = O.score(q, kp, km, [0, N], [0, M])
    # every row of A sums to 1, so S_{m->p} + S_{m->m} = M * g
    np.testing.assert_allclose(mp + mm, M * (H // Hkv), rtol=1e-12)
    np.testing.assert_allclose(s.sum(1), mp[0], rtol=1e-12)


def test_uniform_attention_closed_form():
    """Q = 0 (or all keys equal) makes every row uniform: I_j = M*g/(N+M), P = N/(N+M)."""
    rng = np.random.default_rng(3)
    M, N, H, Hkv, d = 8, 24, 4, 2, 8
    kp, km = _rand(rng, N, Hkv, d), _rand(rng, M, Hkv, d)
    s, mp, mm = O.score(np.zeros((M, H, d)), kp, km, [0, N], [0, M])
    np.testing.assert_allclose(s, M * 2 / (N + M), rtol=1e-13)
    np.testing.assert_allclose(mp / (mp + mm), N / (N + M), rtol=1e-13)
    same = np.broadcast_to(rng.standard_normal((1, Hkv, d)), (N, Hkv, d))
    s2, _, _ = O.score(_rand(rng, M, H, d), same, same[:M], [0, N], [0, M])
    np.testing.assert_allclose(s2, M * 2 / (N + M), rtol=1e-12)


def test_key_shift_invariance_and_permutation_equivariance():
    rng = np.random.default_rng(4)
    M, N, H, d = 10, 33, 2, 8
    q, kp, km = _rand(rng, M, H, d), _rand(rng, N, H, d), _rand(rng, M, H, d)
    s, mp, mm = O.score(q, kp, km, [0, N], [0, M])
    v = rng.standard_normal((1, H, d))
    s2, mp2, _ = O.score(q, kp + v, km + v, [0, N], [0, M])      # a row-constant logit shift
    np.testing.assert_allclose(s2, s, rtol=1e-10)
    perm = rng.permutation(N)
    s3, _, _ = O.score(q, kp[perm], km, [0, N], [0, M])
    np.testing.assert_allclose(s3, s[:, perm], rtol=1e-12)
    kd = kp.copy()
    kd[5] = kd[17]                                                # duplicated key -> equal scores
    s4, _, _ = O.score(q, kd, km, [0, N], [0, M])
    np.testing.assert_allclose(s4[:, 5], s4[:, 17], rtol=1e-13)


def test_dominant_key_collects_all_mass():
    rng = np.random.default_rng(5)
    M, N, H, d = 6, 20, 1, 8
    q = np.abs(_rand(rng, M, H, d)) + 0.5
    kp, km = 0.01 * _rand(rng, N, H, d), 0.01 * _rand(rng, M, H, d)
    kp[11] = 200.0                                                # aligned with every (positive) query
    s, mp, mm = O.score(q, kp, km, [0, N], [0, M])
    assert abs(s[0, 11] - M) < 1e-9 and abs(mp[0, 0] - M) < 1e-9 and mm[0, 0] < 1e-9


def test_row_weights_select_single_row_and_are_linear():
    rng = np.random.default_rng(6)
    M, N, H, d = 5, 9, 1, 4
    q, kp, km = _rand(rng, M, H, d), _rand(rng, N, H, d), _rand(rng, M, H, d)
    a, _ = O.attention_weights(q[:, 0], np.concatenate([kp[:, 0], km[:, 0]]), 1 / math.sqrt(d))
    for i in range(M):
        w = np.zeros(M)
        w[i] = 1
        s, _, _ = O.score(q, kp, km, [0, N], [0, M], row_weights=w)
        np.testing.assert_allclose(s[0], a[i, :N], rtol=1e-13)
    w = rng.uniform(0, 2, M)
    s, mp, mm = O.score(q, kp, km, [0, N], [0, M], row_weights=w)
    np.testing.assert_allclose(s[0], (w[:, None] * a[:, :N]).sum(0), rtol=1e-12)
    np.testing.assert_allclose(mp[0, 0] + mm[0, 0], w.sum(), rtol=1e-12)


def test_gqa_is_sum_over_group_and_batch_is_independent():
    rng = np.random.default_rng(8)
    M, H, Hkv, d = 4, 6, 2, 8
    lens = [11, 5, 17]
    pcu = [0, 11, 16, 33]
    lcu = [0, 4, 8, 12]
    q, kp, km = _rand(rng, 12, H, d), _rand(rng, 33, Hkv, d), _rand(rng, 12, Hkv, d)
    s, mp, mm = O.score(q, kp, km, pcu, lcu)
    g = H // Hkv
    for r in range(3):
        qs, ks, ms = q[lcu[r]:lcu[r + 1]], kp[pcu[r]:pcu[r + 1]], km[lcu[r]:lcu[r + 1]]
        # MHA on keys repeated per query head, summed over each group afterwards
        s1, mp1, mm1 = O.score(qs, np.repeat(ks, g, axis=1), np.repeat(ms, g, axis=1), [0, lens[r]], [0, M])
        np.testing.assert_allclose(s[:, pcu[r]:pcu[r + 1]], s1.reshape(Hkv, g, -1).sum(1), rtol=1e-12)
        np.testing.assert_allclose(mp[r], mp1[0].reshape(Hkv, g).sum(1), rtol=1e-12)
        np.testing.assert_allclose(mm[r], mm1[0].reshape(Hkv, g).sum(1), rtol=1e-12)


def test_bf16_inputs_are_widened_exactly():
    g = torch.Generator().manual_seed(3)
    q = torch.randn(4, 2, 8, generator=g).bfloat16()
    kp = torch.randn(9, 2, 8, generator=g).bfloat16()
    km = torch.randn(4, 2, 8, generator=g).bfloat16()
    s1, _, _ = O.score(q, kp, km, [0, 9], [0, 4])
    s2, _, _ = O.score(q.double().numpy(), kp.double().numpy(), km.double().numpy(), [0, 9], [0, 4])
    assert (s1 == s2).all()
