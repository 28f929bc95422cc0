"""Pins for the oracle's voter-set scores (the paper's voting ablation: mask, prompt, all tokens, a trailing window):
brute force with the softmax written out, additivity over disjoint voter sets, total attention per voter, agreement
with the mask-voting scorer on its special case.  CPU only."""
import math

import numpy as np
import torch

from oracle import maskkv_oracle as O


def _seq(T, H, Hkv, d, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(T, H, d, generator=g, dtype=torch.float64), torch.randn(T, Hkv, d, generator=g, dtype=torch.float64)


def test_brute_force_with_the_softmax_written_out():
    T, n_p, H, Hkv, d = 7, 4, 4, 2, 3
    q, k = _seq(T, H, Hkv, d, 0)
    voters = [1, 5, 6]
    got = O.vote_scores(q, k, voters, n_p)
    want = np.zeros((Hkv, n_p))
    for hk in range(Hkv):
        for h in (2 * hk, 2 * hk + 1):
            for i in voters:
                logits = [sum(float(q[i, h, t]) * float(k[j, hk, t]) for t in range(d)) / math.sqrt(d) for j in range(T)]
                z = sum(math.exp(x) for x in logits)
                for j in range(n_p):
                    want[hk, j] += math.exp(logits[j]) / z
    assert np.abs(got - want).max() < 1e-13


def test_disjoint_voter_sets_add_and_every_voter_spends_one_unit():
    T, n_p, H, Hkv, d = 40, 25, 4, 4, 8
    q, k = _seq(T, H, Hkv, d, 1)
    prompt_rows, mask_rows = list(range(n_p)), list(range(n_p, T))
    all_v = O.vote_scores(q, k, prompt_rows + mask_rows, n_p)
    assert np.abs(all_v - (O.vote_scores(q, k, prompt_rows, n_p) + O.vote_scores(q, k, mask_rows, n_p))).max() < 1e-12
    # over ALL tokens as targets a voter's attention sums to one per query head
    full = O.vote_scores(q, k, mask_rows, T)
    assert np.allclose(full.sum(axis=1), len(mask_rows) * (H // 4), atol=1e-12)
    assert O.vote_scores(q, k, [], n_p).sum() == 0.0
    # the order of the voters and repeats: a sum over rows
    assert np.abs(O.vote_scores(q, k, mask_rows[::-1], n_p) - O.vote_scores(q, k, mask_rows, n_p)).max() < 1e-13
    assert np.abs(O.vote_scores(q, k, [3, 3], n_p) - 2 * O.vote_scores(q, k, [3], n_p)).max() < 1e-13


def test_mask_voting_is_the_scorer_of_the_hot_path():
    T, n_p, H, Hkv, d = 50, 37, 6, 2, 16
    q, k = _seq(T, H, Hkv, d, 2)
    sc, mp, mm = O.score(q[n_p:], k[:n_p], k[n_p:], [0, n_p], [0, T - n_p])
    got = O.vote_scores(q, k, range(n_p, T), n_p)
    assert np.abs(got - sc).max() < 1e-12
    assert np.allclose(got.sum(axis=1), mp[0], atol=1e-12)
    # uniform attention: identical keys give every prompt token |voters| * g / T
    k0 = torch.ones_like(k)
    u = O.vote_scores(q, k0, range(10), n_p)
    assert np.allclose(u, 10 * (H // Hkv) / T, atol=1e-13)
    # a custom scale is honoured: scale 0 is read as the default, a tiny scale flattens the softmax
    flat = O.vote_scores(q, k, range(10), n_p, scale=1e-12)
    assert np.allclose(flat, 10 * (H // Hkv) / T, atol=1e-9)
