"""Pins for the oracle's attention over [compacted prompt ; live region].  CPU only."""
import math

import numpy as np
import torch
import torch.nn.functional as F

from oracle import maskkv_oracle as O


def _case(seed, R=2, H=4, Hkv=2, d=8, M=5, lens=(13, 9)):
    g = torch.Generator().manual_seed(seed)
    pcu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    lcu = [r * M for r in range(R + 1)]
    t = dict(
        q=torch.randn(R * M, H, d, generator=g, dtype=torch.float64),
        kl=torch.randn(R * M, Hkv, d, generator=g, dtype=torch.float64),
        vl=torch.randn(R * M, Hkv, d, generator=g, dtype=torch.float64),
        kp=torch.randn(pcu[-1], Hkv, d, generator=g, dtype=torch.float64),
        vp=torch.randn(pcu[-1], Hkv, d, generator=g, dtype=torch.float64),
        sc=torch.rand(Hkv, pcu[-1], generator=g).numpy(),
    )
    return t, pcu, lcu


def test_attend_matches_library_sdpa():
    t, pcu, lcu = _case(0)
    R, H, Hkv, M = 2, 4, 2, 5
    bud = np.array([[4, 0], [9, 3]])
    idx, off = O.select(t["sc"], bud, pcu)
    kc, vc = O.compact(t["kp"], t["vp"], idx, off, pcu)
    out, lse = O.attend(t["q"], t["kl"], t["vl"], kc, vc, off, lcu, Hkv)
    for r in range(R):
        for h in range(H):
            hk, s = h // 2, r * Hkv + h // 2
            keys = torch.cat([kc[off[s]:off[s + 1]], t["kl"][lcu[r]:lcu[r + 1], hk]])
            vals = torch.cat([vc[off[s]:off[s + 1]], t["vl"][lcu[r]:lcu[r + 1], hk]])
            q = t["q"][lcu[r]:lcu[r + 1], h]
            ref = F.scaled_dot_product_attention(q[None, None], keys[None, None], vals[None, None])[0, 0]
            np.testing.assert_allclose(out[lcu[r]:lcu[r + 1], h], ref.numpy(), rtol=1e-11, atol=1e-13)
            ref_lse = torch.logsumexp(q @ keys.T / math.sqrt(q.shape[-1]), dim=-1)
            np.testing.assert_allclose(lse[h, lcu[r]:lcu[r + 1]], ref_lse.numpy(), rtol=1e-12)


def test_full_budget_equals_full_attention():
    """k >= N for every head: nothing is evicted, so the result is attention over the original K/V."""
    t, pcu, lcu = _case(1)
    R, H, Hkv = 2, 4, 2
    bud = np.array([[13, 13], [9, 9]])
    idx, off = O.select(t["sc"], bud, pcu)
    kc, vc = O.compact(t["kp"], t["vp"], idx, off, pcu)
    out, _ = O.attend(t["q"], t["kl"], t["vl"], kc, vc, off, lcu, Hkv)
    for r in range(R):
        for h in range(H):
            hk = h // 2
            keys = torch.cat([t["kp"][pcu[r]:pcu[r + 1], hk], t["kl"][lcu[r]:lcu[r + 1], hk]])
            vals = torch.cat([t["vp"][pcu[r]:pcu[r + 1], hk], t["vl"][lcu[r]:lcu[r + 1], hk]])
            q = t["q"][lcu[r]:lcu[r + 1], h]
            ref = F.scaled_dot_product_attention(q[None, None], keys[None, None], vals[None, None])[0, 0]
            np.testing.assert_allclose(out[lcu[r]:lcu[r + 1], h], ref.numpy(), rtol=1e-11, atol=1e-13)


def test_closed_forms_single_key_zero_query_and_order_invariance():
    t, pcu, lcu = _case(2, R=1, lens=(6,))
    Hkv = 2
    # Q = 0: every weight equal -> output = mean of [kept V ; live V]
    bud = np.array([[3, 2]])
    idx, off = O.select(t["sc"], bud, pcu)
    kc, vc = O.compact(t["kp"], t["vp"], idx, off, pcu)
    out, lse = O.attend(torch.zeros_like(t["q"]), t["kl"], t["vl"], kc, vc, off, lcu, Hkv)
    for h in range(4):
        hk = h // 2
        vals = torch.cat([vc[off[hk]:off[hk + 1]], t["vl"][:, hk]])
        np.testing.assert_allclose(out[:, h], np.broadcast_to(vals.mean(0).numpy(), out[:, h].shape), rtol=1e-12)
        np.testing.assert_allclose(lse[h], math.log(vals.shape[0]), rtol=1e-12)
    # one live key, empty compacted cache: output = that V row whatever q is
    off0 = np.zeros(3, np.int32)
    out, _ = O.attend(t["q"][:1], t["kl"][:1], t["vl"][:1], kc[:0], vc[:0], off0, [0, 1], Hkv)
    for h in range(4):
        np.testing.assert_allclose(out[0, h], t["vl"][0, h // 2].numpy(), rtol=1e-13)
    # the order of rows inside a compacted segment does not matter
    out1, _ = O.attend(t["q"], t["kl"], t["vl"], kc, vc, off, lcu, Hkv)
    perm = torch.tensor([2, 0, 1, 4, 3])
    out2, _ = O.attend(t["q"], t["kl"], t["vl"], kc[perm], vc[perm], off, lcu, Hkv)
    np.testing.assert_allclose(out1, out2, rtol=1e-12, atol=1e-14)


def test_partial_refresh_rows_are_rows_of_the_full_step_and_match_the_library():
    """With rows_cu the queries are a subset of the live rows while the keys stay all of them: the outputs must be
    the corresponding rows of the full step, and each row must match the library's attention over
    [segment ; all live rows]."""
    t, pcu, lcu = _case(3)
    R, H, Hkv, M = 2, 4, 2, 5
    bud = np.array([[6, 2], [0, 9]])
    idx, off = O.select(t["sc"], bud, pcu)
    kc, vc = O.compact(t["kp"], t["vp"], idx, off, pcu)
    full, full_lse = O.attend(t["q"], t["kl"], t["vl"], kc, vc, off, lcu, Hkv)
    picks = [[4, 1], [2]]                                              # refreshed rows of each request, in list order
    rows = [lcu[r] + i for r in range(R) for i in picks[r]]
    rows_cu = [0, 2, 3]
    out, lse = O.attend(t["q"][rows], t["kl"], t["vl"], kc, vc, off, lcu, Hkv, rows_cu=rows_cu)
    assert out.shape == (3, H, 8) and lse.shape == (H, 3)
    np.testing.assert_allclose(out, full[rows], rtol=1e-12, atol=1e-14)      # the library matmul rounds differently per shape
    np.testing.assert_allclose(lse, full_lse[:, rows], rtol=1e-13)
    for n, row in enumerate(rows):
        r = 0 if n < 2 else 1
        for h in range(H):
            hk, s = h // 2, r * Hkv + h // 2
            keys = torch.cat([kc[off[s]:off[s + 1]], t["kl"][lcu[r]:lcu[r + 1], hk]])
            vals = torch.cat([vc[off[s]:off[s + 1]], t["vl"][lcu[r]:lcu[r + 1], hk]])
            ref = F.scaled_dot_product_attention(t["q"][row, h][None, None, None], keys[None, None], vals[None, None])[0, 0, 0]
            np.testing.assert_allclose(out[n, h], ref.numpy(), rtol=1e-11, atol=1e-13)
    # a request without refreshed rows contributes nothing; no rows at all gives empty outputs
    out2, _ = O.attend(t["q"][rows[2:]], t["kl"], t["vl"], kc, vc, off, lcu, Hkv, rows_cu=[0, 0, 1])
    np.testing.assert_allclose(out2, full[rows[2:]], rtol=1e-12, atol=1e-14)
    out3, lse3 = O.attend(t["q"][:0], t["kl"], t["vl"], kc, vc, off, lcu, Hkv, rows_cu=[0, 0, 0])
    assert out3.shape == (0, H, 8) and lse3.shape == (H, 0)
