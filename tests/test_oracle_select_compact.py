"""Pins for the oracle's eviction (Eq. 16) and row-copy compaction.  CPU only."""
import numpy as np
import torch

from oracle import maskkv_oracle as O


def brute_topk(seg, k):
    """Python's sorted() on (-score, index) tuples, then ascending index."""
    order = sorted(range(len(seg)), key=lambda j: (-float(seg[j]), j))
    return sorted(order[:k])


def test_select_matches_sorted_brute_force():
    rng = np.random.default_rng(0)
    for trial in range(40):
        R, Hkv = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        lens = rng.integers(1, 60, R)
        pcu = np.concatenate([[0], np.cumsum(lens)]).tolist()
        # coarse values so that ties are frequent
        sc = rng.integers(0, 6, (Hkv, pcu[-1])).astype(np.float32) / 4
        bud = np.array([[int(rng.integers(0, lens[r] + 1)) for _ in range(Hkv)] for r in range(R)])
        idx, off = O.select(sc, bud, pcu)
        for r in range(R):
            for h in range(Hkv):
                s = r * Hkv + h
                got = idx[off[s]:off[s + 1]].tolist()
                assert got == brute_topk(sc[h, pcu[r]:pcu[r + 1]], bud[r, h])


def test_select_agrees_with_library_topk_when_scores_are_distinct():
    g = torch.Generator().manual_seed(1)
    sc = torch.rand(3, 500, generator=g)
    bud = np.array([[17, 0, 500]])
    idx, off = O.select(sc.numpy(), bud, [0, 500])
    for h in range(3):
        ref = torch.topk(sc[h], int(bud[0, h])).indices.sort().values.tolist()
        assert idx[off[h]:off[h + 1]].tolist() == ref


def test_select_edge_cases():
    sc = np.ones((1, 10), np.float32)
    idx, off = O.select(sc, np.array([[4]]), [0, 10])
    assert idx.tolist() == [0, 1, 2, 3]                         # exact ties -> lowest indices
    sc = np.array([[5, 1, 5, 5, 0, 5]], np.float32)             # duplicates straddling the cut
    idx, _ = O.select(sc, np.array([[2]]), [0, 6])
    assert idx.tolist() == [0, 2]
    idx, _ = O.select(sc, np.array([[5]]), [0, 6])
    assert idx.tolist() == [0, 1, 2, 3, 5]
    idx, off = O.select(sc, np.array([[0]]), [0, 6])
    assert idx.size == 0 and off.tolist() == [0, 0]
    sc = np.array([[np.nan, 1, -np.inf, 2, np.nan]], np.float32)  # NaN ranks below every number
    idx, _ = O.select(sc, np.array([[3]]), [0, 5])
    assert idx.tolist() == [1, 2, 3]
    idx, _ = O.select(sc, np.array([[4]]), [0, 5])
    assert idx.tolist() == [0, 1, 2, 3]


def test_select_output_is_ascending_unique_in_range():
    rng = np.random.default_rng(2)
    sc = rng.random((2, 300)).astype(np.float32)
    pcu = [0, 100, 300]
    bud = np.array([[10, 100], [200, 1]])
    idx, off = O.select(sc, bud, pcu)
    for r in range(2):
        for h in range(2):
            s = r * 2 + h
            seg = idx[off[s]:off[s + 1]]
            assert (np.diff(seg) > 0).all() and seg.min() >= 0 and seg.max() < pcu[r + 1] - pcu[r]
            kept = set(seg.tolist())
            vals = sc[h, pcu[r]:pcu[r + 1]]
            if len(kept) < len(vals):
                assert vals[list(kept)].min() >= np.delete(vals, list(kept)).max()


def test_compact_is_a_byte_exact_gather():
    g = torch.Generator().manual_seed(3)
    pcu = [0, 20, 50]
    kp = torch.randn(50, 3, 8, generator=g).bfloat16()
    vp = torch.randn(50, 3, 8, generator=g).bfloat16()
    bud = np.array([[3, 0, 20], [7, 30, 1]])
    sc = torch.rand(3, 50, generator=g).numpy()
    idx, off = O.select(sc, bud, pcu)
    kc, vc = O.compact(kp, vp, idx, off, pcu)
    assert kc.dtype == torch.bfloat16 and kc.shape == (int(off[-1]), 8)
    # library gather: index_select on the flattened (token, head) axis
    flat_rows = []
    for r in range(2):
        for h in range(3):
            s = r * 3 + h
            flat_rows += [(pcu[r] + int(j)) * 3 + h for j in idx[off[s]:off[s + 1]]]
    ref_k = kp.reshape(150, 8).index_select(0, torch.tensor(flat_rows, dtype=torch.long))
    ref_v = vp.reshape(150, 8).index_select(0, torch.tensor(flat_rows, dtype=torch.long))
    assert torch.equal(kc.view(torch.int16), ref_k.view(torch.int16))
    assert torch.equal(vc.view(torch.int16), ref_v.view(torch.int16))
