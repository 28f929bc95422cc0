"""GPU parity of the voter sets of the paper's voting ablation (mask tokens, prompt tokens, all tokens, a trailing
window of the prompt) through maskkv_score_all_keys, against the oracle's plain definition: importance of prompt token
j = sum over the voting rows i of A_ij, A = row softmax over all tokens of the sequence.

The call scores every key of [k_prompt ; k_mask] from the rows of q_mask, so a voter set is expressed by passing the
voters' queries as q_mask with their own keys as k_mask and every other token's keys as k_prompt; a prompt token's
importance then comes from scores_live if it votes and from scores if it does not."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from pipeline import assert_scores_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def _sequence(T, H, Hkv, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(T, H, d, generator=g).to(dtype)
    k = torch.randn(T, Hkv, d, generator=g).to(dtype)
    return q, k


def _vote(ctx, q, k, voters, n_prompt):
    """Importance of the n_prompt prompt tokens under the voter set `voters` (row indices, ascending), on the device."""
    from paper_2510_09309_b200 import binding as B
    T, H, d = q.shape
    Hkv = k.shape[1]
    voters = np.asarray(voters, dtype=np.int64)
    others = np.setdiff1d(np.arange(T), voters)
    dev = ctx.device
    qv = q[voters].contiguous().to(dev)
    kv = k[voters].contiguous().to(dev)
    ko = k[others].contiguous().to(dev)
    p = B.Problem(q.dtype, H, Hkv, d, [0, len(others)], [0, len(voters)], dev)
    ws = torch.empty(max(ctx.maskkv_workspace_bytes(p), 16), dtype=torch.uint8, device=dev)
    scores = torch.full((Hkv, max(len(others), 1)), float("nan"), dtype=torch.float32, device=dev)
    live = torch.full((Hkv, max(len(voters), 1)), float("nan"), dtype=torch.float32, device=dev)
    mp = torch.zeros((1, Hkv), dtype=torch.float32, device=dev)
    mm = torch.zeros((1, Hkv), dtype=torch.float32, device=dev)
    ctx.maskkv_score_all_keys(p, qv, ko if len(others) else None, kv, scores if len(others) else None, live, mp, mm, ws)
    torch.cuda.synchronize()
    assert ctx.maskkv_check_status() == 0
    imp = np.zeros((Hkv, T), np.float32)
    imp[:, others] = scores.cpu().numpy()[:, :len(others)]
    imp[:, voters] = live.cpu().numpy()[:, :len(voters)]
    g = H // Hkv
    # every voter spends one unit of attention per query head; the two masses split it between the two tensors
    np.testing.assert_allclose(mp.cpu().numpy() + mm.cpu().numpy(), len(voters) * g, rtol=2e-4)
    np.testing.assert_allclose(imp[:, voters].sum(axis=1), mm.cpu().numpy()[0], rtol=2e-4)
    return imp[:, :n_prompt]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_voter_sets_small(ctx, dtype):
    n_p, n_m, H, Hkv, d = 700, 90, 4, 2, 64
    T = n_p + n_m
    q, k = _sequence(T, H, Hkv, d, dtype, 3)
    sets = {
        "mask": np.arange(n_p, T),
        "prompt": np.arange(n_p),                      # 700 voters: several query blocks per head
        "all": np.arange(T),                           # no non-voting key at all
        "window": np.arange(n_p - 32, n_p),            # the last 32 prompt tokens observe the rest
    }
    got = {}
    for name, voters in sets.items():
        got[name] = _vote(ctx, q, k, voters, n_p)
        ref = O.vote_scores(q, k, voters, n_p)
        assert_scores_close(got[name], ref, what=f"{name}-voting")
    # disjoint voter sets add up (fp32 sums in different orders)
    np.testing.assert_allclose(got["all"], got["prompt"] + got["mask"], rtol=1e-4)


def test_mask_voting_through_both_entry_points_gives_the_same_bits(ctx):
    from paper_2510_09309_b200 import binding as B
    n_p, n_m, H, Hkv, d = 1500, 200, 8, 8, 128
    q, k = _sequence(n_p + n_m, H, Hkv, d, torch.bfloat16, 5)
    dev = ctx.device
    qm, kp, km = q[n_p:].contiguous().to(dev), k[:n_p].contiguous().to(dev), k[n_p:].contiguous().to(dev)
    p = B.Problem(torch.bfloat16, H, Hkv, d, [0, n_p], [0, n_m], dev)
    ws = torch.empty(ctx.maskkv_workspace_bytes(p), dtype=torch.uint8, device=dev)
    outs = []
    for with_live in (False, True):
        scores = torch.zeros((Hkv, n_p), dtype=torch.float32, device=dev)
        live = torch.zeros((Hkv, n_m), dtype=torch.float32, device=dev)
        mp = torch.zeros((1, Hkv), dtype=torch.float32, device=dev); mm = torch.zeros_like(mp)
        if with_live:
            ctx.maskkv_score_all_keys(p, qm, kp, km, scores, live, mp, mm, ws)
        else:
            ctx.maskkv_score(p, qm, kp, km, scores, mp, mm, ws)
        torch.cuda.synchronize()
        outs.append((scores.cpu(), mp.cpu(), mm.cpu(), live.cpu()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])
    assert not outs[0][3].any()                                        # maskkv_score leaves the extra output alone
    full = O.vote_scores(q, k, np.arange(n_p, n_p + n_m), n_p + n_m)
    assert_scores_close(outs[1][3].numpy(), full[:, n_p:], what="live columns")


def test_all_voting_at_4k_sampled_heads(ctx):
    """4,352 voters x 4,352 keys x 8 heads: 17 query blocks per head; two heads against the oracle."""
    n_p, n_m, H, Hkv, d = 4096, 256, 8, 8, 128
    T = n_p + n_m
    q, k = _sequence(T, H, Hkv, d, torch.bfloat16, 7)
    got = _vote(ctx, q, k, np.arange(T), n_p)
    for h in (0, 5):
        ref = O.vote_scores(q[:, h:h + 1], k[:, h:h + 1], np.arange(T), n_p)
        assert_scores_close(got[h:h + 1], ref, what=f"all-voting head {h}")
