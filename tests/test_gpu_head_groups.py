"""Scoring with the KV heads taken in groups (MASKKV_SCORE_HEAD_GROUPS, read when a context is created): both sweeps of a
group run back to back so that the second sweep finds the group's keys in L2.  The grouping changes which CTA sees
which tile, nothing else: scores and masses must match the oracle like the ungrouped call, for group counts that do and
do not divide the number of heads, on a ragged batch."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import assert_scores_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("groups", ["2", "3", "8", "64"])
def test_grouped_scoring_matches_the_oracle(groups, monkeypatch):
    from paper_2510_09309_b200 import binding as B
    monkeypatch.setenv("MASKKV_SCORE_HEAD_GROUPS", groups)
    ctx = B.Context(0)
    try:
        wl = synth.scaled(synth.config(5), "groups", prompt_lens=(1500, 1, 700, 2300), n_mask=200, n_q_heads=8, n_kv_heads=8,
                          mean_budget=64)
        x = synth.layer_inputs(wl, 3, "cpu")
        xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
        p = B.Problem(wl.torch_dtype, 8, 8, wl.head_dim, wl.prompt_cu(), wl.live_cu(), ctx.device)
        ws = torch.empty(max(ctx.maskkv_workspace_bytes(p), 256), dtype=torch.uint8, device=ctx.device)
        scores = torch.full((8, p.sumN), float("nan"), dtype=torch.float32, device=ctx.device)
        mp = torch.full((4, 8), float("nan"), dtype=torch.float32, device=ctx.device)
        mm = torch.full((4, 8), float("nan"), dtype=torch.float32, device=ctx.device)
        before = ctx.maskkv_launch_count()
        ctx.maskkv_score(p, xd["q_mask"], xd["k_prompt"], xd["k_mask"], scores, mp, mm, ws)
        torch.cuda.synchronize()
        n_groups = min(int(groups), 8)
        per = -(-8 // n_groups)
        assert ctx.maskkv_launch_count() - before == 2 * (-(-8 // per))       # two sweeps per group of heads
        ref, ref_p, ref_m = O.score(x["q_mask"], x["k_prompt"], x["k_mask"], wl.prompt_cu(), wl.live_cu())
        assert_scores_close(scores.cpu().numpy(), ref)
        assert_scores_close(mp.cpu().numpy(), ref_p, what="mass_p")
        assert_scores_close(mm.cpu().numpy(), ref_m, what="mass_m")
        assert ctx.maskkv_check_status() == 0
    finally:
        ctx.close()
