"""The scoring kernels evaluate a share of their exponentials as a polynomial on the FMA pipes (relative error up to
2.7e-6 per weight) and the rest on the special-function unit.  What that does to Eq. 7 and to Eq. 16 is checked here on
twenty seeded problems at the full prompt length: scores against the fp64 oracle, and the kept set of the device's own
scores under the band rule at three budgets (the smallest structure-head budget, the mean, the largest information-head
budget of the 32k workload)."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import BAND_RTOL, assert_scores_close

pytestmark = pytest.mark.gpu

SEEDS = 20
BUDGETS = (119, 256, 768)


def test_scores_and_kept_sets_over_twenty_seeds_at_32k():
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        # two heads of the 32k workload (one information head, one structure head); the layer index is the seed
        wl = synth.scaled(synth.config(3), "seeds_32k", n_q_heads=2, n_kv_heads=2)
        N, M = wl.prompt_lens[0], wl.n_mask
        p = B.Problem(wl.torch_dtype, 2, 2, wl.head_dim, wl.prompt_cu(), wl.live_cu(), ctx.device)
        ws = torch.empty(max(ctx.maskkv_workspace_bytes(p), 256), dtype=torch.uint8, device=ctx.device)
        scores = torch.empty((2, N), dtype=torch.float32, device=ctx.device)
        mp = torch.empty((1, 2), dtype=torch.float32, device=ctx.device)
        mm = torch.empty((1, 2), dtype=torch.float32, device=ctx.device)
        worst, inside = 0.0, 0
        for seed in range(SEEDS):
            x = synth.layer_inputs(wl, seed, "cuda")
            ctx.maskkv_score(p, x["q_mask"], x["k_prompt"], x["k_mask"], scores, mp, mm, ws)
            torch.cuda.synchronize()
            ref, ref_p, ref_m = O.score(x["q_mask"].cpu(), x["k_prompt"].cpu(), x["k_mask"].cpu(), [0, N], [0, M])
            got = scores.cpu().numpy()
            worst = max(worst, assert_scores_close(got, ref, what=f"seed {seed}"))
            assert_scores_close(mp.cpu().numpy(), ref_p, what="mass_p")
            assert_scores_close(mm.cpu().numpy(), ref_m, what="mass_m")
            for h in range(2):
                order = np.argsort(-got[h].astype(np.float64), kind="stable")
                for k in BUDGETS:
                    kept = set(order[:k].tolist())
                    c = np.sort(ref[h])[::-1][k - 1]
                    must = np.nonzero(ref[h] > c * (1 + BAND_RTOL))[0]
                    must_not = np.nonzero(ref[h] < c * (1 - BAND_RTOL))[0]
                    assert all(int(j) in kept for j in must), f"seed {seed} head {h} k {k}: a token above the band was evicted"
                    assert not any(int(j) in kept for j in must_not), f"seed {seed} head {h} k {k}: a token below the band was kept"
                    inside += N - len(must) - len(must_not)
        assert ctx.maskkv_check_status() == 0
        print(f"worst relative score error {worst:.2e}; {inside} tokens inside the bands over {SEEDS * 2 * len(BUDGETS)} cuts")
    finally:
        ctx.close()
