"""GPU parity at the full sizes of the five workloads, in the launch configuration bench.py times.

Inputs are generated on the device (seeded), the whole path runs on the device, and the oracle
recomputes sampled (request, head) units one by one from the same bytes copied to the host:
scores and masses of the sampled heads, their kept sets (band rule at the cut), the compacted rows
(byte-exact against the device's own kept indices) and the attention rows of the sampled heads.
Properties that hold at any size are checked on everything: mass identity, budget sums, ascending
unique in-range indices, status flags."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import ATTEND_ATOL, LayerRun, assert_kept_within_band, assert_scores_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def _run_and_check(ctx, wl, layer, k_l, alpha, sample, attend_steps=1, x=None):
    """sample: list of (request, kv_head); x: the layer's inputs when the caller already holds them."""
    if x is None:
        x = synth.layer_inputs(wl, layer, "cuda")
    run = LayerRun(ctx, wl, k_l=k_l)
    run.score(x)
    run.budget(alpha=alpha)
    run.select()
    run.compact(x)
    lives = [synth.live_inputs(wl, layer, st, "cuda") for st in range(attend_steps)]
    outs = []
    for live in lives:
        run.attend(live)
        outs.append(run.out.clone())
    torch.cuda.synchronize()
    assert ctx.maskkv_check_status() == 0

    R, Hkv, H, g, M = wl.n_requests, wl.n_kv_heads, wl.n_q_heads, wl.group, wl.n_mask
    pcu, lcu = wl.prompt_cu(), wl.live_cu()
    mp, mm = run.mass_p.cpu().numpy(), run.mass_m.cpu().numpy()
    bud, off, kept = run.budgets.cpu().numpy(), run.offsets.cpu().numpy(), run.kept.cpu().numpy()
    # properties over the whole problem
    np.testing.assert_allclose(mp + mm, M * g, rtol=2e-4)
    assert (np.diff(off) == bud.reshape(-1)).all()
    lens = np.array(wl.prompt_lens)[:, None]
    assert (bud >= 0).all() and (bud <= lens).all()
    unclamped = (bud < lens).all(axis=1)
    tot = bud.sum(1)
    assert (tot[unclamped] <= Hkv * k_l).all() and (tot[unclamped] > Hkv * k_l - Hkv).all()
    for r in range(R):
        for h in range(Hkv):
            s = r * Hkv + h
            seg = kept[off[s]:off[s + 1]]
            assert (np.diff(seg) > 0).all() and (seg.size == 0 or (seg[0] >= 0 and seg[-1] < wl.prompt_lens[r]))

    # sampled units against the oracle
    for (r, hk) in sample:
        qs = x["q_mask"][lcu[r]:lcu[r + 1], hk * g:(hk + 1) * g].cpu()
        kp = x["k_prompt"][pcu[r]:pcu[r + 1], hk:hk + 1].cpu()
        vp = x["v_prompt"][pcu[r]:pcu[r + 1], hk:hk + 1].cpu()
        km = x["k_mask"][lcu[r]:lcu[r + 1], hk:hk + 1].cpu()
        n = wl.prompt_lens[r]
        sc, smp, smm = O.score(qs, kp, km, [0, n], [0, M])
        got = run.scores[hk, pcu[r]:pcu[r + 1]].cpu().numpy()
        assert_scores_close(got, sc[0], what=f"scores r{r} h{hk}")
        assert_scores_close(mp[r, hk:hk + 1], smp[0], what="mass_p")
        assert_scores_close(mm[r, hk:hk + 1], smm[0], what="mass_m")
        s = r * Hkv + hk
        k = int(bud[r, hk])
        seg = kept[off[s]:off[s + 1]]
        assert_kept_within_band(seg, sc[0], k)
        # compacted rows are byte copies of the rows the device selected
        view = torch.int16
        kc_ref = kp[torch.from_numpy(seg.astype(np.int64)), 0]
        vc_ref = vp[torch.from_numpy(seg.astype(np.int64)), 0]
        assert torch.equal(run.kc[off[s]:off[s + 1]].cpu().view(view), kc_ref.view(view))
        assert torch.equal(run.vc[off[s]:off[s + 1]].cpu().view(view), vc_ref.view(view))
        # attention of the sampled head group over the device's own cache
        for live, out in zip(lives, outs):
            ql = live["q_live"][lcu[r]:lcu[r + 1], hk * g:(hk + 1) * g].cpu()
            kl = live["k_live"][lcu[r]:lcu[r + 1], hk:hk + 1].cpu()
            vl = live["v_live"][lcu[r]:lcu[r + 1], hk:hk + 1].cpu()
            ref, _ = O.attend(ql, kl, vl, kc_ref, vc_ref, np.array([0, k], np.int32), [0, M], 1)
            err = np.abs(out[lcu[r]:lcu[r + 1], hk * g:(hk + 1) * g].float().cpu().numpy() - ref).max()
            assert err <= ATTEND_ATOL[wl.dtype], f"attend r{r} h{hk}: {err:.3e}"
    return run


def test_config3_llada_32k_layers(ctx):
    """configs[2]: N=32768, M=256, 32 heads, adaptive budgets.  Layers 0 and 31 (boundary group, 512 per head on
    average), 1, 15 and 30 (middle group, 238); on each one information head (even) and one structure head (odd)
    against the oracle, everything else through the properties."""
    from paper_2510_09309_b200 import binding as B
    wl = synth.config(3)
    k_layers = B.maskkv_layer_budgets(wl.total_budget(), wl.beta, wl.layer_importance())
    assert k_layers == O.layer_budgets(wl.total_budget(), wl.beta, wl.layer_importance())
    assert k_layers[0] == 512 and k_layers[1] == 238 and k_layers[31] == 512 and k_layers[15] == 238
    samples = {0: [(0, 0), (0, 31)], 1: [(0, 5), (0, 16)], 15: [(0, 14), (0, 9)], 30: [(0, 22), (0, 27)],
               31: [(0, 30), (0, 1)]}
    for layer, sample in samples.items():
        run = _run_and_check(ctx, wl, layer, k_layers[layer], wl.alpha, sample)
        bud = run.budgets.cpu().numpy()[0]
        assert bud[0::2].mean() > 2 * bud[1::2].mean()       # information heads get the larger share
        del run
        torch.cuda.empty_cache()


def test_config4_dream_gqa_16k(ctx):
    """configs[3]: 28 query heads on 4 KV heads, N=16384, M=512, budgets 128 and 512 per KV head."""
    wl = synth.config(4)
    for k in (128, 512):
        _run_and_check(ctx, wl, 3, k, 1.0, [(0, 1)] if k == 128 else [(0, 3)])


def test_config5_ragged_serving(ctx):
    """configs[4]: 8 requests with prompts from 1024 to 32768 tokens; the whole budget sweep B = 64 ... 1024 (the
    clamp at B = 1024 included), each followed by 16 consecutive attention steps with fresh live tensors.  Sampled
    against the oracle: per budget two (request, head) units, chosen so that over the sweep every request and both
    kinds of head occur; the last layer (boundary group) for the sweep, the first and a middle layer at B = 256."""
    from paper_2510_09309_b200 import binding as B
    wl = synth.config(5)
    sweep = ((64, [(3, 7), (0, 12)]), (128, [(1, 0), (7, 21)]), (256, [(2, 9), (5, 4)]), (512, [(4, 18), (6, 3)]),
             (1024, [(0, 2), (6, 30)]))
    x = synth.layer_inputs(wl, 31, "cuda")
    for budget, sample in sweep:
        w2 = synth.scaled(wl, f"ragged_B{budget}", mean_budget=budget)
        k_layers = B.maskkv_layer_budgets(w2.total_budget(), w2.beta, w2.layer_importance())
        assert k_layers == O.layer_budgets(w2.total_budget(), w2.beta, w2.layer_importance())
        run = _run_and_check(ctx, w2, 31, k_layers[31], w2.alpha, sample, attend_steps=16, x=x)
        if budget == 1024:
            assert (run.budgets.cpu().numpy()[0] == 1024).any()   # the 1024-token prompt is clamped
        del run
        torch.cuda.empty_cache()
    del x
    torch.cuda.empty_cache()
    w2 = synth.scaled(wl, "ragged_B256", mean_budget=256)
    k_layers = B.maskkv_layer_budgets(w2.total_budget(), w2.beta, w2.layer_importance())
    for layer, sample in ((0, [(7, 6)]), (16, [(3, 25)])):
        _run_and_check(ctx, w2, layer, k_layers[layer], w2.alpha, sample, attend_steps=2)
        torch.cuda.empty_cache()
