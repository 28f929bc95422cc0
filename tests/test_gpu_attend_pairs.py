"""The attention kernel that takes two (query tile, query head) units per CTA (chosen for launches with many more units
than SMs; pinned here through bit 5 of MASKKV_KERNEL_CHOICE): two query tiles of one head, tiles of different query heads
of a group, an odd number of units per KV head (the last CTA runs one stream), empty and long cache segments, ragged
tails, and the partial-refresh call.  Outputs and log-sum-exps against the oracle on the device's own cache."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import ATTEND_ATOL, LayerRun, to_dev

pytestmark = pytest.mark.gpu

CASES = {
    "mha_two_tiles": dict(base=5, prompt_lens=(300, 1, 700), n_mask=200, n_q_heads=4, n_kv_heads=4, mean_budget=150),
    "gqa_odd_units": dict(base=4, prompt_lens=(515, 90), n_mask=100, n_q_heads=6, n_kv_heads=2, mean_budget=40),
    "gqa_seven": dict(base=4, prompt_lens=(1200,), n_mask=300, n_q_heads=14, n_kv_heads=2, mean_budget=260),
    "long_and_empty": dict(base=5, prompt_lens=(2100, 5), n_mask=129, n_q_heads=2, n_kv_heads=2, mean_budget=1000),
}


@pytest.mark.parametrize("name", list(CASES))
def test_two_units_per_cta_match_the_oracle(name, monkeypatch):
    from paper_2510_09309_b200 import binding as B
    cfg = dict(CASES[name])
    wl = synth.scaled(synth.config(cfg.pop("base")), "pairs_" + name, **cfg)
    x = synth.layer_inputs(wl, 0, "cpu")
    live = synth.live_inputs(wl, 0, 0, "cpu")
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
    ld = {k: to_dev(v) for k, v in live.items()}
    outs = {}
    for choice in ("32", "64"):                              # two units per CTA; one unit per CTA
        monkeypatch.setenv("MASKKV_KERNEL_CHOICE", choice)
        ctx = B.Context(0)
        try:
            run = LayerRun(ctx, wl)
            run.score(xd); run.budget(); run.select(); run.compact(xd)
            if name == "long_and_empty":                     # the second request keeps nothing: live keys only
                bud = run.budgets.clone(); bud[1] = 0
                off = torch.zeros_like(run.offsets); off[1:] = torch.cumsum(bud.reshape(-1), 0)
                run.budgets, run.offsets = bud, off.to(torch.int32)
                run.select(); run.compact(xd)
            run.attend(ld)
            torch.cuda.synchronize()
            assert ctx.maskkv_check_status() == 0
            off, kept = run.offsets.cpu().numpy(), run.kept.cpu().numpy()
            outs[choice] = (run.out.float().cpu().numpy(), run.lse.cpu().numpy(), off, kept)
        finally:
            ctx.close()
    out, lse, off, kept = outs["32"]
    kc, vc = O.compact(x["k_prompt"], x["v_prompt"], kept[:off[-1]], off, wl.prompt_cu())
    ref, ref_lse = O.attend(live["q_live"], live["k_live"], live["v_live"], kc, vc, off, wl.live_cu(), wl.n_kv_heads)
    assert np.abs(out - ref).max() <= ATTEND_ATOL[wl.dtype]
    assert np.abs(lse - ref_lse).max() <= 1e-3
    assert np.array_equal(off, outs["64"][2]) and np.array_equal(kept[:off[-1]], outs["64"][3][:off[-1]])
    assert np.abs(out - outs["64"][0]).max() <= ATTEND_ATOL[wl.dtype]


def test_partial_refresh_rows_with_two_units_per_cta(monkeypatch):
    from paper_2510_09309_b200 import binding as B
    monkeypatch.setenv("MASKKV_KERNEL_CHOICE", "32")
    ctx = B.Context(0)
    try:
        wl = synth.scaled(synth.config(4), "pairs_rows", prompt_lens=(700, 1300), n_mask=300, n_q_heads=8, n_kv_heads=2, mean_budget=64)
        x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
        xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
        ld = {k: to_dev(v) for k, v in live.items()}
        run = LayerRun(ctx, wl)
        run.score(xd); run.budget(); run.select(); run.compact(xd)
        rng = np.random.default_rng(7)
        rows = [np.sort(rng.choice(300, 131, replace=False)), np.sort(rng.choice(300, 1, replace=False))]
        rows_cu = [0, 131, 132]
        idx = np.concatenate([rows[0], 300 + rows[1]])
        q_rows = ld["q_live"][torch.from_numpy(idx).to(ctx.device)].contiguous()
        out = torch.zeros_like(q_rows)
        lse = torch.zeros((8, 132), dtype=torch.float32, device=ctx.device)
        ctx.maskkv_attend_rows(run.p, q_rows, rows_cu, to_dev(np.array(rows_cu, np.int32)), ld["k_live"], ld["v_live"], run.kc, run.vc,
                               run.offsets, run.capacity, out, lse)
        torch.cuda.synchronize()
        assert ctx.maskkv_check_status() == 0
        off, kept = run.offsets.cpu().numpy(), run.kept.cpu().numpy()
        kc, vc = O.compact(x["k_prompt"], x["v_prompt"], kept[:off[-1]], off, wl.prompt_cu())
        ref, ref_lse = O.attend(q_rows.cpu(), live["k_live"], live["v_live"], kc, vc, off, wl.live_cu(), wl.n_kv_heads, rows_cu=rows_cu)
        assert np.abs(out.float().cpu().numpy() - ref).max() <= ATTEND_ATOL[wl.dtype]
        assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 1e-3
    finally:
        ctx.close()
