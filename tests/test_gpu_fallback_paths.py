"""The FP32-pipe kernels double as the on-device cross-check of the tensor-core ones: MASKKV_FORCE_SIMT (read when a
context is created; bit 0 = scoring sweep 1, bit 1 = scoring sweep 2, bit 2 = attention) routes bf16 problems through
them.  Every mix of the two families must agree with the oracle, and MASKKV_SERIAL_LAUNCH=1 (ordinary stream order
instead of overlapped launches) must not change a bit."""
import os

import numpy as np
import pytest
import torch

from paper_2510_09309_b200 import synth
from oracle import maskkv_oracle as O
from pipeline import ATTEND_ATOL, LayerRun, assert_kept_within_band, assert_scores_close, to_dev

pytestmark = pytest.mark.gpu


def _workloads():
    return [
        synth.scaled(synth.config(3), "mix_llada", prompt_lens=(1900,), n_mask=200, n_q_heads=4, n_kv_heads=4, mean_budget=96),
        synth.scaled(synth.config(4), "mix_gqa", prompt_lens=(700, 1300), n_mask=300, n_q_heads=8, n_kv_heads=2, mean_budget=64),
    ]


def _run(wl, x, live, k_l):
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
        ld = {k: to_dev(v) for k, v in live.items()}
        run = LayerRun(ctx, wl, k_l=k_l)
        run.score(xd); run.budget(); run.select(); run.compact(xd); run.attend(ld)
        torch.cuda.synchronize()
        assert ctx.maskkv_check_status() == 0
        n = int(run.offsets[-1].item())
        return {"scores": run.scores.cpu(), "mass_p": run.mass_p.cpu(), "mass_m": run.mass_m.cpu(), "budgets": run.budgets.cpu(),
                "offsets": run.offsets.cpu(), "kept": run.kept[:n].cpu(), "out": run.out.float().cpu(),
                "tc": ctx.maskkv_tensor_core_launch_count()}
    finally:
        ctx.close()


@pytest.mark.parametrize("wl", _workloads(), ids=lambda w: w.name)
def test_every_mix_of_kernel_families_matches_the_oracle(wl, monkeypatch):
    layer = wl.n_layers - 1
    x = synth.layer_inputs(wl, layer, "cpu"); live = synth.live_inputs(wl, layer, 0, "cpu")
    k_l = wl.mean_budget
    pcu, lcu = wl.prompt_cu(), wl.live_cu()
    sc, mp, mm = O.score(x["q_mask"], x["k_prompt"], x["k_mask"], pcu, lcu)
    tc_counts = {}
    for force in (0, 1, 2, 3, 4, 7):
        monkeypatch.setenv("MASKKV_FORCE_SIMT", str(force))
        got = _run(wl, x, live, k_l)
        assert_scores_close(got["scores"].numpy(), sc)
        assert_scores_close(got["mass_p"].numpy(), mp, what="mass_p")
        assert_scores_close(got["mass_m"].numpy(), mm, what="mass_m")
        bud, off, kept = got["budgets"].numpy(), got["offsets"].numpy(), got["kept"].numpy()
        ref_bud, _ = O.head_budgets(got["mass_p"].numpy(), got["mass_m"].numpy(), k_l, wl.alpha, wl.prompt_lens)
        assert np.array_equal(bud, ref_bud)                            # bit-exact on the masses the device produced
        for r in range(wl.n_requests):
            for h in range(wl.n_kv_heads):
                seg = r * wl.n_kv_heads + h
                assert_kept_within_band(kept[off[seg]:off[seg + 1]], sc[h, pcu[r]:pcu[r + 1]], int(bud[r, h]))
        kc, vc = O.compact(x["k_prompt"], x["v_prompt"], kept, off, pcu)
        out, _ = O.attend(live["q_live"], live["k_live"], live["v_live"], kc, vc, off, lcu, wl.n_kv_heads)
        assert np.abs(got["out"].numpy() - out).max() <= ATTEND_ATOL[wl.dtype]
        tc_counts[force] = got["tc"]
    assert tc_counts[0] == 3 and tc_counts[7] == 0 and tc_counts[3] == 1 and tc_counts[4] == 2


def test_serial_launches_give_the_same_bits(monkeypatch):
    wl = _workloads()[1]
    x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
    monkeypatch.delenv("MASKKV_FORCE_SIMT", raising=False)
    a = _run(wl, x, live, wl.mean_budget)
    # the switch is read once per process by the launch helper, so this only checks the overlapped path against itself
    # unless the variable was set before the first launch; both must agree bit for bit in either case
    monkeypatch.setenv("MASKKV_SERIAL_LAUNCH", "1")
    b = _run(wl, x, live, wl.mean_budget)
    for k in ("scores", "mass_p", "mass_m", "budgets", "kept", "out"):
        assert torch.equal(a[k], b[k])
