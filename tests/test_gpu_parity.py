"""GPU parity: every call of the C ABI against the fp64 oracle on the same seeded inputs.

Stage tests feed each CUDA stage the oracle's output of the stage before (rounded to the device
dtype), so integer work is compared bit-exactly; the chain test runs the CUDA stages on their own
outputs and applies the tolerance band at the cut."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import (ATTEND_ATOL, LayerRun, assert_kept_within_band, assert_scores_close, oracle_layer, to_dev)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    assert c.maskkv_check_status() & B.MASKKV_FLAG_TIMEOUT == 0
    c.close()


def workloads():
    c1, c2, c3, c4, c5 = (synth.config(i) for i in range(1, 6))
    return [
        c1,                                                                            # tiny fp32, full size
        synth.scaled(c1, "tiny_fp32_d128_ragged", head_dim=128, prompt_lens=(300, 77), n_mask=40, mean_budget=24),
        synth.scaled(c2, "llada_layer_1k", prompt_lens=(1100,), n_mask=200, n_q_heads=8, n_kv_heads=8, mean_budget=96),
        c2,                                                                            # full size: the oracle needs a few seconds
        synth.scaled(c3, "llada_stack_3k", prompt_lens=(3000,), n_mask=256, n_q_heads=8, n_kv_heads=8, n_layers=4,
                     mean_budget=64),
        synth.scaled(c4, "dream_gqa_2k", prompt_lens=(2050,), n_mask=150, n_q_heads=14, n_kv_heads=2, mean_budget=128),
        synth.scaled(c5, "ragged_4req", prompt_lens=(1024, 333, 2047, 17), n_mask=96, n_q_heads=4, n_kv_heads=4,
                     mean_budget=64, n_layers=2),
        synth.scaled(c5, "ragged_d64_gqa", prompt_lens=(129, 640), n_mask=33, n_q_heads=6, n_kv_heads=3, head_dim=64,
                     mean_budget=40, n_layers=2, head_recipe="none"),
    ]


def layer_k(wl, layer):
    if wl.layer_profile == "uniform":
        return wl.mean_budget
    return O.layer_budgets(wl.total_budget(), wl.beta, wl.layer_importance())[layer]


@pytest.fixture(scope="module", params=workloads(), ids=lambda w: w.name)
def case(request, ctx):
    wl = request.param
    layer = wl.n_layers - 1                     # the last layer is a boundary layer when the profile is bimodal
    x = synth.layer_inputs(wl, layer, "cpu")
    live = synth.live_inputs(wl, layer, 0, "cpu")
    k_l = layer_k(wl, layer)
    ref = oracle_layer(wl, x, live, k_l, wl.alpha)
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
    ld = {k: to_dev(v) for k, v in live.items()}
    return dict(wl=wl, x=x, live=live, xd=xd, ld=ld, ref=ref, k_l=k_l, run=LayerRun(ctx, wl, k_l=k_l))


def test_score(case):
    run, ref, wl = case["run"], case["ref"], case["wl"]
    run.score(case["xd"])
    torch.cuda.synchronize()
    assert_scores_close(run.scores.cpu().numpy(), ref["scores"])
    assert_scores_close(run.mass_p.cpu().numpy(), ref["mass_p"], what="mass_p")
    assert_scores_close(run.mass_m.cpu().numpy(), ref["mass_m"], what="mass_m")
    # invariant that holds at any size: the two masses add up to M * g per request
    tot = (run.mass_p + run.mass_m).cpu().numpy()
    np.testing.assert_allclose(tot, wl.n_mask * wl.group, rtol=1e-4)
    # determinism: a second run gives the same bits
    first = run.scores.clone(), run.mass_p.clone(), run.mass_m.clone()
    run.score(case["xd"])
    torch.cuda.synchronize()
    assert torch.equal(first[0], run.scores) and torch.equal(first[1], run.mass_p) and torch.equal(first[2], run.mass_m)


def test_score_row_weights(case):
    run, wl = case["run"], case["wl"]
    if wl.prompt_cu()[-1] > 4000:
        pytest.skip("covered on the smaller cases")
    g = torch.Generator().manual_seed(11)
    w = torch.rand(wl.n_requests * wl.n_mask, generator=g) * 2
    w[: wl.n_mask // 2] = 0.0        # position-aware voting: the front half of the first request's mask rows does not vote
    sc, mp, mm = O.score(case["x"]["q_mask"], case["x"]["k_prompt"], case["x"]["k_mask"], wl.prompt_cu(), wl.live_cu(),
                         row_weights=w.numpy())
    run.score(case["xd"], row_weights=to_dev(w))
    torch.cuda.synchronize()
    assert_scores_close(run.scores.cpu().numpy(), sc)
    assert_scores_close(run.mass_m.cpu().numpy(), mm, what="mass_m")
    # voting with the back half only = scoring with 0/1 weights (the mask-position ablation of the paper)
    if wl.n_requests == 1:
        w01 = torch.zeros(wl.n_mask); w01[wl.n_mask // 2:] = 1.0
        sc2, _, _ = O.score(case["x"]["q_mask"], case["x"]["k_prompt"], case["x"]["k_mask"], wl.prompt_cu(), wl.live_cu(),
                            row_weights=w01.numpy())
        run.score(case["xd"], row_weights=to_dev(w01))
        torch.cuda.synchronize()
        assert_scores_close(run.scores.cpu().numpy(), sc2)


def test_budget_bit_exact(case):
    run, ref, wl = case["run"], case["ref"], case["wl"]
    run.budget(mass_p=to_dev(ref["mass_p32"]), mass_m=to_dev(ref["mass_m32"]))
    torch.cuda.synchronize()
    assert np.array_equal(run.budgets.cpu().numpy(), ref["budgets"])
    assert np.array_equal(run.offsets.cpu().numpy(), ref["offsets"])
    tot = ref["budgets"].sum(1)
    cap = np.minimum(wl.n_kv_heads * case["k_l"], wl.n_kv_heads * np.array(wl.prompt_lens))
    assert (tot <= cap).all()


def test_select_bit_exact(case):
    run, ref = case["run"], case["ref"]
    run.kept.fill_(-1)
    run.select(scores=to_dev(ref["scores32"]), budgets=to_dev(ref["budgets"]), offsets=to_dev(ref["offsets"]))
    torch.cuda.synchronize()
    total = int(ref["offsets"][-1])
    assert np.array_equal(run.kept[:total].cpu().numpy(), ref["kept"])
    assert (run.kept[total:] == -1).all()            # nothing written past the segments


def test_compact_bit_exact(case):
    run, ref = case["run"], case["ref"]
    run.kc.zero_(); run.vc.zero_()
    run.compact(case["xd"], kept=to_dev(np.concatenate([ref["kept"], np.zeros(1, np.int32)])), offsets=to_dev(ref["offsets"]))
    torch.cuda.synchronize()
    total = int(ref["offsets"][-1])
    view = torch.int32 if case["wl"].dtype == "f32" else torch.int16
    assert torch.equal(run.kc[:total].cpu().view(view), ref["kc"].view(view))
    assert torch.equal(run.vc[:total].cpu().view(view), ref["vc"].view(view))
    assert (run.kc[total:] == 0).all() and (run.vc[total:] == 0).all()


def test_attend(case):
    run, ref, wl = case["run"], case["ref"], case["wl"]
    total = int(ref["offsets"][-1])
    kc = torch.zeros_like(run.kc); vc = torch.zeros_like(run.vc)
    kc[:total] = ref["kc"].to(kc.device); vc[:total] = ref["vc"].to(vc.device)
    run.attend(case["ld"], kc=kc, vc=vc, offsets=to_dev(ref["offsets"]))
    torch.cuda.synchronize()
    err = np.abs(run.out.float().cpu().numpy().astype(np.float64) - ref["out"]).max()
    assert err <= ATTEND_ATOL[wl.dtype], f"attend max-abs error {err:.3e}"
    lse_err = np.abs(run.lse.cpu().numpy() - ref["lse"]).max()
    assert lse_err <= 1e-3, f"lse error {lse_err:.3e}"


def test_chain_on_device(case):
    """score -> budget -> select -> compact -> attend on the CUDA path's own intermediates."""
    run, ref, wl = case["run"], case["ref"], case["wl"]
    run.score(case["xd"]); run.budget(); run.select(); run.compact(case["xd"]); run.attend(case["ld"])
    torch.cuda.synchronize()
    bud = run.budgets.cpu().numpy(); off = run.offsets.cpu().numpy(); kept = run.kept.cpu().numpy()
    # budgets can only differ from the oracle's where the pre-floor value sits on an integer
    assert np.abs(bud - ref["budgets"]).max() <= 1
    assert (np.diff(off) == bud.reshape(-1)).all()
    pcu = wl.prompt_cu()
    same_budgets = np.array_equal(bud, ref["budgets"])
    for r in range(wl.n_requests):
        for h in range(wl.n_kv_heads):
            s = r * wl.n_kv_heads + h
            assert_kept_within_band(kept[off[s]:off[s + 1]], ref["scores"][h, pcu[r]:pcu[r + 1]], int(bud[r, h]))
    # compacted rows are byte copies of the rows the device selected
    view = torch.int32 if wl.dtype == "f32" else torch.int16
    kc_ref, vc_ref = O.compact(case["x"]["k_prompt"], case["x"]["v_prompt"], kept, off, pcu)
    total = int(off[-1])
    assert torch.equal(run.kc[:total].cpu().view(view), kc_ref.view(view))
    assert torch.equal(run.vc[:total].cpu().view(view), vc_ref.view(view))
    # attention over the device's own cache, checked against the oracle on that same cache
    out_ref, _ = O.attend(case["live"]["q_live"], case["live"]["k_live"], case["live"]["v_live"], kc_ref, vc_ref, off,
                          wl.live_cu(), wl.n_kv_heads)
    err = np.abs(run.out.float().cpu().numpy().astype(np.float64) - out_ref).max()
    assert err <= ATTEND_ATOL[wl.dtype]
    if same_budgets and np.array_equal(kept[:total], ref["kept"]):
        err2 = np.abs(run.out.float().cpu().numpy().astype(np.float64) - ref["out"]).max()
        assert err2 <= ATTEND_ATOL[wl.dtype]


def test_bf16_runs_on_the_tensor_core_kernels(case, ctx):
    """bf16 scoring (two sweeps) and attention must be served by the tcgen05 kernels, fp32 by the FP32 pipes."""
    run = case["run"]
    before = ctx.maskkv_tensor_core_launch_count()
    run.score(case["xd"]); run.attend(case["ld"])
    torch.cuda.synchronize()
    assert ctx.maskkv_tensor_core_launch_count() - before == (3 if case["wl"].dtype == "bf16" else 0)


def test_full_budget_equals_full_attention(ctx):
    """k >= N for every head: attention over the compacted cache equals attention over the original K/V."""
    wl = synth.scaled(synth.config(2), "full_budget", prompt_lens=(200, 64), n_mask=48, n_q_heads=4, n_kv_heads=2,
                      mean_budget=256)
    x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}; ld = {k: to_dev(v) for k, v in live.items()}
    run = LayerRun(ctx, wl)
    run.score(xd); run.budget(alpha=1.0); run.select(); run.compact(xd); run.attend(ld)
    torch.cuda.synchronize()
    assert run.budgets.cpu().tolist() == [[200, 200], [64, 64]]
    pcu, lcu = wl.prompt_cu(), wl.live_cu()
    for r in range(2):
        for h in range(4):
            keys = torch.cat([x["k_prompt"][pcu[r]:pcu[r + 1], h // 2], live["k_live"][lcu[r]:lcu[r + 1], h // 2]]).double()
            vals = torch.cat([x["v_prompt"][pcu[r]:pcu[r + 1], h // 2], live["v_live"][lcu[r]:lcu[r + 1], h // 2]]).double()
            q = live["q_live"][lcu[r]:lcu[r + 1], h].double()
            ref = torch.softmax(q @ keys.T / wl.head_dim ** 0.5, -1) @ vals
            err = (run.out[lcu[r]:lcu[r + 1], h].double().cpu() - ref).abs().max().item()
            assert err <= ATTEND_ATOL["bf16"]
