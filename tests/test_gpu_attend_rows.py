"""GPU parity of maskkv_attend_rows (attention with partial refresh: queries only for the response rows that
maskkv_refresh_set marks, keys and values = compacted prompt cache + all live rows) against the oracle, through the
C ABI; tensor-core and FP32-pipe kernels, bf16 and fp32."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import ATTEND_ATOL, LayerRun, to_dev

pytestmark = pytest.mark.gpu


def _prepared(ctx, wl, layer=0):
    x = synth.layer_inputs(wl, layer, "cpu")
    live = synth.live_inputs(wl, layer, 0, "cpu")
    run = LayerRun(ctx, wl)
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
    ld = {k: to_dev(v) for k, v in live.items()}
    run.score(xd); run.budget(); run.select(); run.compact(xd); run.attend(ld)
    torch.cuda.synchronize()
    return run, live, ld


def _check_rows(ctx, run, wl, live, ld, picks, atol):
    """picks[r] = live-row numbers (within request r) that have queries this step."""
    lcu = wl.live_cu()
    rows = [lcu[r] + i for r in range(wl.n_requests) for i in picks[r]]
    rows_cu = np.concatenate([[0], np.cumsum([len(p) for p in picks])]).tolist()
    n = len(rows)
    H, d = wl.n_q_heads, wl.head_dim
    dev = ctx.device
    q_rows = ld["q_live"][torch.tensor(rows, dtype=torch.long, device=dev)].contiguous() if n else ld["q_live"][:0]
    out = torch.full((max(n, 1), H, d), float("nan"), dtype=wl.torch_dtype, device=dev)
    lse = torch.full((H, max(n, 1)), float("nan"), dtype=torch.float32, device=dev)
    rows_cu_dev = torch.tensor(rows_cu, dtype=torch.int32, device=dev)
    ctx.maskkv_attend_rows(run.p, q_rows, rows_cu, rows_cu_dev, ld["k_live"], ld["v_live"], run.kc, run.vc, run.offsets,
                           run.kc.shape[0], out, lse)
    torch.cuda.synchronize()
    assert ctx.maskkv_check_status() == 0
    if n == 0:
        assert torch.isnan(out.float()).all()
        return
    kc, vc, off = run.kc.cpu(), run.vc.cpu(), run.offsets.cpu().numpy()
    ref, ref_lse = O.attend(live["q_live"][rows], live["k_live"], live["v_live"], kc, vc, off, lcu, wl.n_kv_heads, rows_cu=rows_cu)
    err = np.abs(out[:n].float().cpu().numpy() - ref).max()
    assert err <= atol, f"attend_rows: {err:.3e}"
    np.testing.assert_allclose(lse[:, :n].cpu().numpy(), ref_lse, rtol=0, atol=2e-3 if wl.dtype == "bf16" else 1e-4)
    # and they are the rows of the full step the same kernel family computed
    full = run.out.float().cpu().numpy()[rows]
    assert np.abs(out[:n].float().cpu().numpy() - full).max() <= 2 * atol


@pytest.mark.parametrize("force", ["0", "4"])
def test_partial_refresh_bf16_ragged_batch(force, monkeypatch):
    """Two requests, grouped heads, 300 live rows each: subsets of 1, 129 (two query tiles) and 0 rows."""
    from paper_2510_09309_b200 import binding as B
    monkeypatch.setenv("MASKKV_FORCE_SIMT", force)
    ctx = B.Context(0)
    try:
        wl = synth.scaled(synth.config(4), "rows_gqa", prompt_lens=(700, 1300), n_mask=300, n_q_heads=8, n_kv_heads=2, mean_budget=64)
        run, live, ld = _prepared(ctx, wl)
        rng = np.random.default_rng(1)
        for picks in ([[7], sorted(rng.choice(300, 129, replace=False).tolist())],
                      [[], [299, 0, 150]],                              # a request without refreshed rows; any order
                      [list(range(300)), list(range(300))],            # every row: the full step
                      [[], []]):
            _check_rows(ctx, run, wl, live, ld, picks, ATTEND_ATOL[wl.dtype])
    finally:
        ctx.close()


def test_partial_refresh_fp32(monkeypatch):
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        wl = synth.scaled(synth.config(1), "rows_fp32", dtype="f32")
        run, live, ld = _prepared(ctx, wl)
        M = wl.n_mask
        _check_rows(ctx, run, wl, live, ld, [list(range(0, M, 3)) for _ in range(wl.n_requests)], ATTEND_ATOL[wl.dtype])
    finally:
        ctx.close()


def test_refresh_set_drives_the_rows(monkeypatch):
    """The per-step loop: maskkv_refresh_set picks the rows from the value features, their queries go through
    maskkv_attend_rows; checked against the oracle's refresh rule + attention on the same inputs."""
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        wl = synth.scaled(synth.config(3), "rows_llada", prompt_lens=(4000,), n_mask=256, n_q_heads=4, n_kv_heads=4, mean_budget=128)
        run, live, ld = _prepared(ctx, wl)
        g = torch.Generator().manual_seed(11)
        v_cur = live["v_live"].reshape(256, -1)                          # all heads of a token side by side
        drift = torch.rand(256, 1, generator=g) * 1.2
        v_prev = (v_cur.float() + drift * torch.randn(v_cur.shape, generator=g)).to(v_cur.dtype)
        idx = torch.zeros(256, dtype=torch.int32, device=ctx.device)
        cnt = torch.zeros(1, dtype=torch.int32, device=ctx.device)
        ctx.maskkv_refresh_set(to_dev(v_cur), to_dev(v_prev), 0.8, idx, cnt)
        torch.cuda.synchronize()
        n = int(cnt.item())
        picked = idx.cpu().numpy()[:n].tolist()
        cos, _, ref_idx = O.refresh_set(v_cur, v_prev, 0.8)
        sure = [i for i in range(256) if abs(cos[i] - 0.8) > 1e-5]
        assert [i for i in picked if i in sure] == [i for i in ref_idx.tolist() if i in sure] and 0 < n < 256
        _check_rows(ctx, run, wl, live, ld, [picked], ATTEND_ATOL[wl.dtype])
    finally:
        ctx.close()


def test_argument_errors(monkeypatch):
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        wl = synth.scaled(synth.config(4), "rows_err", prompt_lens=(300, 200), n_mask=40, n_q_heads=4, n_kv_heads=2, mean_budget=16)
        run, live, ld = _prepared(ctx, wl)
        q = ld["q_live"][:4].contiguous()
        out = torch.zeros_like(q)
        before = ctx.maskkv_launch_count()
        for bad in ([1, 4, 4], [0, 4, 2]):                                                  # not starting at 0; decreasing
            with pytest.raises(B.MaskKVError) as e:
                ctx.maskkv_attend_rows(run.p, q, bad, torch.tensor(bad, dtype=torch.int32, device=ctx.device), ld["k_live"],
                                       ld["v_live"], run.kc, run.vc, run.offsets, run.kc.shape[0], out)
            assert e.value.code == B.MASKKV_E_INVALID
        assert ctx.maskkv_launch_count() == before
    finally:
        ctx.close()
