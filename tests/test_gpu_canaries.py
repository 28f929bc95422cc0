"""Every output buffer and the workspace sit between guard regions filled with a byte pattern; after the calls the
guards must be untouched.  A cheap stand-in for a memory checker: a write before the first or past the last element of
any output shows up here.  Ragged, odd-sized workloads so that every tail path runs; both kernel families; the calls
beyond the five (all-keys scoring, attention for a row subset, refresh set, layer importance, mask-only projection)
included.  Also: two runs on the same inputs give the same bits (nothing depends on the order of float atomics)."""
import numpy as np
import pytest
import torch

from paper_2510_09309_b200 import synth
from pipeline import LayerRun, to_dev

pytestmark = pytest.mark.gpu
GUARD = 4096          # bytes on each side
PATTERN = 0xA5


class Guarded:
    """A tensor of the given shape/dtype carved out of a byte buffer with GUARD pattern bytes before and after."""

    def __init__(self, shape, dtype, device, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.n = n
        self.raw = torch.full((GUARD + n + GUARD,), PATTERN, dtype=torch.uint8, device=device)
        self.t = self.raw[GUARD:GUARD + n].view(dtype).view(*shape) if n else torch.empty(shape, dtype=dtype, device=device)
        if fill is not None and n:
            self.t.fill_(fill)

    def intact(self):
        return bool((self.raw[:GUARD] == PATTERN).all().item()) and bool((self.raw[GUARD + self.n:] == PATTERN).all().item())


def _guard_run(run, wl, dev):
    g = {}
    for name in ("scores", "mass_p", "mass_m", "budgets", "offsets", "kept", "kc", "vc", "out", "lse", "ws"):
        old = getattr(run, name)
        g[name] = Guarded(tuple(old.shape), old.dtype, dev)
        g[name].t.copy_(old)
        setattr(run, name, g[name].t)
    return g


@pytest.mark.parametrize("force", ["0", "7"])
@pytest.mark.parametrize("which", ["ragged_mha", "ragged_gqa", "tiny"])
def test_guards_around_every_output_of_the_layer_path(which, force, monkeypatch):
    from paper_2510_09309_b200 import binding as B
    monkeypatch.setenv("MASKKV_FORCE_SIMT", force)
    ctx = B.Context(0)
    try:
        wl = {
            "ragged_mha": synth.scaled(synth.config(5), "canary_mha", prompt_lens=(1, 129, 1031, 77), n_mask=67, n_q_heads=4,
                                       n_kv_heads=4, mean_budget=33),
            "ragged_gqa": synth.scaled(synth.config(4), "canary_gqa", prompt_lens=(515, 3), n_mask=259, n_q_heads=6, n_kv_heads=2,
                                       mean_budget=21),
            "tiny": synth.scaled(synth.config(1), "canary_tiny", prompt_lens=(5,), n_mask=3, mean_budget=2),
        }[which]
        dev = ctx.device
        x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
        xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
        ld = {k: to_dev(v) for k, v in live.items()}
        run = LayerRun(ctx, wl)
        guards = _guard_run(run, wl, dev)
        outs = []
        for rep in range(2):
            run.score(xd); run.budget(); run.select(); run.compact(xd); run.attend(ld)
            torch.cuda.synchronize()
            n = int(run.offsets[-1].item())
            outs.append([t.clone() for t in (run.scores, run.mass_p, run.mass_m, run.budgets, run.offsets, run.kept[:n], run.kc[:n],
                                             run.vc[:n], run.out, run.lse)])
        assert ctx.maskkv_check_status() == 0
        for name, gd in guards.items():
            assert gd.intact(), f"{name}: a guard region was written"
        for a, b in zip(*outs):
            assert torch.equal(a, b)                              # same inputs, same bits

        # the calls beyond the five, on the same workload
        Hkv, H, d, M = wl.n_kv_heads, wl.n_q_heads, wl.head_dim, wl.n_mask
        live_scores = Guarded((Hkv, run.p.sumM), torch.float32, dev)
        ctx.maskkv_score_all_keys(run.p, xd["q_mask"], xd["k_prompt"], xd["k_mask"], run.scores, live_scores.t, run.mass_p, run.mass_m, run.ws)
        n_rows = [max(0, M - 1 - r) for r in range(wl.n_requests)]
        rows_cu = np.concatenate([[0], np.cumsum(n_rows)]).tolist()
        lcu = wl.live_cu()
        rows = [lcu[r] + i for r in range(wl.n_requests) for i in range(n_rows[r])]
        q_rows = ld["q_live"][torch.tensor(rows, dtype=torch.long, device=dev)].contiguous()
        out_rows = Guarded((len(rows), H, d), wl.torch_dtype, dev)
        lse_rows = Guarded((H, len(rows)), torch.float32, dev)
        ctx.maskkv_attend_rows(run.p, q_rows, rows_cu, torch.tensor(rows_cu, dtype=torch.int32, device=dev), ld["k_live"], ld["v_live"],
                               run.kc, run.vc, run.offsets, run.kc.shape[0], out_rows.t, lse_rows.t)
        v = ld["v_live"].reshape(run.p.sumM, -1)
        idx = Guarded((run.p.sumM,), torch.int32, dev); cnt = Guarded((1,), torch.int32, dev); cos = Guarded((run.p.sumM,), torch.float32, dev)
        ctx.maskkv_refresh_set(v, v.flip(0).contiguous(), 0.3, idx.t, cnt.t, False, cos.t)
        imp = Guarded((1,), torch.float32, dev)
        ctx.maskkv_layer_importance(v, v.flip(0).contiguous(), imp.t)
        torch.cuda.synchronize()
        assert ctx.maskkv_check_status() == 0
        for name, gd in dict(guards, live_scores=live_scores, out_rows=out_rows, lse_rows=lse_rows, idx=idx, cnt=cnt, cos=cos, imp=imp).items():
            assert gd.intact(), f"{name}: a guard region was written"
    finally:
        ctx.close()


@pytest.mark.parametrize("n_mask,width,vocab,odt", [(70, 200, 777, torch.float32), (300, 136, 1001, torch.bfloat16),
                                                    (129, 64, 8, torch.float32)])
def test_guards_around_the_projection_outputs(n_mask, width, vocab, odt):
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        dev = ctx.device
        x = synth.project_inputs(n_mask + 9, width, vocab, n_mask, "cuda", seed=vocab)
        ld = (vocab + 7) // 8 * 8
        logits = Guarded((n_mask, ld), odt, dev, fill=0)
        ws = Guarded((B.maskkv_mask_project_workspace_bytes(n_mask, width) + 256,), torch.uint8, dev)
        ws_t = ws.t[(256 - ws.t.data_ptr() % 256) % 256:][:B.maskkv_mask_project_workspace_bytes(n_mask, width)]
        outs = []
        for rep in range(2):
            ctx.maskkv_mask_project(x["hidden"], x["w_vocab"], logits.t[:, :vocab], x["positions"], ws_t)
            torch.cuda.synchronize()
            outs.append(logits.t.clone())
        assert ctx.maskkv_check_status() == 0
        assert logits.intact() and ws.intact()
        assert not logits.t[:, vocab:].any()                      # the padding of every row stays as it was
        assert torch.equal(outs[0], outs[1])
    finally:
        ctx.close()
