"""The five calls of a layer allocate nothing and never synchronise: they can be captured into a CUDA graph and replayed
(what a serving loop does).  The replay must reproduce the plain calls bit for bit, also after the inputs have changed."""
import pytest
import torch

from paper_2510_09309_b200 import synth
from pipeline import LayerRun, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def _calls(run, xd, ld):
    run.score(xd); run.budget(); run.select(); run.compact(xd); run.attend(ld)


@pytest.mark.parametrize("config,dtype", [(2, "bf16"), (4, "bf16"), (1, "f32")])
def test_graph_replay_matches_plain_calls(ctx, config, dtype):
    wl = synth.scaled(synth.config(config), "graph", dtype=dtype, prompt_lens=(1500,) if config != 4 else (2100,))
    x0 = synth.layer_inputs(wl, 0, "cpu"); x1 = synth.layer_inputs(wl, 1, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
    xd = {k: to_dev(v) for k, v in x0.items() if torch.is_tensor(v)}
    x1d = {k: to_dev(v) for k, v in x1.items() if torch.is_tensor(v)}
    ld = {k: to_dev(v) for k, v in live.items()}
    run = LayerRun(ctx, wl)

    def snapshot():
        torch.cuda.synchronize()
        n = int(run.offsets[-1].item())
        return [t.clone() for t in (run.scores, run.mass_p, run.mass_m, run.budgets, run.offsets, run.kept[:n], run.kc[:n],
                                    run.vc[:n], run.out, run.lse)]

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        _calls(run, xd, ld)                                   # plain calls, layer 0
        plain0 = snapshot()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            _calls(run, xd, ld)
        for t in (run.scores, run.out, run.kc, run.vc):
            t.zero_()
        graph.replay()
        replay0 = snapshot()
        for k in xd:                                          # new contents behind the same pointers: layer 1
            xd[k].copy_(x1d[k])
        graph.replay()
        replay1 = snapshot()
        _calls(run, xd, ld)
        plain1 = snapshot()
    torch.cuda.synchronize()
    for a, b in zip(plain0, replay0):
        assert torch.equal(a, b)
    for a, b in zip(plain1, replay1):
        assert torch.equal(a, b)
    assert not torch.equal(plain0[0], plain1[0])              # the two layers do differ
    assert ctx.maskkv_check_status() == 0


def test_per_step_calls_replay_from_a_graph(ctx):
    """The calls of a later denoising step - refresh test, attention for the refreshed rows, mask-only projection - in
    one graph: the replay reproduces the plain calls, also after the inputs behind the pointers have changed."""
    from paper_2510_09309_b200 import binding as B
    wl = synth.scaled(synth.config(2), "graph_step", prompt_lens=(1500,))
    x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu"); live1 = synth.live_inputs(wl, 0, 1, "cpu")
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
    ld = {k: to_dev(v) for k, v in live.items()}
    l1d = {k: to_dev(v) for k, v in live1.items()}
    run = LayerRun(ctx, wl)
    _calls(run, xd, ld)
    M, H, d = wl.n_mask, wl.n_q_heads, wl.head_dim
    rows_cu = [0, M // 2]
    q_rows = ld["q_live"][:M // 2]                            # a fixed set of rows has queries this step
    out_rows = torch.zeros_like(q_rows)
    px = synth.project_inputs(M + 64, 256, 3000, M, "cuda", seed=2)
    logits = torch.zeros((M, 3000), dtype=torch.float32, device="cuda")
    p_ws = torch.empty(B.maskkv_mask_project_workspace_bytes(M, 256), dtype=torch.uint8, device="cuda")
    v_prev = to_dev(live1["v_live"].reshape(M, -1))
    idx = torch.zeros(M, dtype=torch.int32, device="cuda"); cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    rows_cu_dev = torch.tensor(rows_cu, dtype=torch.int32, device="cuda")

    def step():
        ctx.maskkv_refresh_set(ld["v_live"].reshape(M, -1), v_prev, 0.05, idx, cnt)
        ctx.maskkv_attend_rows(run.p, q_rows, rows_cu, rows_cu_dev, ld["k_live"], ld["v_live"], run.kc, run.vc, run.offsets,
                               run.kc.shape[0], out_rows)
        ctx.maskkv_mask_project(px["hidden"], px["w_vocab"], logits, px["positions"], p_ws)

    def snapshot():
        torch.cuda.synchronize()
        return [t.clone() for t in (idx[:int(cnt.item())], cnt, out_rows, logits)]

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()
        plain0 = snapshot()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
        out_rows.zero_(); logits.zero_()
        graph.replay()
        replay0 = snapshot()
        for k in ld:
            ld[k].copy_(l1d[k])                               # q_rows is a view of ld["q_live"]: it changes too
        px["hidden"].copy_(px["hidden"].flip(0))
        graph.replay()
        replay1 = snapshot()
        step()
        plain1 = snapshot()
    torch.cuda.synchronize()
    for a, b in zip(plain0, replay0):
        assert torch.equal(a, b)
    for a, b in zip(plain1, replay1):
        assert torch.equal(a, b)
    assert not torch.equal(plain0[2], plain1[2]) and not torch.equal(plain0[3], plain1[3])
    assert ctx.maskkv_check_status() == 0
