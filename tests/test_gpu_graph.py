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
