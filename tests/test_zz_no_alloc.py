"""maskkv_score_noalloc: the scoring call for callers that may not allocate device memory (a serving
loop with a fixed, fully handed-out memory pool; a plugin that receives tensors but no allocator).
Its scratch is an 8 MiB array inside the library instead of a caller-provided workspace.

The check: called through the C ABI twice in a row on different inputs, it must give the same bits as
maskkv_score does with a caller-allocated workspace (the two run the same kernels on the same inputs),
it must agree with the CPU oracle within the scoring tolerance like every other scoring test, and it
must refuse problems whose scratch would not fit.  This file sorts last so that a run that stops at the first failure has already covered
everything else; it also passes when run on its own in a fresh process."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import assert_scores_close, to_dev

pytestmark = pytest.mark.gpu


def _score_both_ways(ctx, B, wl, layer):
    x = synth.layer_inputs(wl, layer, "cpu")
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
    p = B.Problem(wl.torch_dtype, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.prompt_cu(), wl.live_cu(), ctx.device)
    R, Hkv = wl.n_requests, wl.n_kv_heads
    outs = []
    for noalloc in (False, True):
        scores = torch.full((Hkv, p.sumN), float("nan"), dtype=torch.float32, device=ctx.device)
        mp = torch.full((R, Hkv), float("nan"), dtype=torch.float32, device=ctx.device)
        mm = torch.full((R, Hkv), float("nan"), dtype=torch.float32, device=ctx.device)
        if noalloc:
            ctx.maskkv_score_noalloc(p, xd["q_mask"], xd["k_prompt"], xd["k_mask"], scores, mp, mm)
        else:
            ws = torch.empty(ctx.maskkv_workspace_bytes(p), dtype=torch.uint8, device=ctx.device)
            ctx.maskkv_score(p, xd["q_mask"], xd["k_prompt"], xd["k_mask"], scores, mp, mm, ws)
        torch.cuda.synchronize()
        outs.append((scores.cpu().numpy(), mp.cpu().numpy(), mm.cpu().numpy()))
    ref = O.score(x["q_mask"], x["k_prompt"], x["k_mask"], wl.prompt_cu(), wl.live_cu())
    return outs, ref


def test_noalloc_matches_workspace_call_twice_in_a_row():
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    # two different problems back to back: the second call finds the first one's leftovers in the scratch
    cases = [
        (synth.scaled(synth.config(2), "noalloc_a", prompt_lens=(1500, 700), n_mask=96, n_q_heads=8, n_kv_heads=8), 0),
        (synth.scaled(synth.config(4), "noalloc_b", prompt_lens=(900,), n_mask=64, n_q_heads=8, n_kv_heads=2), 1),
        (synth.config(1), 0),
    ]
    for wl, layer in cases:
        ((s0, p0, m0), (s1, p1, m1)), (ref_s, ref_p, ref_m) = _score_both_ways(ctx, B, wl, layer)
        assert np.isfinite(s1).all() and np.isfinite(p1).all() and np.isfinite(m1).all()
        # the same kernels on the same inputs: the same bits, wherever the scratch lives
        assert np.array_equal(s0, s1) and np.array_equal(p0, p1) and np.array_equal(m0, m1)
        # and the paper's Eq. 6-7 / Eq. 14 sums, from the oracle
        assert_scores_close(s1, ref_s, what=f"{wl.name}: scores")
        assert_scores_close(p1, ref_p, what=f"{wl.name}: mass_p")
        assert_scores_close(m1, ref_m, what=f"{wl.name}: mass_m")
    assert ctx.maskkv_check_status() == 0
    ctx.close()


def test_noalloc_rejects_problems_beyond_its_scratch():
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    limit = int(B.lib.maskkv_score_noalloc_max_bytes())
    assert limit == 8 << 20
    # a ragged batch whose scratch need is far above the limit: refused before anything is launched
    lens = [32768] * 8
    pcu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    lcu = [r * 256 for r in range(9)]
    p = B.Problem(torch.bfloat16, 32, 32, 128, pcu, lcu, ctx.device)
    assert ctx.maskkv_workspace_bytes(p) > limit
    before = ctx.maskkv_launch_count()
    dummy = torch.zeros(64, dtype=torch.float32, device=ctx.device)
    rc = B.lib.maskkv_score_noalloc(ctx._h, ctypes.byref(p.desc), dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(),
                                    None, dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), None)
    assert rc == B.MASKKV_E_WORKSPACE
    assert ctx.maskkv_launch_count() == before
    ctx.close()
