"""GPU parity of maskkv_mask_project (appendix, "Mask-only Projection": the vocabulary projection at the masked
positions only) against the fp64 oracle, through the C ABI.

Tolerance.  Products of bf16 values are exact in fp32; the tensor core adds `width` of them into an fp32 accumulator,
so the error of a logit is bounded by width * 2^-24 * sum_k |h_k w_k| (every addition rounded or truncated at the
running sum's magnitude) and in practice stays near sqrt(width) * 2^-24 of the result.  The tests allow
TOL_FACTOR = 2^-17 of the row's sum of magnitudes: 1/32 of the worst-case bound at width 4096, an order of magnitude
above what is observed.  bf16 output adds half a bf16 ulp (2^-9 relative)."""
import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth

pytestmark = pytest.mark.gpu
TOL_FACTOR = 2.0 ** -17


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def _magnitudes(hidden, positions, w):
    return np.abs(hidden.double().numpy())[np.asarray(positions)] @ np.abs(w.double().numpy()).T


def _check(got, hidden, positions, w, bf16_out=False):
    ref = O.mask_project(hidden, positions, w)
    tol = TOL_FACTOR * _magnitudes(hidden, positions, w) + 1e-30
    if bf16_out:
        tol = tol + np.abs(ref) * 2.0 ** -8
    err = np.abs(got.double().numpy() - ref)
    assert (err <= tol).all(), f"worst error {err.max():.3e} at {np.unravel_index(np.argmax(err - tol), err.shape)}, allowed {tol.flat[np.argmax(err - tol)]:.3e}"
    return err.max()


def _run(ctx, x, out_dtype=torch.float32, positions="given", out_stride=None):
    from paper_2510_09309_b200 import binding as B
    hidden, w = x["hidden"], x["w_vocab"]
    pos = x["positions"] if positions == "given" else None
    n_mask = x["positions"].numel()
    vocab = w.shape[0]
    ld = out_stride or (vocab + 7) // 8 * 8                  # rows start on 16-byte boundaries
    buf = torch.full((n_mask, ld), float("nan"), dtype=out_dtype, device=hidden.device)
    out = buf[:, :vocab]
    ws = torch.empty(B.maskkv_mask_project_workspace_bytes(n_mask, hidden.shape[1]), dtype=torch.uint8, device=hidden.device) if pos is not None else None
    ctx.maskkv_mask_project(hidden, w, out, pos, ws)
    torch.cuda.synchronize()
    return out, buf


@pytest.mark.parametrize("n_tokens,width,vocab,n_mask", [
    (300, 192, 1000, 70),        # one row block, ragged vocabulary (not a multiple of 32), three k blocks
    (900, 512, 5000, 300),       # two row blocks, the second with 44 rows (one accumulator unused)
    (400, 200, 777, 129),        # width not a multiple of 64: the last k block reads zeros; 129 rows = second half by one
    (64, 64, 33, 5),             # everything smaller than one tile
    (2048, 1024, 40000, 512),    # several waves of tiles per CTA
    (300, 64, 16, 200),          # pair kernel, a vocabulary of one 16-entry unit
    (300, 72, 8, 130),           # pair kernel, fewer entries than one unit, width 72
    (40, 8, 100, 10),            # width smaller than a k block
    (1000, 128, 2368, 1000),     # four row blocks on 148 one-unit tiles
])
def test_parity_fp32_out(ctx, n_tokens, width, vocab, n_mask):
    x = synth.project_inputs(n_tokens, width, vocab, n_mask, "cuda", seed=n_mask)
    out, _ = _run(ctx, x)
    assert ctx.maskkv_check_status() == 0
    _check(out.cpu(), x["hidden"].cpu(), x["positions"].cpu().numpy(), x["w_vocab"].cpu())


def test_bf16_out_padded_rows_and_positions_with_repeats(ctx):
    x = synth.project_inputs(500, 256, 2000, 96, "cuda", seed=3)
    g = torch.Generator().manual_seed(5)
    x["positions"] = torch.randint(0, 500, (96,), generator=g, dtype=torch.int32).cuda()      # unordered, with repeats
    out, buf = _run(ctx, x, torch.bfloat16, out_stride=2048)
    assert ctx.maskkv_check_status() == 0
    _check(out.float().cpu(), x["hidden"].cpu(), x["positions"].cpu().numpy(), x["w_vocab"].cpu(), bf16_out=True)
    assert torch.isnan(buf[:, 2000:].float()).all()                                          # nothing written past a row's end


def test_rows_in_place_with_strided_operands(ctx):
    g = torch.Generator(device="cuda").manual_seed(11)
    hid_buf = torch.randn((160, 320), generator=g, device="cuda").to(torch.bfloat16)
    w_buf = (torch.randn((700, 264), generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    hidden, w = hid_buf[:, :256], w_buf[:, :256]                                               # row strides 320 and 264
    x = {"hidden": hidden, "w_vocab": w, "positions": torch.arange(150, dtype=torch.int32, device="cuda")}
    out, _ = _run(ctx, x, positions=None)
    assert ctx.maskkv_check_status() == 0
    _check(out.cpu(), hidden.cpu(), np.arange(150), w.cpu())
    # the same rows through the gather give the same bits
    out2, _ = _run(ctx, x)
    assert torch.equal(out, out2)


def test_single_cta_and_pair_kernels_agree_bit_for_bit(monkeypatch):
    """More than 128 masked rows run on pairs of CTAs; bit 0 of MASKKV_KERNEL_CHOICE (read when a context is created) keeps
    them on the one-CTA kernel.  Both add the k blocks in the same order, so the logits must be identical."""
    from paper_2510_09309_b200 import binding as B
    x = synth.project_inputs(700, 448, 3000, 300, "cuda", seed=4)
    outs = []
    for force in ("0", "1"):
        monkeypatch.setenv("MASKKV_KERNEL_CHOICE", force)
        c = B.Context(0)
        try:
            out, _ = _run(c, x)
            assert c.maskkv_check_status() == 0
            outs.append(out.cpu())
        finally:
            c.close()
    assert torch.equal(outs[0], outs[1])
    _check(outs[1], x["hidden"].cpu(), x["positions"].cpu().numpy(), x["w_vocab"].cpu())


def test_seeded_shape_sweep_pair_kernel_against_one_cta_kernel_and_oracle(monkeypatch):
    """Twenty seeded shapes (129-700 masked rows, widths that are multiples of 8 but mostly not of 64, vocabularies
    that are multiples of nothing): the pair kernel must reproduce the one-CTA kernel's bits, and both the oracle."""
    from paper_2510_09309_b200 import binding as B
    rng = np.random.default_rng(20251009)
    shapes = [(int(rng.integers(129, 701)), int(rng.integers(8, 140)) * 8, int(rng.integers(40, 9000))) for _ in range(20)]
    outs = {}
    for force in ("0", "1"):
        monkeypatch.setenv("MASKKV_KERNEL_CHOICE", force)
        c = B.Context(0)
        try:
            for i, (n_mask, width, vocab) in enumerate(shapes):
                x = synth.project_inputs(n_mask + 50, width, vocab, n_mask, "cuda", seed=100 + i)
                dt = torch.bfloat16 if i % 3 == 2 else torch.float32
                out, _ = _run(c, x, dt)
                outs[(force, i)] = out.cpu()
                if force == "8":
                    assert torch.equal(outs[("0", i)], outs[("8", i)]), f"shape {shapes[i]}: the two kernels differ"
                    if i % 4 == 0:
                        _check(out.float().cpu(), x["hidden"].cpu(), x["positions"].cpu().numpy(), x["w_vocab"].cpu(), bf16_out=dt == torch.bfloat16)
            assert c.maskkv_check_status() == 0
        finally:
            c.close()


def test_out_of_range_position_is_flagged_and_gives_a_zero_row(ctx):
    from paper_2510_09309_b200 import binding as B
    x = synth.project_inputs(100, 128, 300, 8, "cuda", seed=2)
    x["positions"][3] = 100
    x["positions"][6] = -1
    out, _ = _run(ctx, x)
    assert ctx.maskkv_check_status() == B.MASKKV_FLAG_BOUNDS
    good = [0, 1, 2, 4, 5, 7]
    assert not out[3].any() and not out[6].any()
    _check(out.cpu()[good], x["hidden"].cpu(), x["positions"].cpu().numpy()[good], x["w_vocab"].cpu())


def test_argument_errors_launch_nothing(ctx):
    from paper_2510_09309_b200 import binding as B
    x = synth.project_inputs(64, 128, 256, 16, "cuda")
    hidden, w, pos = x["hidden"], x["w_vocab"], x["positions"]
    out = torch.zeros((16, 256), dtype=torch.float32, device="cuda")
    ws = torch.empty(B.maskkv_mask_project_workspace_bytes(16, 128), dtype=torch.uint8, device="cuda")
    before = ctx.maskkv_launch_count()
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_mask_project(hidden.float(), w.float(), out, pos, ws)
    assert e.value.code == B.MASKKV_E_UNSUPPORTED
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_mask_project(hidden, w, out, pos, ws[:256])
    assert e.value.code == B.MASKKV_E_WORKSPACE
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_mask_project(hidden[:, :100], w[:, :100], out, pos, ws)                     # width not a multiple of 8
    assert e.value.code == B.MASKKV_E_ALIGN
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_mask_project(hidden, w, torch.zeros((16, 258), dtype=torch.float32, device="cuda")[:, :256], pos, ws)
    assert e.value.code == B.MASKKV_E_ALIGN                                                    # fp32 row stride not a multiple of 4
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_mask_project(hidden[:8], w, out, None, None)                                # 16 rows asked in place, 8 exist
    assert e.value.code == B.MASKKV_E_INVALID
    ctx.maskkv_mask_project(hidden, w, out[:0], pos[:0], None)                                 # no masked position: nothing to do
    assert ctx.maskkv_launch_count() == before
    torch.cuda.synchronize()
    assert ctx.maskkv_check_status() == 0


def test_full_size_llada_vocabulary_sampled(ctx):
    """The workload bench.py times: 256 masked rows of a 33,024-token sequence, width 4096, vocabulary 126,464."""
    x = synth.project_inputs(32768 + 256, 4096, 126464, 256, "cuda", seed=1)
    out, _ = _run(ctx, x)
    assert ctx.maskkv_check_status() == 0
    assert torch.isfinite(out).all()
    g = torch.Generator().manual_seed(9)
    cols = torch.cat([torch.arange(0, 300), torch.arange(126464 - 300, 126464), torch.randint(0, 126464, (3000,), generator=g)]).unique()
    pos = x["positions"].cpu().numpy()
    w_s = x["w_vocab"][cols.cuda()].cpu()
    h_s = x["hidden"][x["positions"].long()].cpu()
    worst = _check(out[:, cols.cuda()].cpu(), h_s, np.arange(256), w_s)
    assert pos.min() >= 32768 + 256 - 320 and worst < 1e-4
    # every tile contributes: column sums of the logits against the oracle's on the sampled columns are covered above;
    # here the remaining property - no column was left unwritten (the buffer started as NaN)
    assert not torch.isnan(out).any()
