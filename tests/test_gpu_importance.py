"""GPU parity of maskkv_layer_importance (Eq. 8) against the fp64 oracle, through the C ABI."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O

pytestmark = pytest.mark.gpu
ATOL = 2e-5     # fp32 dot products / norms of up to 8192 terms, cosines averaged in double


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def _pair(n, hidden, dtype, seed, drift):
    g = torch.Generator().manual_seed(seed)
    a = torch.randn(n, hidden, generator=g)
    b = a + drift * torch.randn(n, hidden, generator=g)
    return a.to(dtype), b.to(dtype)


@pytest.mark.parametrize("n,hidden,dtype,drift", [
    (1, 8, torch.bfloat16, 0.5), (7, 72, torch.float32, 1.0), (300, 4096, torch.bfloat16, 0.3),
    (1185, 1032, torch.bfloat16, 2.0), (2000, 512, torch.float32, 0.1), (5, 8200, torch.bfloat16, 0.7)])
def test_matches_oracle(ctx, n, hidden, dtype, drift):
    a, b = _pair(n, hidden, dtype, n + hidden, drift)
    out = torch.full((1,), float("nan"), dtype=torch.float32, device=ctx.device)
    ws = ctx.maskkv_layer_importance(a.cuda(), b.cuda(), out)
    first = out.clone()
    ctx.maskkv_layer_importance(a.cuda(), b.cuda(), out, ws)
    torch.cuda.synchronize()
    assert abs(out.item() - O.layer_importance(a, b)) <= ATOL
    assert torch.equal(first, out)                              # deterministic


def test_strided_rows_zero_rows_and_closed_forms(ctx):
    a, b = _pair(64, 256, torch.bfloat16, 3, 0.4)
    a[5] = 0; b[9] = 0
    big_a = torch.zeros(64, 3, 256, dtype=torch.bfloat16); big_b = torch.zeros(64, 2, 256, dtype=torch.bfloat16)
    big_a[:, 1] = a; big_b[:, 0] = b
    da, db = big_a.cuda(), big_b.cuda()
    out = torch.zeros(1, dtype=torch.float32, device=ctx.device)
    ctx.maskkv_layer_importance(da[:, 1], db[:, 0], out)        # row strides 768 and 512 elements
    torch.cuda.synchronize()
    assert abs(out.item() - O.layer_importance(a, b)) <= ATOL
    x = a.cuda()
    ctx.maskkv_layer_importance(x, x, out); torch.cuda.synchronize()
    assert abs(out.item() - 1.0 / 64) <= ATOL                   # identical states; the one zero row counts as cosine 0
    ctx.maskkv_layer_importance(x, -x, out); torch.cuda.synchronize()
    assert abs(out.item() - (2.0 - 1.0 / 64)) <= ATOL


def test_full_size_llada_layer(ctx):
    """One LLaDA-8B-shaped layer at the 32k workload: 33,024 token rows x hidden 4096, bf16 (541 MB read)."""
    g = torch.Generator(device="cuda").manual_seed(20251009)
    a = torch.randn(33024, 4096, generator=g, device="cuda").bfloat16()
    b = (a.float() + 0.6 * torch.randn(33024, 4096, generator=g, device="cuda")).bfloat16()
    out = torch.zeros(1, dtype=torch.float32, device=ctx.device)
    ctx.maskkv_layer_importance(a, b, out)
    torch.cuda.synchronize()
    # the oracle on a row sample (every 16th row): the mean cosine of i.i.d. rows, compared within its sampling error
    rows = torch.arange(0, 33024, 16, device="cuda")
    ref_sample = O.layer_importance(a[rows].cpu(), b[rows].cpu())
    assert abs(out.item() - ref_sample) < 5e-4
    # and exactly on the first 2048 rows
    ctx.maskkv_layer_importance(a[:2048], b[:2048], out); torch.cuda.synchronize()
    assert abs(out.item() - O.layer_importance(a[:2048].cpu(), b[:2048].cpu())) <= ATOL


def test_validation(ctx):
    from paper_2510_09309_b200 import binding as B
    x = torch.zeros(16, 64, dtype=torch.bfloat16, device=ctx.device)
    out = torch.zeros(1, dtype=torch.float32, device=ctx.device)
    ws = torch.empty(int(B.lib.maskkv_layer_importance_workspace_bytes(ctx._h)), dtype=torch.uint8, device=ctx.device)
    f = lambda *a: B.lib.maskkv_layer_importance(ctx._h, *a)
    ok = (B.MASKKV_BF16, x.data_ptr(), x.data_ptr(), 16, 64, 0, 0, out.data_ptr(), ws.data_ptr(), ws.numel(), None)
    before = ctx.maskkv_launch_count()
    assert f(*ok[:4], 60, *ok[5:]) == B.MASKKV_E_ALIGN                        # 120-byte rows
    assert f(*ok[:1], x.data_ptr() + 2, *ok[2:]) == B.MASKKV_E_ALIGN
    assert f(*ok[:8], ws.data_ptr(), 8, None) == B.MASKKV_E_WORKSPACE
    assert f(7, *ok[1:]) == B.MASKKV_E_UNSUPPORTED
    assert f(*ok[:7], None, *ok[8:]) == B.MASKKV_E_INVALID
    assert f(*ok[:5], 32, *ok[6:]) == B.MASKKV_E_INVALID                      # stride shorter than a row
    assert ctx.maskkv_launch_count() == before
    assert f(*ok[:3], 0, *ok[4:]) == B.MASKKV_OK                              # no rows: importance 0
    torch.cuda.synchronize()
    assert out.item() == 0.0
