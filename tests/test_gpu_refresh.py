"""GPU parity of maskkv_refresh_set (response-token refresh rule: cos(V_t, V_{t-1}) < delta) against the fp64 oracle,
through the C ABI."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O

pytestmark = pytest.mark.gpu
COS_ATOL = 2e-6     # fp32 dot products and norms of up to 8192 terms
BAND = 1e-5         # rows whose cosine is this close to delta may fall on either side in fp32


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def _pair(n, width, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    a = torch.randn(n, width, generator=g)
    drift = torch.rand(n, 1, generator=g) * 1.5                       # cosines spread between about 0.55 and 1
    b = a + drift * torch.randn(n, width, generator=g)
    return a.to(dtype), b.to(dtype)


def _run(ctx, a, b, delta, refresh_all=False, want_cos=True):
    n = a.shape[0]
    idx = torch.full((max(n, 1),), -7, dtype=torch.int32, device=ctx.device)
    cnt = torch.full((1,), -1, dtype=torch.int32, device=ctx.device)
    cos = torch.full((max(n, 1),), float("nan"), dtype=torch.float32, device=ctx.device) if want_cos else None
    ctx.maskkv_refresh_set(a, b, delta, idx, cnt, refresh_all, cos)
    torch.cuda.synchronize()
    c = int(cnt.item())
    return idx.cpu().numpy()[:c], c, (cos.cpu().numpy()[:n] if want_cos else None)


def _check(ctx, a, b, delta):
    ref_cos, ref_mask, _ = O.refresh_set(a, b, delta)
    idx, c, cos = _run(ctx, a.cuda(), b.cuda(), delta)
    assert np.abs(cos - ref_cos).max(initial=0.0) <= COS_ATOL
    assert np.all(np.diff(idx) > 0)                                   # ascending, no duplicates
    got = np.zeros(a.shape[0], bool); got[idx] = True
    assert np.array_equal(got, cos < np.float32(delta))               # the list is the kernel's own fp32 decision
    sure = np.abs(ref_cos - delta) > BAND
    assert np.array_equal(got[sure], ref_mask[sure])                  # and the oracle's wherever fp32 cannot flip it
    idx2, c2, _ = _run(ctx, a.cuda(), b.cuda(), delta, want_cos=False)
    assert c2 == c and np.array_equal(idx2, idx)


@pytest.mark.parametrize("n,width,dtype", [
    (1, 8, torch.bfloat16), (5, 72, torch.float32), (256, 4096, torch.bfloat16), (1024, 1024, torch.bfloat16),
    (1025, 64, torch.float32), (3000, 256, torch.bfloat16), (37, 8200, torch.bfloat16)])
def test_matches_oracle(ctx, n, width, dtype):
    a, b = _pair(n, width, dtype, n * 31 + width)
    for delta in (0.8, 0.95, -1.0, 1.5):
        _check(ctx, a, b, delta)


def test_periodic_step_empty_input_zero_rows_and_strides(ctx):
    a, b = _pair(300, 128, torch.bfloat16, 5)
    idx, c, cos = _run(ctx, a.cuda(), b.cuda(), 0.9, refresh_all=True)
    assert c == 300 and np.array_equal(idx, np.arange(300))
    assert np.abs(cos - O.refresh_set(a, b, 0.9)[0]).max() <= COS_ATOL
    idx, c, _ = _run(ctx, a.cuda(), b.cuda(), 0.9, refresh_all=True, want_cos=False)
    assert c == 300 and np.array_equal(idx, np.arange(300))
    idx, c, _ = _run(ctx, a[:0].cuda(), b[:0].cuda(), 0.9)
    assert c == 0
    a[3] = 0; b[7] = 0
    big_a = torch.zeros(300, 3, 128, dtype=torch.bfloat16); big_b = torch.zeros(300, 2, 128, dtype=torch.bfloat16)
    big_a[:, 2] = a; big_b[:, 1] = b
    da, db = big_a.cuda(), big_b.cuda()
    ref_cos, ref_mask, ref_idx = O.refresh_set(a, b, 0.85)
    idx, c, cos = _run(ctx, da[:, 2], db[:, 1], 0.85)                 # row strides 384 and 256 elements
    assert cos[3] == 0.0 and cos[7] == 0.0 and 3 in idx and 7 in idx
    sure = np.abs(ref_cos - 0.85) > BAND
    got = np.zeros(300, bool); got[idx] = True
    assert np.array_equal(got[sure], ref_mask[sure])
    assert ctx.maskkv_check_status() == 0


def test_argument_validation(ctx):
    from paper_2510_09309_b200 import binding as B
    a, b = _pair(8, 64, torch.bfloat16, 9)
    da, db = a.cuda(), b.cuda()
    idx = torch.zeros(8, dtype=torch.int32, device=ctx.device); cnt = torch.zeros(1, dtype=torch.int32, device=ctx.device)
    before = ctx.maskkv_launch_count()
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_refresh_set(da[:, :60], db[:, :60], 0.9, idx, cnt)  # 120-byte rows: not a multiple of 16
    assert e.value.code == B.MASKKV_E_ALIGN
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_refresh_set(da, db, float("nan"), idx, cnt)
    assert e.value.code == B.MASKKV_E_INVALID
    with pytest.raises(B.MaskKVError) as e:
        ctx.maskkv_refresh_set(da, db, 0.9, None, cnt)
    assert e.value.code == B.MASKKV_E_INVALID
    assert ctx.maskkv_launch_count() == before                        # a refused call launches nothing
