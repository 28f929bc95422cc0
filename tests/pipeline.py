"""Test helpers: run the CUDA path through the C-ABI binding, run the oracle, compare.

The oracle is never fed anything the CUDA path produced; the CUDA stages may be fed oracle outputs
(rounded to the device dtype) so that each stage is compared on identical inputs."""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth

SCORE_RTOL = 1e-3          # scores, bf16 inputs with fp32 accumulation (relative)
BAND_RTOL = 1e-4           # kept-index sets are compared outside this relative band around the cut
ATTEND_ATOL = {"bf16": 2e-2, "f32": 1e-5}


def to_dev(x, device="cuda"):
    if isinstance(x, np.ndarray):
        x = torch.from_numpy(x)
    return x.to(device).contiguous()


class LayerRun:
    """Owns the device buffers of one layer's pass through the five calls."""

    def __init__(self, ctx, wl: synth.Workload, capacity: Optional[int] = None, k_l: Optional[int] = None):
        from paper_2510_09309_b200 import binding as B
        self.B, self.ctx, self.wl = B, ctx, wl
        dev = ctx.device
        self.p = B.Problem(wl.torch_dtype, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.prompt_cu(), wl.live_cu(), dev)
        R, Hkv, H = wl.n_requests, wl.n_kv_heads, wl.n_q_heads
        self.k_l = wl.mean_budget if k_l is None else k_l
        bound = sum(min(2 * Hkv * self.k_l, Hkv * n) for n in wl.prompt_lens)
        self.capacity = bound if capacity is None else capacity
        self.scores = torch.full((Hkv, self.p.sumN), float("nan"), dtype=torch.float32, device=dev)
        self.mass_p = torch.zeros((R, Hkv), dtype=torch.float32, device=dev)
        self.mass_m = torch.zeros((R, Hkv), dtype=torch.float32, device=dev)
        self.budgets = torch.zeros((R, Hkv), dtype=torch.int32, device=dev)
        self.offsets = torch.zeros(R * Hkv + 1, dtype=torch.int32, device=dev)
        self.kept = torch.full((max(self.capacity, 1),), -1, dtype=torch.int32, device=dev)
        self.kc = torch.zeros((max(self.capacity, 1), wl.head_dim), dtype=wl.torch_dtype, device=dev)
        self.vc = torch.zeros_like(self.kc)
        self.out = torch.zeros((self.p.sumM, H, wl.head_dim), dtype=wl.torch_dtype, device=dev)
        self.lse = torch.zeros((H, self.p.sumM), dtype=torch.float32, device=dev)
        self.ws = torch.empty(max(ctx.maskkv_workspace_bytes(self.p), 16), dtype=torch.uint8, device=dev)

    def score(self, x: Dict[str, torch.Tensor], row_weights=None):
        self.ctx.maskkv_score(self.p, x["q_mask"], x["k_prompt"], x["k_mask"], self.scores, self.mass_p, self.mass_m,
                              self.ws, row_weights)

    def budget(self, alpha=None, mass_p=None, mass_m=None, k_l_per_request=None):
        self.ctx.maskkv_budget(self.p, self.k_l, self.wl.alpha if alpha is None else alpha,
                               self.mass_p if mass_p is None else mass_p, self.mass_m if mass_m is None else mass_m,
                               self.capacity, self.budgets, self.offsets, k_l_per_request)

    def select(self, scores=None, budgets=None, offsets=None):
        self.ctx.maskkv_select(self.p, self.scores if scores is None else scores,
                               self.budgets if budgets is None else budgets,
                               self.offsets if offsets is None else offsets, self.kept, self.ws)

    def compact(self, x, kept=None, offsets=None):
        self.ctx.maskkv_compact(self.p, x["k_prompt"], x["v_prompt"], self.kept if kept is None else kept,
                                self.offsets if offsets is None else offsets, self.capacity, self.kc, self.vc)

    def attend(self, live, kc=None, vc=None, offsets=None):
        self.ctx.maskkv_attend(self.p, live["q_live"], live["k_live"], live["v_live"], self.kc if kc is None else kc,
                               self.vc if vc is None else vc, self.offsets if offsets is None else offsets,
                               (self.kc if kc is None else kc).shape[0], self.out, self.lse)


def oracle_layer(wl: synth.Workload, x, live, k_l: int, alpha: float, heads: Optional[Sequence[int]] = None):
    """The whole path in the oracle.  (heads is unused here; full problem.)"""
    pcu, lcu = wl.prompt_cu(), wl.live_cu()
    sc, mp, mm = O.score(x["q_mask"], x["k_prompt"], x["k_mask"], pcu, lcu)
    # the path hands fp32 scores and masses to the next stage; the oracle takes its decisions on the same precision
    sc32, mp32, mm32 = sc.astype(np.float32), mp.astype(np.float32), mm.astype(np.float32)
    bud, off = O.head_budgets(mp32, mm32, k_l, alpha, wl.prompt_lens)
    idx, off2 = O.select(sc32, bud, pcu)
    assert (off == off2).all()
    kc, vc = O.compact(x["k_prompt"], x["v_prompt"], idx, off, pcu)
    out, lse = O.attend(live["q_live"], live["k_live"], live["v_live"], kc, vc, off, lcu, wl.n_kv_heads)
    return dict(scores=sc, scores32=sc32, mass_p=mp, mass_m=mm, mass_p32=mp32, mass_m32=mm32, budgets=bud, offsets=off,
                kept=idx, kc=kc, vc=vc, out=out, lse=lse)


def assert_scores_close(got: np.ndarray, ref: np.ndarray, rtol=SCORE_RTOL, what="scores"):
    err = np.abs(got.astype(np.float64) - ref) / np.maximum(np.abs(ref), 1e-30)
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    assert err.max() <= rtol, f"{what}: max relative error {err.max():.3e} > {rtol}"
    return float(err.max())


def assert_kept_within_band(kept: np.ndarray, ref_scores: np.ndarray, k: int, band=BAND_RTOL):
    """Eq. 16 up to the tolerance band at the cut: with c the oracle's k-th largest score, every token
    scoring above c(1+band) is kept, none below c(1-band) is, the count is exactly k, and the list is
    strictly ascending."""
    n = ref_scores.shape[0]
    assert kept.shape[0] == k
    if k == 0:
        return 0
    assert (np.diff(kept) > 0).all() and kept[0] >= 0 and kept[-1] < n
    if k == n:
        return 0
    c = np.sort(ref_scores)[::-1][k - 1]
    must = np.nonzero(ref_scores > c * (1 + band))[0]
    must_not = np.nonzero(ref_scores < c * (1 - band))[0]
    ks = set(kept.tolist())
    assert all(int(j) in ks for j in must), "a token above the band was evicted"
    assert not any(int(j) in ks for j in must_not), "a token below the band was kept"
    return n - len(must) - len(must_not)
