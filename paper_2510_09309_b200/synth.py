"""Seeded synthetic inputs for the MaskKV compress-and-attend path.

This module only draws random tensors and applies the *structure* of the
workloads (planted heavy-hitter keys, information/structure head bias).  It
contains none of the method's arithmetic (no softmax, no scoring, no budget
rule, no top-k): both the CUDA path and the CPU oracle are fed from here and
neither depends on the other.

Shapes and layouts (all row-major, ``head_dim`` contiguous):

    q_mask   [sum(M_r), H,    d]   queries of the mask tokens at the first step
    k_prompt [sum(N_r), H_kv, d]   prompt keys        v_prompt  same shape
    k_mask   [sum(M_r), H_kv, d]   mask-token keys    v_mask    same shape
    q_live / k_live / v_live       a later denoising step's live region,
                                   shapes as q_mask / k_mask / v_mask

Values are drawn in fp32, structure is applied in fp32, and the result is
rounded to the workload dtype exactly once; those bytes go to both sides.
A CPU generator and a CUDA generator with the same seed give different
streams: a test always generates on one device and copies.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Sequence

import torch

BASE_SEED = 20251009 * 1000

# tensor ids for the sub-stream hash
_T_Q, _T_KP, _T_VP, _T_KM, _T_VM, _T_PLANT, _T_W, _T_QL, _T_KL, _T_VL = range(10)


@dataclass(frozen=True)
class Workload:
    """One synthetic workload (one of the five configurations or a scaled-down variant)."""
    name: str
    config_id: int
    dtype: str                       # "f32" | "bf16"
    n_layers: int
    n_q_heads: int                   # H
    n_kv_heads: int                  # H_kv
    head_dim: int                    # d
    prompt_lens: Sequence[int]       # N_r per request
    n_mask: int                      # M per request
    planted_per_head: Optional[int] = None   # count; None -> planted_frac * N_r
    planted_frac: float = 0.01
    planted_gain: float = 2.5        # logit standard deviations per unit query projection
    head_recipe: str = "none"        # "none" | "info_structure"
    mean_budget: int = 256           # B: nominal budget per head per layer
    alpha: float = 1.0               # head-budget mixing (Eq. 15); 1 -> uniform
    beta: float = 0.4                # layer-budget base fraction (Eq. 9)
    layer_profile: str = "uniform"   # "uniform" | "bimodal"
    attend_steps: int = 1

    @property
    def n_requests(self) -> int:
        return len(self.prompt_lens)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    def prompt_cu(self) -> List[int]:
        cu = [0]
        for n in self.prompt_lens:
            cu.append(cu[-1] + int(n))
        return cu

    def live_cu(self) -> List[int]:
        return [r * self.n_mask for r in range(self.n_requests + 1)]

    def layer_importance(self) -> List[float]:
        """Offline layer-importance profile handed to the layer-budget rule."""
        if self.layer_profile == "bimodal":
            prof = [0.2] * self.n_layers
            prof[0] = 0.6
            prof[-1] = 0.6
            return prof
        return [1.0] * self.n_layers

    def total_budget(self) -> int:
        """k_p: the budget summed over layers, in per-head units."""
        return self.n_layers * self.mean_budget


# Pinned prompt lengths of the ragged serving sweep: torch.randint(1024, 32769, (8,)) from a
# CPU generator seeded BASE_SEED + 5 gave (11821, 24615, 30881, 4417, 25124, 24565, 4504, 4321);
# the first and last are replaced by the two ends of the range so that the budget clamp and the
# maximum-length segment are always exercised.  Several lengths are odd, so segment starts
# are not 16-byte aligned; the kernels must cope with that.
RAGGED_PROMPT_LENS = (1024, 24615, 30881, 4417, 25124, 24565, 4504, 32768)


def config(i: int, **over) -> Workload:
    """The five configurations (1-based, as in the prose)."""
    if i == 1:
        w = Workload("tiny_fp32", 1, "f32", 1, 4, 4, 64, (512,), 64, planted_per_head=8,
                     planted_gain=3.0, mean_budget=32, alpha=1.0)
    elif i == 2:
        w = Workload("llada_layer_4k", 2, "bf16", 1, 32, 32, 128, (4096,), 256, mean_budget=256, alpha=1.0)
    elif i == 3:
        w = Workload("llada_stack_32k", 3, "bf16", 32, 32, 32, 128, (32768,), 256, mean_budget=256,
                     alpha=0.1, beta=0.4, layer_profile="bimodal", head_recipe="info_structure")
    elif i == 4:
        w = Workload("dream_gqa_16k", 4, "bf16", 28, 28, 4, 128, (16384,), 512, mean_budget=512, alpha=1.0)
    elif i == 5:
        w = Workload("ragged_serving", 5, "bf16", 32, 32, 32, 128, RAGGED_PROMPT_LENS, 256, mean_budget=256,
                     alpha=0.1, beta=0.4, layer_profile="bimodal", head_recipe="info_structure",
                     attend_steps=16)
    else:
        raise ValueError(f"no config {i}")
    return replace(w, **over) if over else w


def _gen(device, wl: Workload, layer: int, tensor_id: int, extra: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    h = (wl.config_id * 1_000_003 + layer * 10_007 + tensor_id * 101 + extra * 7) & 0x7FFFFFFF
    g.manual_seed(BASE_SEED + wl.config_id + (h << 8))
    return g


def _randn(shape, g: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def _unit(x: torch.Tensor, dim: int = -1) -> torch.Tensor:
    return x / x.norm(dim=dim, keepdim=True).clamp_min(1e-20)


def _set_component(x: torch.Tensor, w: torch.Tensor, value) -> torch.Tensor:
    """x: [T, heads, d]; w: [heads, d] unit vectors.  Replace x's component along w by `value`
    (a float or a per-head tensor [heads])."""
    proj = (x * w.unsqueeze(0)).sum(-1, keepdim=True)
    if torch.is_tensor(value):
        value = value.view(1, -1, 1)
    return x + (value - proj) * w.unsqueeze(0)


def layer_inputs(wl: Workload, layer: int = 0, device="cpu") -> Dict[str, torch.Tensor]:
    """First-step tensors of one layer: q_mask, k_prompt, v_prompt, k_mask, v_mask (+ planted index lists)."""
    dev = torch.device(device)
    H, Hkv, d, M, R = wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.n_mask, wl.n_requests
    g = wl.group
    sumN, sumM = wl.prompt_cu()[-1], R * M
    q = _randn((sumM, H, d), _gen(dev, wl, layer, _T_Q), dev)
    kp = _randn((sumN, Hkv, d), _gen(dev, wl, layer, _T_KP), dev)
    vp = _randn((sumN, Hkv, d), _gen(dev, wl, layer, _T_VP), dev)
    km = _randn((sumM, Hkv, d), _gen(dev, wl, layer, _T_KM), dev)
    vm = _randn((sumM, Hkv, d), _gen(dev, wl, layer, _T_VM), dev)

    cu = wl.prompt_cu()
    # mean mask-query direction per (request, KV head), taken BEFORE the head bias below is applied, so that the
    # planted keys and the information/structure bias live in different directions and do not interact
    u_dirs = [_unit(q[r * M:(r + 1) * M].view(M, Hkv, g, d).mean(dim=(0, 2))) for r in range(R)]
    if wl.head_recipe == "info_structure":
        # Even heads lean on the prompt (target prompt mass 0.7 before planting), odd heads on the mask
        # region (0.2): an exact logit offset t_h on the mask keys along a private direction w_h that every
        # other row - and the planting direction - is made orthogonal to.
        assert g == 1, "info/structure recipe is defined for MHA shapes"
        w = _unit(_randn((H, d), _gen(dev, wl, layer, _T_W), dev))
        p_target = torch.where(torch.arange(H, device=dev) % 2 == 0, 0.7, 0.2).to(torch.float32)
        kp = _set_component(kp, w, 0.0)
        km = _set_component(km, w, math.sqrt(d))
        for r in range(R):
            n_r = cu[r + 1] - cu[r]
            t_h = torch.log(n_r * (1.0 - p_target) / (p_target * M))
            sl = slice(r * M, (r + 1) * M)
            q[sl] = _set_component(q[sl], w, t_h)
            u_r = u_dirs[r]
            u_dirs[r] = _unit(u_r - (u_r * w).sum(-1, keepdim=True) * w)

    planted = []
    gp = _gen(dev, wl, layer, _T_PLANT)
    for r in range(R):
        n_r = cu[r + 1] - cu[r]
        cnt = wl.planted_per_head if wl.planted_per_head is not None else max(1, int(round(wl.planted_frac * n_r)))
        cnt = min(cnt, n_r)
        u = u_dirs[r]                                              # [H_kv, d] mean mask-query direction
        per_head = []
        for h in range(Hkv):
            idx = torch.randperm(n_r, generator=gp, device=dev)[:cnt]
            kp[cu[r] + idx, h] += wl.planted_gain * math.sqrt(d) * u[h]
            per_head.append(idx.sort().values.cpu())
        planted.append(per_head)

    dt = wl.torch_dtype
    return {
        "q_mask": q.to(dt).contiguous(), "k_prompt": kp.to(dt).contiguous(), "v_prompt": vp.to(dt).contiguous(),
        "k_mask": km.to(dt).contiguous(), "v_mask": vm.to(dt).contiguous(), "planted": planted,
    }


def live_inputs(wl: Workload, layer: int = 0, step: int = 0, device="cpu") -> Dict[str, torch.Tensor]:
    """A later denoising step's live region: an independent draw of q_live, k_live, v_live."""
    dev = torch.device(device)
    H, Hkv, d, R, M = wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.n_requests, wl.n_mask
    dt = wl.torch_dtype
    return {
        "q_live": _randn((R * M, H, d), _gen(dev, wl, layer, _T_QL, step + 1), dev).to(dt).contiguous(),
        "k_live": _randn((R * M, Hkv, d), _gen(dev, wl, layer, _T_KL, step + 1), dev).to(dt).contiguous(),
        "v_live": _randn((R * M, Hkv, d), _gen(dev, wl, layer, _T_VL, step + 1), dev).to(dt).contiguous(),
    }


def scaled(wl: Workload, name: str, **over) -> Workload:
    """A scaled-down variant of a config that keeps its structure (for tests the oracle finishes in seconds)."""
    return replace(wl, name=name, **over)


def project_inputs(n_tokens: int, width: int, vocab: int, n_mask: int, device="cpu", seed: int = 0,
                   w_std: float = 0.02) -> Dict[str, torch.Tensor]:
    """Inputs of the mask-only projection: final hidden states [n_tokens, width] (unit variance, as after the final
    normalisation), an output embedding [vocab, width] (normal, std 0.02 as at initialisation) and the masked
    positions (int32, ascending: the last n_mask * 5 / 4 rows with every fifth already decoded, as late in a
    generation).  bf16; generated in pieces so that the full-size embedding never exists in fp32."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(BASE_SEED + 77_003 + seed)
    hidden = torch.randn((n_tokens, width), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    w = torch.empty((vocab, width), dtype=torch.bfloat16, device=dev)
    step = 8192
    for v0 in range(0, vocab, step):
        rows = min(step, vocab - v0)
        w[v0:v0 + rows] = (torch.randn((rows, width), generator=g, device=dev, dtype=torch.float32) * w_std).to(torch.bfloat16)
    span = min(n_tokens, n_mask + n_mask // 4)
    cand = torch.arange(n_tokens - span, n_tokens, dtype=torch.int64)
    keep = torch.ones(span, dtype=torch.bool)
    drop = span - min(span, n_mask)
    if drop > 0:
        keep[torch.arange(drop) * 5 % span] = False
    pos = cand[keep][:n_mask]
    if pos.numel() < n_mask:                                   # fewer tokens than masks: repeat rows
        pos = torch.arange(n_mask, dtype=torch.int64) % max(n_tokens, 1)
    return {"hidden": hidden, "w_vocab": w, "positions": pos.to(torch.int32).to(dev)}
