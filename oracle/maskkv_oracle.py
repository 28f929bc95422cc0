"""CPU oracle for the MaskKV compress-and-attend path (TEST INFRASTRUCTURE, not product code).

A plain, slow, fp64 restatement of what the path computes, written from the paper's
definitions (Stage 1: Eq. 6-7; Stage 2: Eq. 9-16; the attention formula of the appendix proof,
Step 3).  Nothing here is tiled, fused, reordered or "online": every softmax materialises its
whole row.  numpy's matmul / exp / sort are the only library primitives used as steps.

It shares no code with the CUDA path and must never be imported by it.  Only the tests,
the smoke check and the benchmark's CPU-baseline leg may call into this module.

Notation (the paper overloads letters; this file uses one meaning each):
    N   prompt length of a request (n_p)          M   number of mask / live queries (n_m)
    H   query heads, H_kv key/value heads, g = H / H_kv
    d   head dimension                             k_l per-head mean budget of layer l (Eq. 13)
    k_{l,h} budget of KV head h in layer l (Eq. 15)

Readings taken where the paper is silent:
    * K_full is the request's N prompt keys followed by its M mask keys, no attention mask.
    * No smoothing or pooling of I is specified, so none is applied; `row_weights` (default 1)
      weights each mask row's vote and is the only hook.
    * Grouped-query attention: I, S_{m->p}, S_{m->m} are summed over the g query heads that share
      a KV head (each with its own softmax); H_kv takes the place of N_h in Eq. 15.
    * Floors of values that are integers in exact arithmetic use floor(x + 1e-6).
    * Budgets are clamped to [0, N]; budget lost to floors or clamping stays unallocated.
    * argtopk uses the total order (score descending, index ascending); kept indices are
      reported in ascending index order.  NaN scores rank below every number.
    * Eq. 8 (layer importance): a zero hidden-state row counts as cosine 0.
    * Mask-only projection: the input is the final (already normalised) hidden state; no bias term.

Pins: tests/test_oracle_*.py (brute force, closed forms, invariants, library special cases,
hand-derived budget examples under tests/golden/).  No function here is "parity unpinned".
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


def _f64(x) -> np.ndarray:
    """Widen any array-like (numpy array or CPU torch tensor, bf16 included) to float64, exactly."""
    if hasattr(x, "detach"):
        x = x.detach().cpu()
        if str(x.dtype) == "torch.bfloat16":
            x = x.float()
        x = x.numpy()
    return np.asarray(x, dtype=F64)


def attention_weights(q: np.ndarray, k: np.ndarray, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 6: A = softmax_row(q k^T * scale) for one head.  q [m, d], k [n, d] -> (A [m, n], lse [m]).

    The row maximum is subtracted before exponentiation (a mathematical identity of softmax)."""
    s = (q @ k.T) * scale
    mx = s.max(axis=1, keepdims=True)
    e = np.exp(s - mx)
    z = e.sum(axis=1, keepdims=True)
    return e / z, (mx + np.log(z))[:, 0]


def score(q_mask, k_prompt, k_mask, prompt_cu: Sequence[int], live_cu: Sequence[int],
          scale: Optional[float] = None, row_weights=None):
    """Eq. 6-7 and the two sums of Eq. 14, for a ragged batch.

    q_mask [sumM, H, d]; k_prompt [sumN, H_kv, d]; k_mask [sumM, H_kv, d]; *_cu cumulative lengths.
    Returns scores [H_kv, sumN] (I_j), mass_p [R, H_kv] (S_{m->p}), mass_m [R, H_kv] (S_{m->m})."""
    q_mask, k_prompt, k_mask = _f64(q_mask), _f64(k_prompt), _f64(k_mask)
    H, d = q_mask.shape[1], q_mask.shape[2]
    Hkv = k_prompt.shape[1]
    g = H // Hkv
    R = len(prompt_cu) - 1
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(d)
    w_all = np.ones(q_mask.shape[0], F64) if row_weights is None else _f64(row_weights)
    scores = np.zeros((Hkv, prompt_cu[-1]), F64)
    mass_p = np.zeros((R, Hkv), F64)
    mass_m = np.zeros((R, Hkv), F64)
    for r in range(R):
        p0, p1, l0, l1 = prompt_cu[r], prompt_cu[r + 1], live_cu[r], live_cu[r + 1]
        n = p1 - p0
        w = w_all[l0:l1]
        for hk in range(Hkv):
            k_full = np.concatenate([k_prompt[p0:p1, hk], k_mask[l0:l1, hk]], axis=0)
            imp = np.zeros(n, F64)
            sm = 0.0
            for h in range(hk * g, (hk + 1) * g):
                a, _ = attention_weights(q_mask[l0:l1, h], k_full, scale)
                imp += (w[:, None] * a[:, :n]).sum(axis=0)          # I_j = sum_i A_ij  (Eq. 7)
                sm += float((w * a[:, n:].sum(axis=1)).sum())       # mask-to-mask attention
            scores[hk, p0:p1] = imp
            mass_p[r, hk] = imp.sum()                                # mask-to-prompt attention
            mass_m[r, hk] = sm
    return scores, mass_p, mass_m


def vote_scores(q, k, voters, n_prompt: int, scale: Optional[float] = None):
    """The voting ablation (which tokens' attention ranks the prompt): I_j = sum over i in `voters` of A_ij for the
    n_prompt prompt tokens j, with A = softmax_row(q k^T * scale) over ALL tokens of the sequence [prompt ; response].
    Mask-Voting takes the mask rows as voters, Prompt-Voting the prompt rows, All-Voting every row, a window the last
    few prompt rows.  One request: q [T, H, d], k [T, H_kv, d], voters = row indices.  Returns I [H_kv, n_prompt],
    summed over the query heads that share a KV head as in `score`."""
    q, k = _f64(q), _f64(k)
    H, d = q.shape[1], q.shape[2]
    Hkv = k.shape[1]
    g = H // Hkv
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(d)
    rows = np.asarray(voters, dtype=np.int64)
    out = np.zeros((Hkv, n_prompt), F64)
    for hk in range(Hkv):
        for h in range(hk * g, (hk + 1) * g):
            if rows.size == 0:
                continue
            a, _ = attention_weights(q[rows, h], k[:, hk], scale)
            out[hk] += a[:, :n_prompt].sum(axis=0)
    return out


def layer_importance(h_in, h_out) -> float:
    """Eq. 8: I^(l) = 1 - (1/n) sum_i cos_sim(h_in_i, h_out_i) over the n token rows of one layer.

    h_in, h_out [n, hidden]: hidden states entering and leaving the layer's attention sub-layer (whether h_out carries
    the residual is the caller's choice; the paper does not say).  Reading for a zero row, where the cosine is
    undefined: it counts as cosine 0."""
    a, b = _f64(h_in), _f64(h_out)
    dot = (a * b).sum(axis=1)
    na = np.sqrt((a * a).sum(axis=1))
    nb = np.sqrt((b * b).sum(axis=1))
    den = na * nb
    cos = np.where(den > 0, dot / np.where(den > 0, den, 1.0), 0.0)
    return float(1.0 - cos.sum() / a.shape[0])


def refresh_set(v_cur, v_prev, delta: float, step: Optional[int] = None, t_r: Optional[int] = None):
    """Response-token refresh rule of the feature cache the method builds on (appendix, "Response tokens"):
    S_shift = { i : cos(V_i^(t), V_i^(t-1)) < delta },  S_period = all rows when t mod T_r = 0,  S = S_period U S_shift.

    v_cur, v_prev [n, width]: the value features of the n response tokens at this step and the previous one (all heads
    of a token side by side).  Returns (cos [n] float64, refresh [n] bool, indices of the refreshed rows, ascending).
    Reading for a zero row, where the cosine is undefined: cosine 0, as in layer_importance."""
    a, b = _f64(v_cur), _f64(v_prev)
    dot = (a * b).sum(axis=1)
    den = np.sqrt((a * a).sum(axis=1)) * np.sqrt((b * b).sum(axis=1))
    cos = np.where(den > 0, dot / np.where(den > 0, den, 1.0), 0.0)
    refresh = cos < delta
    if step is not None and t_r is not None and t_r > 0 and step % t_r == 0:
        refresh = np.ones_like(refresh)
    return cos, refresh, np.nonzero(refresh)[0].astype(np.int32)


def mask_project(hidden, positions, w_vocab):
    """Mask-only projection (appendix, "Mask-only Projection"): the vocabulary projection of the final hidden states,
    taken at the masked positions only - logits[m, v] = sum_k hidden[positions[m], k] * w_vocab[v, k].

    hidden [n_tokens, width], positions [n_mask] (any order, repeats allowed), w_vocab [vocab, width] (one row per
    vocabulary entry, as an output embedding is stored).  Returns logits [n_mask, vocab] float64: by definition the rows
    `positions` of the all-token projection, which is what the paper's change must leave untouched."""
    h, w = _f64(hidden), _f64(w_vocab)
    pos = np.asarray(positions, dtype=np.int64)
    if pos.size and (pos.min() < 0 or pos.max() >= h.shape[0]):
        raise IndexError("mask position outside the sequence")
    return h[pos] @ w.T


def guarded_floor(x: float) -> int:
    return int(math.floor(x + 1e-6))


def layer_budgets(k_p: int, beta: float, importance: Sequence[float],
                  is_boundary: Optional[Sequence[bool]] = None) -> List[int]:
    """Eq. 9-13: split the total budget k_p over layers.  Boundary group defaults to {first, last}."""
    L = len(importance)
    if is_boundary is None:
        is_boundary = [l == 0 or l == L - 1 for l in range(L)]
    k_base = guarded_floor(beta * k_p / L)                         # Eq. 9
    k_imp = k_p - L * k_base                                       # Eq. 10
    i_b = sum(float(importance[l]) for l in range(L) if is_boundary[l])
    i_m = sum(float(importance[l]) for l in range(L) if not is_boundary[l])
    n_b = sum(1 for l in range(L) if is_boundary[l])
    n_m = L - n_b
    k_group_b = (k_imp * i_b) / (i_b + i_m) if (i_b + i_m) > 0 else 0.0   # Eq. 11
    k_group_m = k_imp - k_group_b                                  # Eq. 12
    out = []
    for l in range(L):                                             # Eq. 13
        if is_boundary[l]:
            out.append(k_base + guarded_floor(k_group_b / n_b))
        else:
            out.append(k_base + guarded_floor(k_group_m / n_m))
    return out


def head_budgets(mass_p, mass_m, k_l, alpha: float, prompt_lens: Sequence[int],
                 capacity: Optional[int] = None):
    """Eq. 14-15 + clamp + exclusive prefix sum.

    mass_p, mass_m [R, H_kv] (fp32 values are widened); k_l an int or one int per request.
    Returns budgets int32 [R, H_kv] and offsets int32 [R*H_kv + 1].  Operation order (fp64, no fused
    multiply-add): P = Sp/(Sp+Sm); T = sum_h P_h in ascending h; Phat = P/T;
    x = alpha*k_l + ((1-alpha)*(H_kv*k_l))*Phat; k = floor(x + 1e-6) clamped to [0, N_r].
    If `capacity` is given, a segment that would run past it is clipped (and everything after is 0)."""
    sp, sm = _f64(mass_p), _f64(mass_m)
    R, Hkv = sp.shape
    kl = [int(k_l)] * R if np.isscalar(k_l) else [int(v) for v in k_l]
    budgets = np.zeros((R, Hkv), np.int32)
    for r in range(R):
        p = [float(sp[r, h]) / (float(sp[r, h]) + float(sm[r, h])) for h in range(Hkv)]   # Eq. 14
        t = 0.0
        for h in range(Hkv):
            t = t + p[h]
        for h in range(Hkv):
            phat = p[h] / t
            x = alpha * kl[r] + ((1.0 - alpha) * float(Hkv * kl[r])) * phat               # Eq. 15
            k = guarded_floor(x) if math.isfinite(x) else 0
            budgets[r, h] = min(max(k, 0), int(prompt_lens[r]))
    offsets = np.zeros(R * Hkv + 1, np.int32)
    run = 0
    flat = budgets.reshape(-1)
    for s in range(R * Hkv):
        if capacity is not None and run + int(flat[s]) > capacity:
            flat[s] = max(0, capacity - run)
        offsets[s] = run
        run += int(flat[s])
    offsets[R * Hkv] = run
    return budgets, offsets


def select(scores, budgets, prompt_cu: Sequence[int]) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 16 per (request, KV head): the k_{l,h} best prompt tokens, ascending request-local index.

    scores [H_kv, sumN] (any float type; compared as given), budgets [R, H_kv].
    Returns kept_idx (ragged, concatenated in (r, h) order) and offsets [R*H_kv + 1]."""
    sc = np.asarray(scores.detach().cpu().numpy() if hasattr(scores, "detach") else scores)
    budgets = np.asarray(budgets)
    R, Hkv = budgets.shape
    kept: List[np.ndarray] = []
    offsets = [0]
    for r in range(R):
        p0, p1 = prompt_cu[r], prompt_cu[r + 1]
        for h in range(Hkv):
            seg = sc[h, p0:p1].astype(F64)
            nan = np.isnan(seg)
            seg = np.where(nan, 0.0, seg)
            k = int(budgets[r, h])
            # total order: numbers before NaNs, then score descending, then index ascending
            order = np.lexsort((np.arange(seg.size), -seg, nan))
            top = np.sort(order[:k]).astype(np.int32)
            kept.append(top)
            offsets.append(offsets[-1] + k)
    idx = np.concatenate(kept) if kept else np.zeros(0, np.int32)
    return idx.astype(np.int32), np.asarray(offsets, np.int32)


def compact(k_prompt, v_prompt, kept_idx, offsets, prompt_cu: Sequence[int]):
    """Gather the kept rows: Kc[offsets[s]+t] = K_prompt[prompt_cu[r] + kept_idx[offsets[s]+t], h, :], s = r*H_kv + h.

    Returns (Kc, Vc) [total, d] in the dtype of the inputs (a pure copy: bit-exact)."""
    kp = k_prompt.detach().cpu() if hasattr(k_prompt, "detach") else k_prompt
    vp = v_prompt.detach().cpu() if hasattr(v_prompt, "detach") else v_prompt
    Hkv = kp.shape[1]
    R = len(prompt_cu) - 1
    total = int(offsets[-1])
    kc = kp[:0, 0].new_zeros((total, kp.shape[2])) if hasattr(kp, "new_zeros") else np.zeros((total, kp.shape[2]), kp.dtype)
    vc = vp[:0, 0].new_zeros((total, vp.shape[2])) if hasattr(vp, "new_zeros") else np.zeros((total, vp.shape[2]), vp.dtype)
    for r in range(R):
        for h in range(Hkv):
            s = r * Hkv + h
            for t in range(int(offsets[s]), int(offsets[s + 1])):
                row = prompt_cu[r] + int(kept_idx[t])
                kc[t] = kp[row, h]
                vc[t] = vp[row, h]
    return kc, vc


def attend(q_live, k_live, v_live, kc, vc, offsets, live_cu: Sequence[int], n_kv_heads: int,
           scale: Optional[float] = None, rows_cu: Optional[Sequence[int]] = None):
    """Attention of a later step over [compacted prompt segment ; live keys] (appendix proof, Step 3:
    out_m = sum_j alpha_mj V_j with alpha = softmax(q_m k_j / sqrt(d_k))).

    q_live [sumM, H, d]; k_live, v_live [sumM, H_kv, d]; kc, vc [total, d]; offsets [R*H_kv+1].
    Returns out [sumM, H, d] fp64 and lse [H, sumM] fp64 (log of the softmax denominator).

    rows_cu (partial refresh of the feature cache, appendix "Response tokens"): only some response rows are recomputed
    at a step, so q_live then holds the queries of those rows only, rows_cu[r] .. rows_cu[r+1] for request r, while the
    keys and values stay the segment followed by ALL live rows; out and lse are then per query row."""
    q, kl, vl, kc, vc = _f64(q_live), _f64(k_live), _f64(v_live), _f64(kc), _f64(vc)
    H, d = q.shape[1], q.shape[2]
    Hkv = n_kv_heads
    g = H // Hkv
    R = len(live_cu) - 1
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(d)
    out = np.zeros_like(q)
    lse = np.zeros((H, q.shape[0]), F64)
    q_cu = live_cu if rows_cu is None else rows_cu
    for r in range(R):
        l0, l1 = live_cu[r], live_cu[r + 1]
        q0, q1 = q_cu[r], q_cu[r + 1]
        if q1 == q0:
            continue
        for h in range(H):
            hk = h // g
            s = r * Hkv + hk
            keys = np.concatenate([kc[int(offsets[s]):int(offsets[s + 1])], kl[l0:l1, hk]], axis=0)
            vals = np.concatenate([vc[int(offsets[s]):int(offsets[s + 1])], vl[l0:l1, hk]], axis=0)
            a, ls = attention_weights(q[q0:q1, h], keys, scale)
            out[q0:q1, h] = a @ vals
            lse[h, q0:q1] = ls
    return out, lse
