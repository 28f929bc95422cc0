"""ctypes binding of libmaskkv.so: argument marshalling only, one Python function per C entry point.

Every step of the path runs in the CUDA library; this module owns no arithmetic.  Tensors are torch
tensors used purely as device memory; the current torch stream is passed to every call.  If the
library is missing the import fails loudly: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmaskkv.so")

MASKKV_OK = 0
MASKKV_E_INVALID, MASKKV_E_UNSUPPORTED, MASKKV_E_ALIGN, MASKKV_E_WORKSPACE = -1, -2, -3, -4
MASKKV_E_CAPACITY, MASKKV_E_CUDA, MASKKV_E_TIMEOUT = -5, -6, -7
MASKKV_F32, MASKKV_BF16 = 0, 1
MASKKV_FLAG_TIMEOUT, MASKKV_FLAG_CAPACITY, MASKKV_FLAG_BOUNDS, MASKKV_FLAG_FALLBACK = 1, 2, 4, 8

EXPORTS = (
    "maskkv_create", "maskkv_destroy", "maskkv_status_string", "maskkv_check_status", "maskkv_selftest_wait_expiry", "maskkv_selftest_exp_rate", "maskkv_launch_count", "maskkv_last_cuda_error",
    "maskkv_tensor_core_launch_count",
    "maskkv_workspace_bytes",
    "maskkv_layer_budgets", "maskkv_layer_importance", "maskkv_layer_importance_workspace_bytes", "maskkv_refresh_set", "maskkv_mask_project", "maskkv_mask_project_workspace_bytes", "maskkv_score", "maskkv_score_all_keys", "maskkv_score_noalloc", "maskkv_score_noalloc_max_bytes", "maskkv_budget", "maskkv_select", "maskkv_compact", "maskkv_attend", "maskkv_attend_rows",
)


class maskkv_desc_t(C.Structure):
    _fields_ = [
        ("dtype", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("n_requests", C.c_int32), ("softmax_scale", C.c_float),
        ("prompt_cu", C.POINTER(C.c_int32)), ("live_cu", C.POINTER(C.c_int32)),
        ("prompt_cu_dev", C.c_void_p), ("live_cu_dev", C.c_void_p),
        ("q_token_stride", C.c_int64), ("q_head_stride", C.c_int64),
        ("kv_token_stride", C.c_int64), ("kv_head_stride", C.c_int64),
    ]


class MaskKVError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} ({code})")
        self.code = code


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2510_09309_b200.build` "
            "(there is no CPU or PyTorch fallback for the MaskKV path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    dp = C.POINTER(maskkv_desc_t)
    lib.maskkv_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.maskkv_destroy.argtypes = [vp]
    lib.maskkv_status_string.argtypes = [C.c_int]
    lib.maskkv_status_string.restype = C.c_char_p
    lib.maskkv_check_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    lib.maskkv_last_cuda_error.argtypes = [vp]
    lib.maskkv_last_cuda_error.restype = C.c_char_p
    lib.maskkv_selftest_wait_expiry.argtypes = [vp, vp]
    lib.maskkv_selftest_exp_rate.argtypes = [vp, i32, vp, C.POINTER(C.c_int64), vp]
    lib.maskkv_launch_count.argtypes = [vp]
    lib.maskkv_launch_count.restype = C.c_uint64
    lib.maskkv_tensor_core_launch_count.argtypes = [vp]
    lib.maskkv_tensor_core_launch_count.restype = C.c_uint64
    lib.maskkv_workspace_bytes.argtypes = [vp, dp]
    lib.maskkv_workspace_bytes.restype = sz
    lib.maskkv_layer_budgets.argtypes = [i64, C.c_double, i32, C.POINTER(C.c_double), C.POINTER(C.c_uint8), C.POINTER(i32)]
    lib.maskkv_layer_importance_workspace_bytes.argtypes = [vp]
    lib.maskkv_layer_importance_workspace_bytes.restype = sz
    lib.maskkv_layer_importance.argtypes = [vp, i32, vp, vp, i64, i32, i64, i64, vp, vp, sz, vp]
    lib.maskkv_refresh_set.argtypes = [vp, i32, vp, vp, i64, i32, i64, i64, C.c_float, i32, vp, vp, vp, vp]
    lib.maskkv_mask_project_workspace_bytes.argtypes = [i64, i32]
    lib.maskkv_mask_project_workspace_bytes.restype = sz
    lib.maskkv_mask_project.argtypes = [vp, i32, vp, i64, i32, i64, vp, i32, vp, i32, i64, i32, vp, i64, vp, sz, vp]
    lib.maskkv_score.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.maskkv_score_all_keys.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.maskkv_score_noalloc.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.maskkv_score_noalloc_max_bytes.argtypes = []
    lib.maskkv_score_noalloc_max_bytes.restype = sz
    lib.maskkv_budget.argtypes = [vp, dp, i32, vp, C.c_double, vp, vp, i64, vp, vp, vp]
    lib.maskkv_select.argtypes = [vp, dp, vp, vp, vp, vp, vp, sz, vp]
    lib.maskkv_compact.argtypes = [vp, dp, vp, vp, vp, vp, i64, vp, vp, vp]
    lib.maskkv_attend.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp]
    lib.maskkv_attend_rows.argtypes = [vp, dp, vp, C.POINTER(C.c_int32), vp, vp, vp, vp, vp, vp, i64, vp, vp, vp]
    for name in EXPORTS:
        if name not in ("maskkv_status_string", "maskkv_workspace_bytes", "maskkv_launch_count", "maskkv_tensor_core_launch_count",
                        "maskkv_score_noalloc_max_bytes", "maskkv_last_cuda_error",
                        "maskkv_layer_importance_workspace_bytes", "maskkv_mask_project_workspace_bytes"):
            getattr(lib, name).restype = C.c_int
    return lib


lib = _load()


def maskkv_mask_project_workspace_bytes(n_mask: int, width: int) -> int:
    return int(lib.maskkv_mask_project_workspace_bytes(int(n_mask), int(width)))


def status_string(code: int) -> str:
    return lib.maskkv_status_string(code).decode()


def _check(code: int, what: str, handle=None) -> None:
    if code != MASKKV_OK:
        if code == MASKKV_E_CUDA and handle:
            what = f"{what} [{lib.maskkv_last_cuda_error(handle).decode()}]"
        raise MaskKVError(code, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def maskkv_layer_budgets(k_p: int, beta: float, importance: Sequence[float],
                         is_boundary: Optional[Sequence[bool]] = None) -> list:
    """Eq. 9-13 on the host (needs no GPU)."""
    n = len(importance)
    imp = (C.c_double * n)(*[float(x) for x in importance])
    bnd = None if is_boundary is None else (C.c_uint8 * n)(*[1 if b else 0 for b in is_boundary])
    out = (C.c_int32 * n)()
    _check(lib.maskkv_layer_budgets(int(k_p), float(beta), n, imp, bnd, out), "maskkv_layer_budgets")
    return list(out)


class Problem:
    """A descriptor plus the host/device copies of its cumulative-length arrays (kept alive together)."""

    def __init__(self, dtype: torch.dtype, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 prompt_cu: Sequence[int], live_cu: Sequence[int], device, softmax_scale: float = 0.0,
                 q_strides=(0, 0), kv_strides=(0, 0)):
        self.R = len(prompt_cu) - 1
        self.H, self.Hkv, self.d = n_q_heads, n_kv_heads, head_dim
        self.prompt_cu, self.live_cu = [int(x) for x in prompt_cu], [int(x) for x in live_cu]
        self.sumN, self.sumM = self.prompt_cu[-1], self.live_cu[-1]
        self.torch_dtype = dtype
        self.device = torch.device(device)
        self._pcu_host = (C.c_int32 * (self.R + 1))(*self.prompt_cu)
        self._lcu_host = (C.c_int32 * (self.R + 1))(*self.live_cu)
        self._pcu_dev = torch.tensor(self.prompt_cu, dtype=torch.int32, device=self.device)
        self._lcu_dev = torch.tensor(self.live_cu, dtype=torch.int32, device=self.device)
        self.desc = maskkv_desc_t(
            MASKKV_F32 if dtype == torch.float32 else MASKKV_BF16, n_q_heads, n_kv_heads, head_dim, self.R,
            float(softmax_scale), self._pcu_host, self._lcu_host,
            self._pcu_dev.data_ptr(), self._lcu_dev.data_ptr(),
            int(q_strides[0]), int(q_strides[1]), int(kv_strides[0]), int(kv_strides[1]))


class Context:
    """maskkv_ctx handle.  Methods carry the C names and take torch CUDA tensors as raw device memory."""

    def __init__(self, device=0):
        self.device = torch.device("cuda", device if isinstance(device, int) else torch.device(device).index or 0)
        self._h = C.c_void_p()
        _check(lib.maskkv_create(C.byref(self._h), self.device.index), "maskkv_create")

    def close(self):
        if self._h:
            lib.maskkv_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def maskkv_launch_count(self) -> int:
        return int(lib.maskkv_launch_count(self._h))

    def maskkv_tensor_core_launch_count(self) -> int:
        return int(lib.maskkv_tensor_core_launch_count(self._h))

    def maskkv_workspace_bytes(self, p: Problem) -> int:
        return int(lib.maskkv_workspace_bytes(self._h, C.byref(p.desc)))

    def maskkv_selftest_wait_expiry(self):
        """Enqueues a wait that nothing satisfies: it gives up after about a second and raises MASKKV_FLAG_TIMEOUT."""
        _check(lib.maskkv_selftest_wait_expiry(self._h, _stream()), "maskkv_selftest_wait_expiry", self._h)

    def maskkv_selftest_exp_rate(self, iters: int, scratch: torch.Tensor) -> int:
        """Enqueues the exponential-rate measurement kernel; returns the number of exponentials it evaluates."""
        n = C.c_int64(0)
        _check(lib.maskkv_selftest_exp_rate(self._h, int(iters), scratch.data_ptr(), C.byref(n), _stream()),
               "maskkv_selftest_exp_rate", self._h)
        return int(n.value)

    def maskkv_check_status(self) -> int:
        flags = C.c_uint32(0)
        rc = lib.maskkv_check_status(self._h, _stream(), C.byref(flags))
        if rc not in (MASKKV_OK, MASKKV_E_TIMEOUT):
            _check(rc, "maskkv_check_status")
        return int(flags.value)

    def maskkv_layer_importance(self, h_in, h_out, out, workspace=None):
        """Eq. 8 for one layer: h_in, h_out [n_tokens, hidden] (bf16 or fp32, rows may be strided), out a 1-element fp32 tensor."""
        if workspace is None:
            workspace = torch.empty(int(lib.maskkv_layer_importance_workspace_bytes(self._h)), dtype=torch.uint8, device=h_in.device)
        dt = MASKKV_F32 if h_in.dtype == torch.float32 else MASKKV_BF16
        _check(lib.maskkv_layer_importance(self._h, dt, _ptr(h_in), _ptr(h_out), h_in.shape[0], h_in.shape[1], h_in.stride(0),
                                           h_out.stride(0), _ptr(out), _ptr(workspace), workspace.numel(), _stream()),
               "maskkv_layer_importance", self._h)
        return workspace

    def maskkv_refresh_set(self, v_cur, v_prev, delta: float, idx_out, count_out, refresh_all: bool = False, cos_out=None):
        """Response-token refresh rule: v_cur, v_prev [n_tokens, width] (bf16 or fp32, rows may be strided); idx_out int32
        [n_tokens] receives the ascending row numbers with cos < delta (all rows when refresh_all), count_out int32 [1]
        their number, cos_out fp32 [n_tokens] (optional) the cosines."""
        dt = MASKKV_F32 if v_cur.dtype == torch.float32 else MASKKV_BF16
        n, width = (v_cur.shape[0], v_cur.shape[1]) if v_cur.dim() == 2 else (0, 0)
        _check(lib.maskkv_refresh_set(self._h, dt, _ptr(v_cur), _ptr(v_prev), n, width, v_cur.stride(0) if n else 0,
                                      v_prev.stride(0) if n else 0, float(delta), 1 if refresh_all else 0, _ptr(cos_out),
                                      _ptr(idx_out), _ptr(count_out), _stream()), "maskkv_refresh_set", self._h)

    def maskkv_mask_project(self, hidden, w_vocab, logits_out, positions=None, workspace=None):
        """Mask-only projection: logits_out[m] = w_vocab @ hidden[positions[m]] (bf16 operands; logits_out fp32 or bf16
        [n_mask, vocab]).  positions int32 [n_mask] on the device, or None for the first n_mask rows of hidden; workspace
        of maskkv_mask_project_workspace_bytes(n_mask, width) bytes when positions is given."""
        if hidden.dtype != torch.bfloat16 or w_vocab.dtype != torch.bfloat16:
            dt = MASKKV_F32
        else:
            dt = MASKKV_BF16
        n_mask = logits_out.shape[0]
        _check(lib.maskkv_mask_project(self._h, dt, _ptr(hidden), hidden.shape[0], hidden.shape[1], hidden.stride(0),
                                       _ptr(positions), n_mask, _ptr(w_vocab), w_vocab.shape[0], w_vocab.stride(0),
                                       MASKKV_F32 if logits_out.dtype == torch.float32 else MASKKV_BF16, _ptr(logits_out),
                                       logits_out.stride(0) if n_mask else 0, _ptr(workspace),
                                       0 if workspace is None else workspace.numel() * workspace.element_size(), _stream()),
               "maskkv_mask_project", self._h)

    def maskkv_score(self, p: Problem, q_mask, k_prompt, k_mask, scores, mass_p, mass_m, workspace, row_weights=None):
        _check(lib.maskkv_score(self._h, C.byref(p.desc), _ptr(q_mask), _ptr(k_prompt), _ptr(k_mask), _ptr(row_weights),
                                _ptr(scores), _ptr(mass_p), _ptr(mass_m), _ptr(workspace),
                                0 if workspace is None else workspace.numel() * workspace.element_size(), _stream()),
               "maskkv_score", self._h)

    def maskkv_score_all_keys(self, p: Problem, q_mask, k_prompt, k_mask, scores, scores_live, mass_p, mass_m, workspace,
                              row_weights=None):
        """maskkv_score that also returns the column sums over the live keys (scores_live fp32 [H_kv, sum_M]); with the
        voters' queries as q_mask, their keys as k_mask and all other keys as k_prompt this scores any voter set."""
        _check(lib.maskkv_score_all_keys(self._h, C.byref(p.desc), _ptr(q_mask), _ptr(k_prompt), _ptr(k_mask), _ptr(row_weights),
                                         _ptr(scores), _ptr(scores_live), _ptr(mass_p), _ptr(mass_m), _ptr(workspace),
                                         0 if workspace is None else workspace.numel() * workspace.element_size(), _stream()),
               "maskkv_score_all_keys", self._h)

    def maskkv_score_noalloc(self, p: Problem, q_mask, k_prompt, k_mask, scores, mass_p, mass_m, row_weights=None):
        """maskkv_score without a workspace argument, for callers that may not allocate device memory: the
        scratch is an 8 MiB array built into the library (see include/maskkv.h for the limits and the rules on
        the first call and on overlapping calls)."""
        _check(lib.maskkv_score_noalloc(self._h, C.byref(p.desc), _ptr(q_mask), _ptr(k_prompt), _ptr(k_mask),
                                        _ptr(row_weights), _ptr(scores), _ptr(mass_p), _ptr(mass_m), _stream()),
               "maskkv_score_noalloc", self._h)

    def maskkv_budget(self, p: Problem, k_l: int, alpha: float, mass_p, mass_m, capacity: int, budgets, offsets,
                      k_l_per_request=None):
        _check(lib.maskkv_budget(self._h, C.byref(p.desc), int(k_l), _ptr(k_l_per_request), float(alpha), _ptr(mass_p),
                                 _ptr(mass_m), int(capacity), _ptr(budgets), _ptr(offsets), _stream()), "maskkv_budget", self._h)

    def maskkv_select(self, p: Problem, scores, budgets, offsets, kept_idx, workspace=None):
        _check(lib.maskkv_select(self._h, C.byref(p.desc), _ptr(scores), _ptr(budgets), _ptr(offsets), _ptr(kept_idx),
                                 _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                 _stream()), "maskkv_select", self._h)

    def maskkv_compact(self, p: Problem, k_prompt, v_prompt, kept_idx, offsets, capacity: int, kc, vc):
        _check(lib.maskkv_compact(self._h, C.byref(p.desc), _ptr(k_prompt), _ptr(v_prompt), _ptr(kept_idx), _ptr(offsets),
                                  int(capacity), _ptr(kc), _ptr(vc), _stream()), "maskkv_compact", self._h)

    def maskkv_attend(self, p: Problem, q_live, k_live, v_live, kc, vc, offsets, capacity: int, out, lse=None):
        _check(lib.maskkv_attend(self._h, C.byref(p.desc), _ptr(q_live), _ptr(k_live), _ptr(v_live), _ptr(kc), _ptr(vc),
                                 _ptr(offsets), int(capacity), _ptr(out), _ptr(lse), _stream()), "maskkv_attend", self._h)

    def maskkv_attend_rows(self, p: Problem, q_rows, rows_cu: Sequence[int], rows_cu_dev, k_live, v_live, kc, vc, offsets,
                           capacity: int, out_rows, lse_rows=None):
        """maskkv_attend for a subset of query rows (partial refresh): q_rows / out_rows [rows, H, d] hold the refreshed
        rows of every request one after the other; rows_cu (host list, length n_requests + 1) and rows_cu_dev (the same
        numbers as an int32 device tensor, owned by the caller) are their cumulative counts; keys and values remain the
        compacted cache followed by all live rows."""
        host = (C.c_int32 * len(rows_cu))(*[int(x) for x in rows_cu])
        _check(lib.maskkv_attend_rows(self._h, C.byref(p.desc), _ptr(q_rows), host, _ptr(rows_cu_dev), _ptr(k_live), _ptr(v_live),
                                      _ptr(kc), _ptr(vc), _ptr(offsets), int(capacity), _ptr(out_rows), _ptr(lse_rows), _stream()),
               "maskkv_attend_rows", self._h)
