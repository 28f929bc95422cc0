"""The error path of the bounded waits, without faulting or hanging anything: maskkv_selftest_wait_expiry enqueues a
thread that waits for a signal nothing sends.  The wait must run out after about a second, the kernel must return, the
status word must carry the TIMEOUT flag (and maskkv_check_status the matching return code), and the context must go on
working."""
import ctypes
import time

import pytest
import torch

from paper_2510_09309_b200 import synth
from pipeline import LayerRun, to_dev

pytestmark = pytest.mark.gpu


def test_a_lost_signal_ends_in_a_status_word_and_the_context_stays_usable():
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        assert ctx.maskkv_check_status() == 0
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ctx.maskkv_selftest_wait_expiry()
        torch.cuda.synchronize()                                  # returns: the wait is bounded
        waited = time.perf_counter() - t0
        assert 0.5 < waited < 10.0, f"the wait lasted {waited:.2f} s"
        flags = ctypes.c_uint32(0)
        rc = B.lib.maskkv_check_status(ctx._h, None, ctypes.byref(flags))
        assert rc == B.MASKKV_E_TIMEOUT and flags.value == B.MASKKV_FLAG_TIMEOUT
        assert "wait" in B.status_string(rc).lower() or "time" in B.status_string(rc).lower()
        assert ctx.maskkv_check_status() == 0                     # reading the status cleared it
        # the same context runs a layer afterwards, with clean status
        wl = synth.scaled(synth.config(2), "after_expiry", prompt_lens=(900,))
        x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
        xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
        ld = {k: to_dev(v) for k, v in live.items()}
        run = LayerRun(ctx, wl)
        run.score(xd); run.budget(); run.select(); run.compact(xd); run.attend(ld)
        torch.cuda.synchronize()
        assert ctx.maskkv_check_status() == 0
        assert torch.isfinite(run.out.float()).all() and int(run.offsets[-1].item()) > 0
    finally:
        ctx.close()


def test_exp_rate_measurement_counts_its_work_and_rejects_bad_arguments():
    """maskkv_selftest_exp_rate: the count it returns is grid x threads x 32 x iters, a launch of a few thousand rounds
    gives a rate between a half and slightly more than the nominal 16 results per clock per SM, and bad arguments launch
    nothing."""
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(0)
    try:
        scratch = torch.zeros(4, dtype=torch.float32, device=ctx.device)
        sms = torch.cuda.get_device_properties(0).multi_processor_count
        n0 = ctx.maskkv_launch_count()
        assert ctx.maskkv_selftest_exp_rate(10, scratch) == sms * 2 * 1024 * 32 * 10
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best = 0.0
        for _ in range(4):
            e0.record()
            n = ctx.maskkv_selftest_exp_rate(2000, scratch)
            e1.record()
            torch.cuda.synchronize()
            best = max(best, n / (e0.elapsed_time(e1) * 1e-3))
        per_clock_per_sm = best / sms / 1.965e9                    # at the maximum clock: a lower bound of the per-clock rate
        assert 8.0 < per_clock_per_sm < 17.0, per_clock_per_sm
        assert float(scratch.abs().sum()) == 0.0
        n1 = ctx.maskkv_launch_count()
        cnt = ctypes.c_int64(0)
        for iters, ptr in ((0, scratch.data_ptr()), (-3, scratch.data_ptr()), (1 << 21, scratch.data_ptr()), (10, None)):
            assert B.lib.maskkv_selftest_exp_rate(ctx._h, iters, ptr, ctypes.byref(cnt), None) == B.MASKKV_E_INVALID
        assert B.lib.maskkv_selftest_exp_rate(ctx._h, 10, scratch.data_ptr(), None, None) == B.MASKKV_E_INVALID
        assert ctx.maskkv_launch_count() == n1 and n1 == n0 + 5
        assert ctx.maskkv_check_status() == 0
    finally:
        ctx.close()
