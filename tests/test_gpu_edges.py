"""GPU edge cases of the C ABI: degenerate segments, clamps, capacity clipping, ties, special values,
strided inputs and argument validation (a failed validation must launch nothing)."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import maskkv_oracle as O
from paper_2510_09309_b200 import synth
from pipeline import ATTEND_ATOL, LayerRun, assert_scores_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2510_09309_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def _problem(ctx, dtype, H, Hkv, d, lens, M):
    from paper_2510_09309_b200 import binding as B
    pcu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    lcu = [r * M for r in range(len(lens) + 1)]
    return B.Problem(dtype, H, Hkv, d, pcu, lcu, ctx.device), pcu, lcu


def test_select_ties_duplicates_and_special_values(ctx):
    p, pcu, _ = _problem(ctx, torch.bfloat16, 3, 3, 64, [10, 6, 5, 40000], 4)
    sc = np.zeros((3, pcu[-1]), np.float32)
    sc[0, 0:10] = 1.0                                   # all equal -> lowest indices
    sc[0, 10:16] = [5, 1, 5, 5, 0, 5]                   # duplicates straddling the cut
    sc[0, 16:21] = [np.nan, 1, -np.inf, 2, np.nan]      # NaN below every number
    rng = np.random.default_rng(0)
    sc[0, 21:] = rng.integers(0, 50, 40000) / 7.0       # long segment (beyond the shared-memory cache) with many ties
    sc[1] = rng.standard_normal(pcu[-1])                # negative values and zeros
    sc[1, 3] = 0.0; sc[1, 4] = -0.0
    sc[2] = rng.random(pcu[-1])
    bud = np.array([[4, 10, 0], [2, 5, 6], [3, 4, 5], [20000, 1, 39999]], np.int32)
    idx, off = O.select(sc, bud, pcu)
    kept = torch.full((int(off[-1]) + 8,), -1, dtype=torch.int32, device=ctx.device)
    ctx.maskkv_select(p, to_dev(sc), to_dev(bud), to_dev(off), kept)
    torch.cuda.synchronize()
    assert np.array_equal(kept[:int(off[-1])].cpu().numpy(), idx)
    assert (kept[int(off[-1]):] == -1).all()
    assert ctx.maskkv_check_status() == 0


def test_budget_clamp_capacity_and_per_request_k(ctx):
    from paper_2510_09309_b200 import binding as B
    p, pcu, _ = _problem(ctx, torch.bfloat16, 2, 2, 64, [1000, 40, 1000], 4)
    mp = np.array([[3, 1], [1, 1], [2, 2]], np.float32); mm = np.array([[1, 3], [1, 1], [2, 2]], np.float32)
    kl = np.array([100, 50, 10], np.int32)
    bud = torch.zeros((3, 2), dtype=torch.int32, device=ctx.device); off = torch.zeros(7, dtype=torch.int32, device=ctx.device)
    for cap in (10 ** 6, 215, 0):
        ctx.maskkv_budget(p, 0, 0.0, to_dev(mp), to_dev(mm), cap, bud, off, k_l_per_request=to_dev(kl))
        torch.cuda.synchronize()
        rb, ro = O.head_budgets(mp, mm, kl, 0.0, [1000, 40, 1000], capacity=cap)
        assert np.array_equal(bud.cpu().numpy(), rb) and np.array_equal(off.cpu().numpy(), ro)
        flags = ctx.maskkv_check_status()
        assert bool(flags & B.MASKKV_FLAG_CAPACITY) == (cap < 290)
    # golden fixtures through the device kernel
    from golden_io import head_budget_cases
    for c in head_budget_cases():
        Hkv = len(c["expected"])
        pp, _, _ = _problem(ctx, torch.bfloat16, Hkv, Hkv, 64, [c["n"]], 4)
        b = torch.zeros((1, Hkv), dtype=torch.int32, device=ctx.device); o = torch.zeros(Hkv + 1, dtype=torch.int32, device=ctx.device)
        mp32 = np.array([c["mass_p"]], np.float32); mm32 = np.array([c["mass_m"]], np.float32)
        ctx.maskkv_budget(pp, c["k_l"], c["alpha"], to_dev(mp32), to_dev(mm32), 10 ** 6, b, o)
        torch.cuda.synchronize()
        rb, _ = O.head_budgets(mp32, mm32, c["k_l"], c["alpha"], [c["n"]])
        assert np.array_equal(b.cpu().numpy(), rb)


def test_budget_random_bit_exact(ctx):
    rng = np.random.default_rng(5)
    for trial in range(20):
        R, Hkv = int(rng.integers(1, 9)), int(rng.choice([1, 4, 8, 32]))
        lens = rng.integers(1, 5000, R).tolist()
        p, _, _ = _problem(ctx, torch.bfloat16, Hkv, Hkv, 128, lens, 8)
        mp = rng.uniform(0.01, 300, (R, Hkv)).astype(np.float32); mm = rng.uniform(0.01, 300, (R, Hkv)).astype(np.float32)
        k_l, alpha = int(rng.integers(0, 3000)), float(rng.choice([0.0, 0.1, 0.37, 1.0]))
        b = torch.zeros((R, Hkv), dtype=torch.int32, device=ctx.device); o = torch.zeros(R * Hkv + 1, dtype=torch.int32, device=ctx.device)
        ctx.maskkv_budget(p, k_l, alpha, to_dev(mp), to_dev(mm), 2 ** 31 - 1, b, o)
        torch.cuda.synchronize()
        rb, ro = O.head_budgets(mp, mm, k_l, alpha, lens)
        assert np.array_equal(b.cpu().numpy(), rb) and np.array_equal(o.cpu().numpy(), ro)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_empty_and_degenerate_segments(ctx, dtype):
    """Zero budgets (attend sees only live keys), one-token prompts, a request with one mask row."""
    wl = synth.scaled(synth.config(2), "degenerate", dtype=dtype, prompt_lens=(1, 257, 31), n_mask=5, n_q_heads=4,
                      n_kv_heads=2, head_dim=64, mean_budget=0)
    x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}; ld = {k: to_dev(v) for k, v in live.items()}
    for k_l in (0, 1, 300):
        run = LayerRun(ctx, wl, capacity=2000, k_l=k_l)
        run.score(xd); run.budget(alpha=1.0); run.select(); run.compact(xd); run.attend(ld)
        torch.cuda.synchronize()
        sc, mp, mm = O.score(x["q_mask"], x["k_prompt"], x["k_mask"], wl.prompt_cu(), wl.live_cu())
        assert_scores_close(run.scores.cpu().numpy(), sc)
        bud, off = O.head_budgets(mp.astype(np.float32), mm.astype(np.float32), k_l, 1.0, wl.prompt_lens)
        assert np.array_equal(run.budgets.cpu().numpy(), bud)
        kept = run.kept.cpu().numpy(); offd = run.offsets.cpu().numpy()
        kc, vc = O.compact(x["k_prompt"], x["v_prompt"], kept, offd, wl.prompt_cu())
        out, _ = O.attend(live["q_live"], live["k_live"], live["v_live"], kc, vc, offd, wl.live_cu(), wl.n_kv_heads)
        err = np.abs(run.out.float().cpu().numpy() - out).max()
        assert err <= ATTEND_ATOL[dtype]
    assert ctx.maskkv_check_status() == 0


def test_strided_inputs(ctx):
    """Q/K/V taken as views of a fused [tokens, (H + 2 H_kv), d] projection output: non-packed strides."""
    from paper_2510_09309_b200 import binding as B
    wl = synth.scaled(synth.config(2), "strided", prompt_lens=(300,), n_mask=64, n_q_heads=4, n_kv_heads=2, mean_budget=32)
    x = synth.layer_inputs(wl, 0, "cpu")
    H, Hkv, d, N, M = 4, 2, 128, 300, 64
    fused_p = torch.zeros(N, H + 2 * Hkv, d, dtype=torch.bfloat16); fused_m = torch.zeros(M, H + 2 * Hkv, d, dtype=torch.bfloat16)
    fused_p[:, H:H + Hkv] = x["k_prompt"]; fused_m[:, :H] = x["q_mask"]; fused_m[:, H:H + Hkv] = x["k_mask"]
    fp, fm = to_dev(fused_p), to_dev(fused_m)
    ts = (H + 2 * Hkv) * d
    p = B.Problem(torch.bfloat16, H, Hkv, d, [0, N], [0, M], ctx.device, q_strides=(ts, d), kv_strides=(ts, d))
    scores = torch.zeros((Hkv, N), dtype=torch.float32, device=ctx.device)
    mp = torch.zeros((1, Hkv), dtype=torch.float32, device=ctx.device); mm = torch.zeros_like(mp)
    ws = torch.empty(ctx.maskkv_workspace_bytes(p), dtype=torch.uint8, device=ctx.device)
    ctx.maskkv_score(p, fm, fp[:, H:], fm[:, H:], scores, mp, mm, ws)
    torch.cuda.synchronize()
    sc, _, _ = O.score(x["q_mask"], x["k_prompt"], x["k_mask"], [0, N], [0, M])
    assert_scores_close(scores.cpu().numpy(), sc)


def test_validation_launches_nothing(ctx):
    from paper_2510_09309_b200 import binding as B
    p, _, _ = _problem(ctx, torch.bfloat16, 4, 2, 128, [64], 8)
    good = torch.zeros(64 * 2 * 128 + 64, dtype=torch.bfloat16, device=ctx.device)
    f = torch.zeros(4096, dtype=torch.float32, device=ctx.device)
    ws = torch.empty(max(ctx.maskkv_workspace_bytes(p), 16), dtype=torch.uint8, device=ctx.device)

    def score_rc(desc, q, k, km, sc, ws_t, ws_bytes):
        return B.lib.maskkv_score(ctx._h, ctypes.byref(desc), q, k, km, None, sc, f.data_ptr(), f.data_ptr(), ws_t, ws_bytes, None)

    ok = (good.data_ptr(), good.data_ptr(), good.data_ptr(), f.data_ptr(), ws.data_ptr(), ws.numel())
    assert score_rc(p.desc, ok[0] + 2, *ok[1:]) == B.MASKKV_E_ALIGN
    assert score_rc(p.desc, None, *ok[1:]) == B.MASKKV_E_INVALID
    assert score_rc(p.desc, *ok[:4], ws.data_ptr(), 8) == B.MASKKV_E_WORKSPACE
    assert score_rc(p.desc, *ok[:4], None, 0) == B.MASKKV_E_WORKSPACE
    for field, val, code in (("head_dim", 96, B.MASKKV_E_UNSUPPORTED), ("dtype", 7, B.MASKKV_E_UNSUPPORTED),
                             ("n_kv_heads", 3, B.MASKKV_E_INVALID), ("n_requests", 0, B.MASKKV_E_INVALID),
                             ("kv_token_stride", 100, B.MASKKV_E_ALIGN)):
        q, _, _ = _problem(ctx, torch.bfloat16, 4, 2, 128, [64], 8)
        setattr(q.desc, field, val)
        assert score_rc(q.desc, *ok) == code, field
    assert B.lib.maskkv_budget(ctx._h, ctypes.byref(p.desc), 10, None, 1.5, f.data_ptr(), f.data_ptr(), 10, f.data_ptr(), f.data_ptr(), None) == B.MASKKV_E_INVALID
    assert B.lib.maskkv_budget(ctx._h, ctypes.byref(p.desc), -1, None, 0.5, f.data_ptr(), f.data_ptr(), 10, f.data_ptr(), f.data_ptr(), None) == B.MASKKV_E_INVALID
    assert B.lib.maskkv_select(ctx._h, ctypes.byref(p.desc), None, f.data_ptr(), f.data_ptr(), f.data_ptr(), None, 0, None) == B.MASKKV_E_INVALID
    assert B.lib.maskkv_attend(None, ctypes.byref(p.desc), *([f.data_ptr()] * 6), 16, f.data_ptr(), f.data_ptr(), None) == B.MASKKV_E_INVALID
    torch.cuda.synchronize()
    assert (f == 0).all() and ctx.maskkv_check_status() == 0


@pytest.mark.parametrize("d,n_mask", [(128, 256), (64, 130)])
def test_attend_long_segments_shared_by_two_ctas(ctx, d, n_mask):
    """Few (query tile, head) units with long kept segments: two CTAs of a cluster split the key tiles of a unit and
    merge their partial softmax through distributed shared memory.  Uneven shares, ragged tails and segments of very
    different length (one of them empty) included."""
    wl = synth.scaled(synth.config(2), "long_segments", dtype="bf16", prompt_lens=(4096,), n_mask=n_mask, n_q_heads=4,
                      n_kv_heads=4, head_dim=d, mean_budget=1536)
    x = synth.layer_inputs(wl, 0, "cpu"); live = synth.live_inputs(wl, 0, 0, "cpu")
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}; ld = {k: to_dev(v) for k, v in live.items()}
    run = LayerRun(ctx, wl, capacity=4 * 1536, k_l=1536)
    budgets = torch.tensor([[1536, 0, 2999, 1609]], dtype=torch.int32)      # 12 / 0 / 24 / 13 key tiles + the live ones
    offsets = torch.tensor([0, 1536, 1536, 4535, 6144], dtype=torch.int32)
    run.score(xd)
    run.select(budgets=to_dev(budgets), offsets=to_dev(offsets)); run.compact(xd, offsets=to_dev(offsets))
    run.attend(ld, offsets=to_dev(offsets))
    torch.cuda.synchronize()
    kept = run.kept.cpu().numpy(); offd = offsets.numpy()
    kc, vc = O.compact(x["k_prompt"], x["v_prompt"], kept, offd, wl.prompt_cu())
    assert torch.equal(run.kc.cpu(), kc)
    out, lse = O.attend(live["q_live"], live["k_live"], live["v_live"], kc, vc, offd, wl.live_cu(), wl.n_kv_heads)
    assert np.abs(run.out.float().cpu().numpy() - out).max() <= ATTEND_ATOL["bf16"]
    assert np.abs(run.lse.cpu().numpy() - lse).max() <= 1e-3
    assert ctx.maskkv_check_status() == 0


def test_compact_reads_prompt_values_from_pinned_host_memory(ctx):
    """maskkv_compact is the path's only reader of v_prompt: a caller may leave the prompt values in pinned
    (device-mapped) host memory and pass that pointer; only the kept rows cross the bus."""
    wl = synth.scaled(synth.config(2), "host_values", dtype="bf16", prompt_lens=(3000, 700), n_mask=64, n_q_heads=4,
                      n_kv_heads=4, head_dim=128, mean_budget=200)
    x = synth.layer_inputs(wl, 0, "cpu")
    xd = {k: to_dev(v) for k, v in x.items() if torch.is_tensor(v)}
    run = LayerRun(ctx, wl)
    run.score(xd); run.budget(); run.select(); run.compact(xd)
    torch.cuda.synchronize()
    kc_dev, vc_dev = run.kc.clone(), run.vc.clone()
    run.kc.zero_(); run.vc.zero_()
    host = dict(xd)
    host["v_prompt"] = x["v_prompt"].to(wl.torch_dtype).pin_memory()          # stays on the host
    host["k_prompt"] = x["k_prompt"].to(wl.torch_dtype).pin_memory()
    run.compact(host)
    torch.cuda.synchronize()
    assert torch.equal(run.kc, kc_dev) and torch.equal(run.vc, vc_dev)
    assert ctx.maskkv_check_status() == 0


def test_select_in_registers_crowded_threshold_bin_and_ties(ctx):
    """Segments of at most 32768 keys take the register-resident cluster kernel.  Cases: most keys inside one bin of the
    first radix digit with the cut inside that bin (the candidate lists do not fit one CTA: digits are then found with
    cluster-summed histograms), the same with exact ties at the cut, a short candidate list (ranked by counting), NaNs,
    and tiny segments next to full ones."""
    lens = [32768, 30001, 7, 32768]
    p, pcu, _ = _problem(ctx, torch.bfloat16, 2, 2, 64, lens, 4)
    rng = np.random.default_rng(11)
    sc = rng.random((2, pcu[-1])).astype(np.float32) * 8.0                  # spread over several octaves
    # request 0, head 0: 24000 keys packed into [1.5, 1.5 + 2^-11) (one bin of the first digit), random low bits
    crowd = (1.5 + rng.integers(0, 1 << 12, 24000) * 2.0 ** -23).astype(np.float32)
    pos = rng.permutation(32768)[:24000]
    sc[0, pos] = crowd
    # request 0, head 1: the same crowd collapsed onto four values (thousands of exact ties at the cut)
    sc[1, pos] = (1.5 + rng.integers(0, 4, 24000) * 2.0 ** -23).astype(np.float32)
    # request 1: ordinary scores with a few NaNs and infinities
    a = pcu[1]
    sc[0, a + 5] = np.nan; sc[0, a + 17] = np.inf; sc[1, a + 3] = -np.inf; sc[1, a + 9] = np.nan
    bud = np.array([[15000, 15000], [300, 29999], [3, 7], [1, 32768]], np.int32)
    idx, off = O.select(sc, bud, pcu)
    kept = torch.full((int(off[-1]) + 8,), -1, dtype=torch.int32, device=ctx.device)
    ctx.maskkv_select(p, to_dev(sc), to_dev(bud), to_dev(off), kept)
    torch.cuda.synchronize()
    assert np.array_equal(kept[:int(off[-1])].cpu().numpy(), idx)
    assert (kept[int(off[-1]):] == -1).all()
    assert ctx.maskkv_check_status() == 0


@pytest.mark.parametrize("force", ["2", "4", "8", "128", "384"])
def test_both_select_kernels_on_crowded_bins_ties_and_ragged_batches(force, monkeypatch):
    """The selection runs on clusters (few segments), on one CTA per segment (batches; keys in registers, or staged in
    shared memory for segments beyond 32768 scores) or on persistent CTAs that copy the next segment's scores to shared
    memory while they work (more segments than SMs); bits 1 / 2 / 3 / 7 of MASKKV_KERNEL_CHOICE pin the choice, bit 8
    puts the persistent kernel on three CTAs so that each walks many segments.  All must reproduce the oracle exactly on
    the crowded-bin / tie / NaN case above and on a ragged batch of 100 segments (starts at every offset from a 16-byte
    boundary) with budgets from 0 to everything."""
    from paper_2510_09309_b200 import binding as B
    monkeypatch.setenv("MASKKV_KERNEL_CHOICE", force)
    c = B.Context(0)
    try:
        test_select_in_registers_crowded_threshold_bin_and_ties(c)
        rng = np.random.default_rng(int(force))
        lens = [int(x) for x in rng.integers(1, 9000, 25)]
        p, pcu, _ = _problem(c, torch.bfloat16, 4, 4, 64, lens, 4)
        sc = np.exp(rng.standard_normal((4, pcu[-1]))).astype(np.float32)
        sc[:, ::7] = np.float32(0.5)                                                   # ties everywhere
        bud = np.stack([rng.integers(0, n + 1, 4) for n in lens]).astype(np.int32)
        bud[3] = 0; bud[5] = lens[5]
        idx, off = O.select(sc, bud, pcu)
        kept = torch.full((int(off[-1]) + 8,), -1, dtype=torch.int32, device=c.device)
        c.maskkv_select(p, to_dev(sc), to_dev(bud), to_dev(off), kept)
        torch.cuda.synchronize()
        assert np.array_equal(kept[:int(off[-1])].cpu().numpy(), idx)
        assert (kept[int(off[-1]):] == -1).all()
        assert c.maskkv_check_status() == 0
    finally:
        c.close()


@pytest.mark.parametrize("segments", [8, 48])
def test_cluster_select_when_every_key_of_a_segment_is_equal(segments, monkeypatch):
    """All scores of a segment equal (zeros, or all NaN) with 0 < k < N: the keys share all 32 bits, so the cluster
    kernel skips every radix pass and goes straight from the exchange of the common prefix to the exchange of the
    threshold counts.  The kept set is the k lowest indices.  Repeated, on the one-wave variant (8 segments) and the
    two-CTAs-per-SM variant (48 segments), with the cluster kernel pinned."""
    from paper_2510_09309_b200 import binding as B
    monkeypatch.setenv("MASKKV_KERNEL_CHOICE", "4")
    c = B.Context(0)
    try:
        rng = np.random.default_rng(segments)
        heads = 4
        lens = [int(x) for x in rng.integers(200, 32769, segments // heads)]
        lens[0] = 32768
        p, pcu, _ = _problem(c, torch.bfloat16, heads, heads, 64, lens, 4)
        sc = np.zeros((heads, pcu[-1]), np.float32)
        sc[1::2] = np.float32("nan")                                               # odd heads: all NaN
        bud = np.stack([rng.integers(1, n, heads) for n in lens]).astype(np.int32)
        idx, off = O.select(sc, bud, pcu)
        for r in range(len(lens)):
            for h in range(heads):
                s0 = r * heads + h
                assert np.array_equal(idx[off[s0]:off[s0 + 1]], np.arange(bud[r, h]))
        scd, budd, offd = to_dev(sc), to_dev(bud), to_dev(off)
        kept = torch.empty((int(off[-1]),), dtype=torch.int32, device=c.device)
        ref = torch.from_numpy(idx).to(c.device)
        for it in range(300):
            kept.fill_(-1)
            c.maskkv_select(p, scd, budd, offd, kept)
            assert torch.equal(kept, ref), f"repeat {it}"
        assert c.maskkv_check_status() == 0
    finally:
        c.close()


def test_attend_fp32_offsets_beyond_capacity_are_clipped_and_flagged(ctx):
    """The FP32-pipe attention is told how many rows the cache holds: offsets that point past them (a caller's mistake)
    must raise MASKKV_FLAG_BOUNDS and must not be followed.  The rows behind the declared capacity hold NaN here, so a
    read past it would show in the output."""
    from paper_2510_09309_b200 import binding as B
    wl = synth.scaled(synth.config(1), "cap_clip", prompt_lens=(64,), n_mask=16, n_q_heads=2, n_kv_heads=2, mean_budget=8)
    live = {k: to_dev(v) for k, v in synth.live_inputs(wl, 0, 0, "cpu").items()}
    p = B.Problem(wl.torch_dtype, 2, 2, wl.head_dim, wl.prompt_cu(), wl.live_cu(), ctx.device)
    capacity = 12
    store_k = torch.full((40, wl.head_dim), float("nan"), dtype=torch.float32, device=ctx.device)
    store_v = torch.full((40, wl.head_dim), float("nan"), dtype=torch.float32, device=ctx.device)
    store_k[:capacity] = torch.randn(capacity, wl.head_dim, device=ctx.device)
    store_v[:capacity] = torch.randn(capacity, wl.head_dim, device=ctx.device)
    offsets = to_dev(np.array([0, 8, 30], np.int32))            # the second segment claims rows 8..29 of a 12-row cache
    out = torch.zeros((16, 2, wl.head_dim), dtype=torch.float32, device=ctx.device)
    lse = torch.zeros((2, 16), dtype=torch.float32, device=ctx.device)
    assert ctx.maskkv_check_status() == 0
    ctx.maskkv_attend(p, live["q_live"], live["k_live"], live["v_live"], store_k, store_v, offsets, capacity, out, lse)
    torch.cuda.synchronize()
    assert ctx.maskkv_check_status() & B.MASKKV_FLAG_BOUNDS
    assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    # the clipped segment is rows 8..11: the oracle on that cache gives the same numbers
    ref, _ = O.attend(live["q_live"].cpu(), live["k_live"].cpu(), live["v_live"].cpu(), store_k[:capacity].cpu(),
                      store_v[:capacity].cpu(), np.array([0, 8, 12], np.int32), wl.live_cu(), 2)
    assert np.abs(out.cpu().numpy() - ref).max() <= 1e-5


def test_select_more_segments_than_sms(ctx):
    """160 full segments of 32768 scores plus a ragged tail of requests: more segments than SMs, so the launch takes the
    persistent kernel by itself and every CTA walks at least two segments.  Bit-exact against the oracle, twice."""
    rng = np.random.default_rng(160)
    heads = 4
    lens = [32768] * 40 + [int(x) for x in rng.integers(1, 32769, 6)]
    p, pcu, _ = _problem(ctx, torch.bfloat16, heads, heads, 64, lens, 4)
    sc = (rng.random((heads, pcu[-1]), dtype=np.float32) * np.float32(1e-3)).astype(np.float32)
    sc[:, ::11] = np.float32(2.5e-4)                                                    # ties at a common value
    bud = np.stack([rng.integers(0, min(n, 1024) + 1, heads) for n in lens]).astype(np.int32)
    bud[1, 0] = lens[1]; bud[2, 1] = 0
    idx, off = O.select(sc, bud, pcu)
    scd, budd, offd = to_dev(sc), to_dev(bud), to_dev(off)
    kept = torch.empty((int(off[-1]) + 8,), dtype=torch.int32, device=ctx.device)
    for _ in range(2):
        kept.fill_(-1)
        ctx.maskkv_select(p, scd, budd, offd, kept)
        torch.cuda.synchronize()
        assert np.array_equal(kept[:int(off[-1])].cpu().numpy(), idx)
        assert (kept[int(off[-1]):] == -1).all()
    assert ctx.maskkv_check_status() == 0


@pytest.mark.parametrize("force", ["0", "128"])
def test_select_short_cut_and_its_fallbacks_on_awkward_score_distributions(force, monkeypatch):
    """The register-resident selection takes a sampled short cut when it can and the full search when it cannot; either
    way the kept set is the oracle's, bit for bit.  Distributions chosen to hit every exit: sorted ascending and
    descending scores (the one-key-per-thread sample is then as unrepresentative as it gets), a plateau of equal scores
    straddling the cut, all but a handful of scores equal, two far-apart clusters, one negative score, one -0, one NaN
    and one +inf hidden among positive scores, budgets from 1 to most of the segment, full and ragged lengths.  With
    MASKKV_KERNEL_CHOICE=128 the same runs through the persistent kernel (bulk-copied scores, segment starts at every
    offset from a 16-byte boundary)."""
    from paper_2510_09309_b200 import binding as B
    monkeypatch.setenv("MASKKV_KERNEL_CHOICE", force)
    c = B.Context(0)
    try:
        rng = np.random.default_rng(77)
        lens = [32768, 32768, 32767, 20001, 9000, 32768, 4097, 32768, 12345, 32768, 32768, 31000]
        heads = 2
        p, pcu, _ = _problem(c, torch.bfloat16, heads, heads, 64, lens, 4)
        sc = np.empty((heads, pcu[-1]), np.float32)
        bud = np.empty((len(lens), heads), np.int32)
        for r, n in enumerate(lens):
            seg = slice(pcu[r], pcu[r + 1])
            base = (rng.random(n) ** 6).astype(np.float32) * np.float32(1e-2)
            variants = [
                np.sort(base), np.sort(base)[::-1].copy(),                                  # 0, 1: sorted both ways
                np.where(np.arange(n) % 3 == 0, np.float32(5e-3), base),                      # 2: plateau of ties
                np.where(rng.random(n) < 2e-3, base + 1, np.float32(1e-4)).astype(np.float32),  # 3: nearly all equal
                np.where(rng.random(n) < 0.5, base, base + np.float32(100)).astype(np.float32),  # 4: two clusters
                base.copy(), base.copy(), base.copy(), base.copy(),                           # 5-8: one special value each
                base.copy(), np.full(n, np.float32(0.25)), base.copy(),                       # 9: plain, 10: all equal, 11: plain
            ]
            variants[5][n // 2] = np.float32(-1e-3)
            variants[6][n // 3] = np.float32(-0.0)
            variants[7][n - 5] = np.float32("nan")
            variants[8][7] = np.float32("inf")
            for h in range(heads):
                sc[h, seg] = variants[r] if h == 0 else variants[(r + 5) % len(variants)]
            bud[r] = [[1, 300], [256, 2900], [700, 64], [5, 1500], [n // 2, 17], [256, 256], [4000, 9], [512, 33],
                      [100, n - 1], [3100, 129], [777, 1], [n - 3, 450]][r]
        idx, off = O.select(sc, bud, pcu)
        scd, budd, offd = to_dev(sc), to_dev(bud), to_dev(off)
        kept = torch.empty((int(off[-1]) + 8,), dtype=torch.int32, device=c.device)
        for _ in range(2):
            kept.fill_(-1)
            c.maskkv_select(p, scd, budd, offd, kept)
            torch.cuda.synchronize()
            got = kept[:int(off[-1])].cpu().numpy()
            for s0 in range(len(lens) * heads):
                assert np.array_equal(got[off[s0]:off[s0 + 1]], idx[off[s0]:off[s0 + 1]]), f"segment {s0}"
            assert (kept[int(off[-1]):] == -1).all()
        assert c.maskkv_check_status() == 0
    finally:
        c.close()
