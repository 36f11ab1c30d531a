"""GPU parity: the CUDA library, called through its C ABI, against the float64 CPU oracle on
the same seeded inputs.  Scores/statistics within 1e-3 relative, decisions bit-exact."""
import numpy as np
import pytest
import torch

from helpers import (UNIT_BITS, assert_scores_close, assert_stats_close, near_threshold,
                     oracle_to_blob, parse_blob)
from paper_2603_03592_b200 import synth

pytestmark = pytest.mark.gpu
ACT, GRAD = 0, 1


@pytest.fixture(scope="module")
def sb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_03592_b200 import binding
    binding.lib()                      # a missing library is an error, never a fallback
    return binding


def dev(a, dtype):
    return torch.as_tensor(np.ascontiguousarray(a)).to(dtype).cuda()


def run_distance(sb, x_bf16, m_f32):
    B = x_bf16.shape[0]
    scores = torch.empty(1 + B, 3, dtype=torch.float32, device="cuda")
    stats = torch.empty(1 + B, 8, dtype=torch.float32, device="cuda")
    sb.sentinel_distance(x_bf16, m_f32, scores, stats)
    torch.cuda.synchronize()
    return scores.cpu().numpy(), stats.cpu().numpy()


def oracle_distance_all(oracle_mod, xb, m64):
    B = xb.shape[0]
    g = np.empty((1 + B, 3))
    s = np.empty((1 + B, 8))
    g[0], s[0], _ = oracle_mod.distance(xb, m64)
    for b in range(B):
        g[1 + b], s[1 + b], _ = oracle_mod.distance(xb[b], m64[b])
    return g, s


SHAPES = [(1, 1, 8), (2, 3, 8), (1, 7, 16), (3, 5, 520), (4, 33, 1024), (8, 128, 512),
          (2, 19, 4104), (5, 64, 2048), (64, 2, 64), (3, 1, 8192), (2, 300, 136),
          (1, 2, 65536), (2, 5000, 8), (64, 1, 8)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_distance_matches_oracle_over_shapes(sb, oracle_mod, shape):
    """Stateless Omega_i(x, m): tiny, ragged (d not a multiple of the warp tile), multi-tile."""
    B, T, d = shape
    g = torch.Generator(device="cuda").manual_seed(1000 + B * 7 + T * 13 + d)
    x = (torch.randn(B, T, d, generator=g, device="cuda") * 1.7 + 0.3).to(torch.bfloat16)
    m = (0.6 * x.float() + 0.8 * torch.randn(B, T, d, generator=g, device="cuda")).contiguous()
    scores, stats = run_distance(sb, x, m)
    ref_g, ref_s = oracle_distance_all(oracle_mod, synth.bits(x), m.double().cpu().numpy())
    scale = float(x.float().abs().mean())
    assert_scores_close(scores, ref_g, scale, str(shape))
    assert_stats_close(stats, ref_s, float(x.float().std()) if x.numel() > 1 else scale,
                       float(m.std()) if m.numel() > 1 else scale, str(shape))


def test_distance_degenerate_inputs(sb, oracle_mod):
    B, T, d = 3, 9, 264
    g = torch.Generator(device="cuda").manual_seed(5)
    rnd = torch.randn(B, T, d, generator=g, device="cuda")
    cases = {
        "zero_reference": (rnd.to(torch.bfloat16), torch.zeros(B, T, d, device="cuda")),
        "constant_x": (torch.full((B, T, d), -1.0, device="cuda").to(torch.bfloat16), rnd.clone()),
        "constant_both": (torch.full((B, T, d), 2.0, device="cuda").to(torch.bfloat16),
                          torch.full((B, T, d), 0.03, device="cuda")),
        "all_zero": (torch.zeros(B, T, d, device="cuda").to(torch.bfloat16), torch.zeros(B, T, d, device="cuda")),
        "identical": (rnd.to(torch.bfloat16), rnd.to(torch.bfloat16).float()),
        "large_mean": ((rnd * 0.5 + 40.0).to(torch.bfloat16), rnd * 0.5 + 40.0),
    }
    xz = rnd.clone()
    xz[:, ::3] = 0.0
    xz[:, 1::5] = -0.0
    cases["signed_zeros"] = (xz.to(torch.bfloat16), torch.zeros(B, T, d, device="cuda"))
    one_const = rnd.clone()
    one_const[1] = 0.75                              # one sample constant, the tensor is not
    cases["one_constant_sample"] = (one_const.to(torch.bfloat16), rnd * 0.1)
    for name, (x, m) in cases.items():
        scores, stats = run_distance(sb, x, m.contiguous())
        ref_g, ref_s = oracle_distance_all(oracle_mod, synth.bits(x), m.double().cpu().numpy())
        scale = max(float(x.float().abs().mean()), 1e-3)
        assert_scores_close(scores, ref_g, scale, name)
        assert_stats_close(stats, ref_s, max(float(x.float().std()), 1e-3), max(float(m.std()), 1e-3), name)
        if name in ("constant_x", "constant_both", "all_zero"):
            assert np.all(stats[:, 1] == 0.0), name          # variance of a constant: exactly 0
        if name == "one_constant_sample":
            assert stats[2, 1] == 0.0 and scores[2, 1] == pytest.approx(1.0, rel=1e-6)
        if name == "signed_zeros":
            assert scores[0, 2] == pytest.approx(np.count_nonzero(x.float().cpu().numpy()) / x.numel(), rel=1e-6)


def test_distance_non_finite_units(sb, oracle_mod):
    B, T, d = 4, 6, 128
    g = torch.Generator(device="cuda").manual_seed(6)
    x = torch.randn(B, T, d, generator=g, device="cuda")
    x[1, 2, 77] = float("inf")
    x[3, 5, 127] = float("nan")
    x = x.to(torch.bfloat16)
    m = torch.randn(B, T, d, generator=g, device="cuda")
    scores, stats = run_distance(sb, x, m)
    ref_g, _ = oracle_distance_all(oracle_mod, synth.bits(x), m.double().cpu().numpy())
    assert np.all(np.isnan(scores[[0, 2, 4]])) and np.all(np.isnan(stats[[0, 2, 4]]))
    assert_scores_close(scores, ref_g, 0.8, "nonfinite")


def test_scaling_and_permutation_invariants_on_gpu(sb):
    B, T, d = 2, 64, 256
    g = torch.Generator(device="cuda").manual_seed(7)
    x = torch.randn(B, T, d, generator=g, device="cuda").to(torch.bfloat16)
    m = torch.randn(B, T, d, generator=g, device="cuda")
    s1, t1 = run_distance(sb, x, m)
    s8, t8 = run_distance(sb, (x.float() * -8).to(torch.bfloat16), m)
    assert t8[:, 2] == pytest.approx(8 * t1[:, 2], rel=1e-6)         # norm scales by |c|
    assert t8[:, 1] == pytest.approx(64 * t1[:, 1], rel=1e-5)        # variance by c^2
    perm = torch.randperm(T, generator=g, device="cuda")
    sp, tp = run_distance(sb, x[:, perm].contiguous(), m[:, perm].contiguous())
    assert sp == pytest.approx(s1, rel=1e-5)
    assert tp[:, :3] == pytest.approx(t1[:, :3], rel=1e-5, abs=1e-7)


# ---------------------------------------------------------------------------------------------
# stateful path

def make_pair(sb, oracle_mod, w, **kw):
    okw = dict(kw)
    gkw = {}
    names = {"l": "window_steps", "c": "ban_violations", "t_forgiveness": "forgiveness_steps",
             "gamma_g": "gamma_grow", "gamma_s": "gamma_shrink", "lam": "lambda_min", "eps": "iqr_eps"}
    for k, v in kw.items():
        gkw[names.get(k, k)] = v
    gv = sb.Verifier(w.B, w.T, w.d, **gkw)
    params = oracle_mod.Params(B=w.B, T=w.T, d=w.d, **okw)
    return gv, oracle_mod.Verifier(params), params


def compare_thresholds(gv, ov, kind, rel=1e-3):
    """The multiplier k moves by whole factors, so it must agree to rounding; quartiles and
    bounds are functions of scores that agree to 1e-3, and tau = q2 -+ k*IQR can cancel, so
    they are compared on the scale of the median."""
    gt, gvalid = gv.sentinel_get_thresholds(kind)
    ot, ovalid = ov.thresholds(kind)
    assert np.array_equal(gvalid, ovalid)
    for L in range(2):
        for i in range(ovalid.shape[1]):
            if ovalid[L, i]:
                assert gt[L, i, 3] == pytest.approx(ot[L, i, 3], rel=1e-12), "multiplier k"
                tol = rel * np.maximum(np.abs(ot[L, i]), abs(ot[L, i, 1]))
                assert np.all(np.abs(gt[L, i] - ot[L, i]) <= tol), (L, i, gt[L, i], ot[L, i])


def multiplier_events(gv, ov, params, kind):
    """Alg. 5 compares every window entry with a fence; an entry that lies on a fence to within
    the score tolerance may fall on either side, which moves k by one whole widen/narrow step.
    Returns the number of (level, metric) windows where that happened; anything else fails."""
    gt, gvalid = gv.sentinel_get_thresholds(kind)
    ot, ovalid = ov.thresholds(kind)
    assert np.array_equal(gvalid, ovalid)
    events = 0
    lg, ls = np.log(params.gamma_g[kind]), np.log(params.gamma_s[kind])
    for L in range(2):
        for i in range(ovalid.shape[1]):
            if not ovalid[L, i] or gt[L, i, 3] == pytest.approx(ot[L, i, 3], rel=1e-12):
                continue
            r = np.log(gt[L, i, 3] / ot[L, i, 3])
            n = params.n_max[kind]
            whole = any(abs(r - (a * lg + b * ls)) < 1e-9 for a in range(-n, n + 1) for b in range(-n, n + 1))
            assert whole, "k differs by no whole number of steps: %r vs %r" % (gt[L, i, 3], ot[L, i, 3])
            events += 1
    return events


def lockstep(sb, oracle_mod, w, gv, ov, params, steps, boundary=0, kinds=(ACT, GRAD), resync=True):
    """Runs the stream of workload `w` through both sides.  Returns per-step records."""
    near_events, flagged_steps, corrupted, k_events = 0, 0, 0, 0
    for t in range(steps):
        for kind in kinds:
            x, name = synth.microbatch(w, boundary, kind, t, "cuda")
            xb = synth.bits(x)
            scale = max(float(x.float().abs().mean()), 1e-12)
            if t < w.warmup:
                gs = gv.update_reference(x, kind)
                os_, _ = ov.update_reference(xb, kind)
                torch.cuda.synchronize()
                assert_scores_close(gs.cpu().numpy(), os_, scale, "warm-up step %d kind %d" % (t, kind))
                ev = multiplier_events(gv, ov, params, kind)
                if ev:
                    k_events += ev
                    gv.sentinel_import_state(oracle_to_blob(ov, params))
                continue
            corrupted += name is not None
            thr, valid = ov.thresholds(kind)
            gs, gf = gv.verify(x, kind)
            os_, of, _ = ov.verify(xb, kind)
            torch.cuda.synchronize()
            gs, gf = gs.cpu().numpy(), gf.cpu().numpy().view(np.uint32)
            assert_scores_close(gs, os_, scale, "step %d kind %d (%s)" % (t, kind, name))
            flagged_steps += bool(np.any(of & UNIT_BITS))
            if not np.array_equal(gf, of):
                near = near_threshold(os_, thr, valid, w.B)
                differ = (gf ^ of) & UNIT_BITS
                assert np.all(near[differ != 0]), "flags differ away from a bound at step %d: %s vs %s" % (t, gf, of)
                near_events += 1
                assert resync, "near-threshold disagreement"
                gv.sentinel_import_state(oracle_to_blob(ov, params))   # oracle -> library
            ev = multiplier_events(gv, ov, params, kind)
            if ev:
                k_events += ev
                gv.sentinel_import_state(oracle_to_blob(ov, params))
    return {"near": near_events, "flagged": flagged_steps, "corrupted": corrupted, "k_events": k_events}


def compare_state(gv, ov, params, m_scale_rel=1e-5):
    st = parse_blob(gv.sentinel_export_state(), params.B, params.T, params.d, params.l)
    assert (st["violations"], st["clean_streak"], st["banned"]) == ov.counters()
    for kind in (ACT, GRAD):
        ks = st["kinds"][kind]
        assert ks["steps"] == ov.steps(kind)
        m_ref = ov.ema(kind)
        tol = m_scale_rel * max(float(np.abs(m_ref).max()), 1e-30)
        assert np.max(np.abs(ks["m"].astype(np.float64) - m_ref)) <= tol
        assert st["n_metrics"] == ov.nm
        for L in range(2):
            for i in range(ov.nm):
                href = ov.history(kind, L, i)
                assert ks["hist"][L][i].size == href.size
                floor = 1e-3 * (np.abs(href).mean() if i in (0, 3) and href.size else 1.0)
                assert np.all(np.abs(ks["hist"][L][i] - href) <= 1e-3 * np.maximum(np.abs(href), floor))


def test_config1_scenario(sb, oracle_mod):
    """B=8 x T=128 x d=512, N(0,1): 16 clean warm-up microbatches, then sample 3 times 10."""
    w = synth.WORKLOADS["cfg1"]
    gv, ov, params = make_pair(sb, oracle_mod, w)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, w.warmup, kinds=(ACT,))
    compare_thresholds(gv, ov, ACT)
    x, name = synth.microbatch(w, 0, ACT, w.warmup, "cuda")
    assert name == "scale_sample3"
    gs, gf = gv.verify(x, ACT)
    os_, of, commit = ov.verify(synth.bits(x), ACT)
    gf = gf.cpu().numpy().view(np.uint32)
    assert np.array_equal(gf, of)
    assert not commit and (gf[4] & sb.FLAG_L1) and not (gf[0] & sb.FLAG_COMMITTED)
    assert_scores_close(gs.cpu().numpy(), os_, 0.8, "verify")
    assert gs[4, 0] > 5 * gs[1, 0]
    compare_state(gv, ov, params)
    compare_thresholds(gv, ov, ACT)
    assert rec["near"] == 0 and rec["k_events"] == 0
    gv.close()


STREAMS = [
    ("cfg2", (6, 40, 1024), 60),       # lognormal channel scales; additive noise, gradient sign flips
    ("cfg3", (4, 96, 520), 90),        # zeroed token rows, stale replays (needs > 50 steps)
    ("cfg4", (4, 24, 2056), 50),       # Student-t activations; uniform noise on one sample
]


@pytest.mark.parametrize("name,shape,steps", STREAMS, ids=[s[0] for s in STREAMS])
def test_streams_in_lockstep(sb, oracle_mod, name, shape, steps):
    """The recipe of each benchmark configuration at a size the oracle finishes in seconds
    (several row tiles, ragged d), with a corruption rate raised so that every kind occurs."""
    w = synth.scaled(synth.WORKLOADS[name], name + "_small", *shape, corrupt_rate=0.25)
    gv, ov, params = make_pair(sb, oracle_mod, w)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, steps)
    assert rec["corrupted"] >= 5
    compare_state(gv, ov, params)
    for kind in (ACT, GRAD):
        compare_thresholds(gv, ov, kind)
    assert rec["near"] <= 1 and rec["k_events"] <= 3, rec
    print(name, rec)
    gv.close()


@pytest.mark.parametrize("shape,l", [((5, 2, 8), 4), ((3, 4, 16), 9), ((16, 8, 64), 6)],
                         ids=["5x2x8_l4", "3x4x16_l9", "16x8x64_l6"])
def test_long_streams_with_small_windows(sb, oracle_mod, shape, l):
    """Many more steps than the window holds, on tensors so small that the sign-flip ratio takes
    few distinct values: the windows wrap again and again and are full of equal entries, which
    is what the incrementally maintained ascending copies have to get right."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "tiny_stream", *shape, corrupt_rate=0.3, warmup=6)
    gv, ov, params = make_pair(sb, oracle_mod, w, l=l)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, 70)
    compare_state(gv, ov, params)
    for kind in (ACT, GRAD):
        compare_thresholds(gv, ov, kind)
    assert rec["near"] + rec["k_events"] <= 6, rec
    gv.close()


def test_stream_at_the_largest_batch_and_window(sb, oracle_mod):
    """B = 64 samples (the compiled maximum) with the longest window that fits: 63 * 65 = 4095
    entries per kind across the two levels."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "max_b", 64, 6, 72, corrupt_rate=0.2, warmup=8)
    gv, ov, params = make_pair(sb, oracle_mod, w, l=63)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, 75, kinds=(ACT,))
    compare_state(gv, ov, params)
    compare_thresholds(gv, ov, ACT)
    assert rec["near"] <= 2 and rec["k_events"] <= 4, rec
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(64, 6, 72, window_steps=64)             # 64 * 65 = 4160 > 4096
    assert e.value.code == sb.ERR_UNSUPPORTED
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(65, 6, 72, window_steps=10)
    assert e.value.code == sb.ERR_UNSUPPORTED
    gv.close()


def test_many_boundaries_on_separate_streams(sb, oracle_mod):
    """Config-5 pattern: independent handles, one CUDA stream each, interleaved act/grad."""
    w = synth.scaled(synth.WORKLOADS["cfg5"], "cfg5_small", 4, 32, 512, corrupt_rate=0.2, boundaries=4)
    pairs = [make_pair(sb, oracle_mod, w) for _ in range(w.boundaries)]
    streams = [torch.cuda.Stream() for _ in range(w.boundaries)]
    steps = w.warmup + 24
    outs = []
    for t in range(steps):
        for b, ((gv, ov, params), s) in enumerate(zip(pairs, streams)):
            for kind in (ACT, GRAD):
                x, _ = synth.microbatch(w, b, kind, t, "cuda")
                torch.cuda.current_stream().synchronize()
                x.record_stream(s)
                with torch.cuda.stream(s):
                    if t < w.warmup:
                        gv.update_reference(x, kind, stream=s)
                        ov.update_reference(synth.bits(x), kind)
                    else:
                        gs, gf = gv.verify(x, kind, stream=s)
                        os_, of, _ = ov.verify(synth.bits(x), kind)
                        outs.append((gs, gf, os_, of, float(x.float().abs().mean())))
    torch.cuda.synchronize()
    for gs, gf, os_, of, scale in outs:
        assert_scores_close(gs.cpu().numpy(), os_, scale, "multi-stream")
        assert np.array_equal(gf.cpu().numpy().view(np.uint32), of)
    for gv, ov, params in pairs:
        compare_state(gv, ov, params)
        gv.close()


def test_import_oracle_state_then_verify(sb, oracle_mod):
    """Load the oracle's state into the library and compare one verified step: isolates the
    finalize logic from differences accumulated in the history."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "cfg2_tiny", 3, 16, 264)
    gv, ov, params = make_pair(sb, oracle_mod, w, l=7)
    for t in range(12):                                  # more steps than the window holds
        for kind in (ACT, GRAD):
            ov.update_reference(synth.bits(synth.clean(w, 0, kind, t, "cuda")), kind)
    gv.sentinel_import_state(oracle_to_blob(ov, params))
    for kind in (ACT, GRAD):
        gt, gvalid = gv.sentinel_get_thresholds(kind)
        ot, ovalid = ov.thresholds(kind)
        assert np.array_equal(gt, ot) and np.array_equal(gvalid, ovalid)     # exact round trip
    for t in range(12, 20):
        for kind in (ACT, GRAD):
            x = synth.clean(w, 0, kind, t, "cuda")
            if t == 15:
                x = (x.float() * 2.5).to(torch.bfloat16)
            gs, gf = gv.verify(x, kind)
            os_, of, _ = ov.verify(synth.bits(x), kind)
            assert np.array_equal(gf.cpu().numpy().view(np.uint32), of)
            assert_scores_close(gs.cpu().numpy(), os_, float(x.float().abs().mean()), "after import")
            compare_thresholds(gv, ov, kind)
    compare_state(gv, ov, params)
    # export -> import into a fresh handle -> identical behaviour
    blob = gv.sentinel_export_state()
    gv2 = sb.Verifier(w.B, w.T, w.d, window_steps=7)
    gv2.sentinel_import_state(blob)
    x = synth.clean(w, 0, ACT, 20, "cuda")
    a = gv.verify(x, ACT)
    b = gv2.verify(x, ACT)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert bytes(gv.sentinel_export_state()) == bytes(gv2.sentinel_export_state())
    gv.close(); gv2.close()


def test_counters_ban_forgiveness_and_reset(sb, oracle_mod):
    w = synth.scaled(synth.WORKLOADS["cfg1"], "cfg1_small", 4, 16, 128)
    gv, ov, params = make_pair(sb, oracle_mod, w, c=3, t_forgiveness=4)
    for t in range(16):
        x = synth.clean(w, 0, ACT, t, "cuda")
        gv.update_reference(x, ACT)
        ov.update_reference(synth.bits(x), ACT)
    script = [3.0, 1, 1, 1, 1, 1, 3.0, 1, 3.0, 3.0, 1, "reset", 1, 4096.0, 1]
    t = 16
    for item in script:
        if item == "reset":
            gv.sentinel_reset_worker()
            ov.reset_worker()
            continue
        x = (synth.clean(w, 0, ACT, t, "cuda").float() * float(item)).to(torch.bfloat16)
        t += 1
        gs, gf = gv.verify(x, ACT)
        os_, of, _ = ov.verify(synth.bits(x), ACT)
        assert np.array_equal(gf.cpu().numpy().view(np.uint32), of), item
        c = gv.sentinel_get_counters()
        assert (c["violations"], c["clean_streak"], c["banned"]) == ov.counters()
        assert c["steps_act"] == ov.steps(ACT) and c["error"] == 0
    assert of[0] & sb.FLAG_BANNED                       # the 4096x step was severe
    gv.close()


def test_non_finite_and_no_warmup_paths(sb, oracle_mod):
    w = synth.scaled(synth.WORKLOADS["cfg1"], "cfg1_small", 3, 8, 64)
    gv, ov, params = make_pair(sb, oracle_mod, w)
    x = synth.clean(w, 0, ACT, 0, "cuda")
    gs, gf = gv.verify(x, ACT)                           # no warm-up at all
    os_, of, _ = ov.verify(synth.bits(x), ACT)
    assert np.array_equal(gf.cpu().numpy().view(np.uint32), of)
    assert of[0] == (sb.FLAG_COMMITTED | sb.FLAG_NO_THRESHOLDS)
    bad = synth.clean(w, 0, ACT, 1, "cuda").float()
    bad[1, 3, 5] = float("nan")
    bad = bad.to(torch.bfloat16)
    gs, gf = gv.verify(bad, ACT)
    os_, of, _ = ov.verify(synth.bits(bad), ACT)
    assert np.array_equal(gf.cpu().numpy().view(np.uint32), of)
    assert_scores_close(gs.cpu().numpy(), os_, 0.8, "nan step")
    gv.update_reference(bad, ACT)                        # refused: nothing changes
    ov.update_reference(synth.bits(bad), ACT)
    compare_state(gv, ov, params)
    gv.close()


@pytest.mark.parametrize("d", [392, 1024, 2568])
def test_token_statistics_buffer(sb, oracle_mod, d):
    """Per-token partial sums: sum_c x, sum_c x^2, sum_c |x-m|, sign mismatches, against the
    oracle's token sums taken with the oracle's reference; rows of one and of several tiles."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "cfg2_tok", 3, 21, d)
    gv, ov, params = make_pair(sb, oracle_mod, w)
    buf = torch.full((w.B, w.T, 4), -1.0, dtype=torch.float32, device="cuda")
    gv.sentinel_set_token_stats_buffer(buf)
    for t in range(3):
        x = synth.clean(w, 0, ACT, t, "cuda")
        m = ov.ema(ACT)
        gv.update_reference(x, ACT)
        ov.update_reference(synth.bits(x), ACT)
        xv = oracle_mod.bf16_to_f64(synth.bits(x))
        want = oracle_mod.token_sums(synth.bits(x), m)
        got = buf.cpu().numpy().astype(np.float64)
        scale = np.array([np.sqrt(w.d) * xv.std(), 1.0, 1.0, 1.0])
        tol = 1e-3 * np.maximum(np.abs(want), scale)
        # where the EMA cancels to zero up to rounding (bf16 inputs in the ratio -beta/(1-beta))
        # its sign, hence one mismatch count, is decided by rounding noise on either side
        tol[..., 3] += (np.abs(m) <= 1e-9 * np.abs(m).mean()).sum(-1)
        assert np.all(np.abs(got - want) <= tol)
    gv.sentinel_set_token_stats_buffer(None)
    buf.fill_(-1.0)
    gv.update_reference(synth.clean(w, 0, ACT, 3, "cuda"), ACT)
    torch.cuda.synchronize()
    assert torch.all(buf == -1.0)
    gv.close()


@pytest.mark.parametrize("shape", [(3, 7, 264), (4, 64, 2048)], ids=["3x7x264", "4x64x2048"])
def test_gradient_replacement(sb, oracle_mod, shape):
    """Alg. 4 on the device: untouched after a clean step, the reference (bf16) or zeros after
    a flagged one.  The library rounds its fp32 reference, the oracle its float64 one, so the
    bf16 results may differ by one unit in the last place where the two references straddle a
    rounding boundary (or by the EMA's own absolute accuracy where it nearly cancels): at most
    1 element in 1000."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "cfg2_repl", *shape)
    gv, ov, params = make_pair(sb, oracle_mod, w)
    for t in range(10):
        g = synth.clean(w, 0, GRAD, t, "cuda")
        gv.update_reference(g, GRAD)
        ov.update_reference(synth.bits(g), GRAD)
    did = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    g = synth.clean(w, 0, GRAD, 10, "cuda")
    gv.verify(g, GRAD)
    ov.verify(synth.bits(g), GRAD)
    out = g.clone()
    gv.sentinel_replace_if_flagged(out, GRAD, 0, did)
    ref, ref_did = ov.replace_if_flagged(synth.bits(g), GRAD)
    assert int(did) == 0 and not ref_did and torch.equal(out, g)

    bad = (synth.clean(w, 0, GRAD, 11, "cuda").float() * 40.0).to(torch.bfloat16)
    _, gf = gv.verify(bad, GRAD)
    _, of, _ = ov.verify(synth.bits(bad), GRAD)
    assert np.array_equal(gf.cpu().numpy().view(np.uint32), of) and (of[0] & 0xFFFF)
    for fill in (0, 1):
        out = bad.clone()
        gv.sentinel_replace_if_flagged(out, GRAD, fill, did)   # enqueued right behind the verify
        ref, ref_did = ov.replace_if_flagged(synth.bits(bad), GRAD, fill)
        assert int(did) == 1 and ref_did
        got = synth.bits(out)
        gv_, rv_ = oracle_mod.bf16_to_f64(got), oracle_mod.bf16_to_f64(ref)
        # one bf16 ulp of the value, plus the absolute accuracy of an fp32 EMA (elements where
        # the EMA nearly cancels are tiny, and there the two references differ relatively a lot)
        tol = 2.0 ** -7 * np.abs(rv_) + 1e-6 * rv_.std()
        assert np.all(np.abs(gv_ - rv_) <= tol)
        assert np.count_nonzero(got != ref) <= 1e-3 * got.size, np.count_nonzero(got != ref)
        if fill:
            assert not got.any()
    out = torch.ones_like(bad)                                 # the other kind was never flagged
    gv.sentinel_replace_if_flagged(out, ACT, 0, did)
    assert int(did) == 0 and torch.all(out == 1)
    gv.close()


@pytest.mark.parametrize("k,stride", [(40, 41), (41, 42), (1024, 1025), (264, 264), (523, 530)],
                         ids=["k40_s41", "k41_s42", "k1024_s1025", "k264_dense", "k523_s530"])
def test_compressed_signal_layout(sb, oracle_mod, k, stride):
    """x[:, :, :k] of a [B, T, stride] tensor (the subspace-compressed signal of the SWARM
    appendix, whose last channel is not verified): rows start on odd 2-byte boundaries and k
    need not be a multiple of 8.  The oracle sees the packed slice."""
    B, T = 3, 29
    w = synth.scaled(synth.WORKLOADS["cfg2"], "compressed", B, T, stride)
    gv = sb.Verifier(B, T, k)
    params = oracle_mod.Params(B=B, T=T, d=k)
    ov = oracle_mod.Verifier(params)
    buf = torch.full((B, T, 4), -1.0, dtype=torch.float32, device="cuda")
    gv.sentinel_set_token_stats_buffer(buf)
    for t in range(14):
        wide = synth.clean(w, 0, ACT, t, "cuda")
        if t == 12:
            wide = (wide.float() * 5).to(torch.bfloat16)
        wide[:, :, k:] = 1000.0                                # never looked at
        packed = wide[:, :, :k].contiguous()
        scale = float(packed.float().abs().mean())
        if t < 8:
            gs = torch.empty(1 + B, 3, device="cuda")
            gv.sentinel_update_reference_strided(wide, ACT, gs)
            os_, _ = ov.update_reference(synth.bits(packed), ACT)
        else:
            gs = torch.empty(1 + B, 3, device="cuda")
            gf = torch.empty(1 + B, dtype=torch.int32, device="cuda")
            gv.sentinel_verify_strided(wide, ACT, gs, gf)
            os_, of, _ = ov.verify(synth.bits(packed), ACT)
            assert np.array_equal(gf.cpu().numpy().view(np.uint32), of), t
        assert_scores_close(gs.cpu().numpy(), os_, scale, "compressed step %d" % t)
        xv = oracle_mod.bf16_to_f64(synth.bits(packed))
        assert np.allclose(buf.cpu().numpy()[..., 0], xv.sum(-1), rtol=1e-3, atol=1e-3 * np.sqrt(k))
    compare_state(gv, ov, params)
    gv.close()


@pytest.mark.parametrize("k,stride,offset", [(1024, 1025, 0), (512, 515, 3), (2056, 2057, 5), (264, 272, 7),
                                             (8, 9, 1), (1528, 1536, 2)],
                         ids=["k1024_s1025", "k512_s515_o3", "k2056_s2057_o5", "k264_s272_o7", "k8_s9_o1", "k1528_s1536_o2"])
def test_compressed_signal_layout_with_rows_on_any_2_byte_boundary(sb, oracle_mod, k, stride, offset):
    """The same layout with k a multiple of 8, where the library puts x in place with a funnel
    shift and keeps the 128/256-bit path: every misalignment of a row start (strides and base
    offsets that walk through all residues mod 16 bytes), a last row that ends with the
    allocation, both reference formats."""
    B, T = 3, 29
    w = synth.scaled(synth.WORKLOADS["cfg2"], "compressed_shift", B, T, stride)
    n = B * T * stride
    for bf16 in (0, 1):
        gv = sb.Verifier(B, T, k, ema_bf16=bf16)
        params = oracle_mod.Params(B=B, T=T, d=k, ema_bf16=bf16)
        ov = oracle_mod.Verifier(params)
        for t in range(12):
            src = synth.clean(w, 0, GRAD, t, "cuda")
            if t == 10:
                src = (src.float() * 5).to(torch.bfloat16)
            # the tensor ends exactly where its allocation ends; its base is `offset` elements in
            flat = torch.empty(offset + n, dtype=torch.bfloat16, device="cuda")
            wide = flat[offset:].view(B, T, stride)
            wide.copy_(src)
            wide[:, :, k:] = 1000.0                            # never looked at
            packed = wide[:, :, :k].contiguous()
            scale = float(packed.float().abs().mean())
            gs = torch.empty(1 + B, 3, device="cuda")
            if t < 7:
                gv.sentinel_update_reference_strided(wide, GRAD, gs)
                os_, _ = ov.update_reference(synth.bits(packed), GRAD)
            else:
                gf = torch.empty(1 + B, dtype=torch.int32, device="cuda")
                gv.sentinel_verify_strided(wide, GRAD, gs, gf)
                os_, of, _ = ov.verify(synth.bits(packed), GRAD)
                assert np.array_equal(gf.cpu().numpy().view(np.uint32), of), t
            assert_scores_close(gs.cpu().numpy(), os_, scale, "shifted step %d" % t)
        if bf16:
            st = parse_blob(gv.sentinel_export_state(), B, T, k, 100)
            assert np.array_equal(st["kinds"][GRAD]["m"].astype(np.float64), ov.ema(GRAD))   # bit for bit
        else:
            compare_state(gv, ov, params)
        gv.close()


def test_runs_are_bit_reproducible(sb):
    w = synth.scaled(synth.WORKLOADS["cfg2"], "cfg2_rep", 4, 50, 1024)
    blobs, outs = [], []
    for _ in range(2):
        gv = sb.Verifier(w.B, w.T, w.d)
        o = []
        for t in range(6):
            for kind in (ACT, GRAD):
                x, _ = synth.microbatch(w, 0, kind, t, "cuda")
                o.append(gv.update_reference(x, kind) if t < 3 else gv.verify(x, kind)[0])
        outs.append(torch.stack(o).cpu())
        blobs.append(bytes(gv.sentinel_export_state()))
        gv.close()
    assert torch.equal(outs[0], outs[1])
    assert blobs[0] == blobs[1]


def test_verify_host_matches_device_call(sb):
    w = synth.scaled(synth.WORKLOADS["cfg1"], "cfg1_host", 4, 32, 256)
    a, b = sb.Verifier(w.B, w.T, w.d), sb.Verifier(w.B, w.T, w.d)
    for t in range(5):
        x = synth.clean(w, 0, ACT, t, "cuda")
        a.update_reference(x, ACT)
        b.update_reference(x, ACT)
    x = (synth.clean(w, 0, ACT, 5, "cuda").float() * 4).to(torch.bfloat16)
    ds, df = a.verify(x, ACT)
    hx = x.cpu().pin_memory()
    hs = torch.empty(1 + w.B, 3, dtype=torch.float32).pin_memory()
    hf = torch.empty(1 + w.B, dtype=torch.int32).pin_memory()
    b.sentinel_verify_host(hx, ACT, hs, hf)
    assert torch.equal(ds.cpu(), hs) and torch.equal(df.cpu(), hf)
    a.close(); b.close()


def test_argument_errors_never_reach_the_gpu(sb):
    odd = sb.Verifier(2, 4, 12)                           # d % 8 != 0: strided entry points only
    xo = torch.zeros(2, 4, 12, dtype=torch.bfloat16, device="cuda")
    so, fo = torch.zeros(3, 3, device="cuda"), torch.zeros(3, dtype=torch.int32, device="cuda")
    with pytest.raises(sb.SentinelError) as e:
        odd.sentinel_verify(xo, 0, so, fo)
    assert e.value.code == sb.ERR_UNALIGNED
    odd.sentinel_verify_strided(xo, 0, so, fo)
    Lo, st_ = sb.lib(), torch.cuda.current_stream().cuda_stream
    assert Lo.sentinel_verify_strided(odd._h, xo.data_ptr(), 0, 2, 4, 12, 11, st_, so.data_ptr(), fo.data_ptr()) == sb.ERR_INVALID_ARG
    assert Lo.sentinel_verify_strided(odd._h, xo.data_ptr() + 1, 0, 2, 4, 12, 12, st_, so.data_ptr(), fo.data_ptr()) == sb.ERR_UNALIGNED
    assert Lo.sentinel_verify_strided(odd._h, xo.data_ptr(), 0, 2, 4, 16, 16, st_, so.data_ptr(), fo.data_ptr()) == sb.ERR_SHAPE_MISMATCH
    torch.cuda.synchronize()
    odd.close()
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(65, 4, 8)
    assert e.value.code == sb.ERR_UNSUPPORTED
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(64, 4, 8, window_steps=100)
    assert e.value.code == sb.ERR_UNSUPPORTED
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(40, 4, 8, window_steps=100)           # 100 * 41 > 4096
    assert e.value.code == sb.ERR_UNSUPPORTED
    sb.Verifier(39, 4, 8, window_steps=100).close()      # 100 * 40 fits
    for bad in (dict(beta=(1.0, 0.5)), dict(gamma_grow=(0.9, 1.1)), dict(window_steps=0), dict(device=99)):
        with pytest.raises(sb.SentinelError) as e:
            sb.Verifier(2, 4, 8, **bad)
        assert e.value.code == sb.ERR_INVALID_ARG
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(0, 4, 8)
    assert e.value.code == sb.ERR_INVALID_ARG

    v = sb.Verifier(2, 4, 16)
    x = torch.zeros(2, 4, 16, dtype=torch.bfloat16, device="cuda")
    scores = torch.zeros(3, 3, device="cuda")
    flags = torch.zeros(3, dtype=torch.int32, device="cuda")
    before = bytes(v.sentinel_export_state())
    L, h = sb.lib(), v._h
    s = torch.cuda.current_stream().cuda_stream
    assert L.sentinel_verify(h, x.data_ptr(), 0, 2, 4, 8, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_SHAPE_MISMATCH
    assert b"differs" in L.sentinel_last_error(h)
    assert L.sentinel_verify(h, x.data_ptr() + 2, 0, 2, 4, 16, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_UNALIGNED
    assert L.sentinel_verify(h, x.data_ptr(), 2, 2, 4, 16, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_INVALID_ARG
    assert L.sentinel_verify(h, None, 0, 2, 4, 16, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_INVALID_ARG
    assert L.sentinel_verify(h, x.data_ptr(), 0, 2, 4, 16, s, None, flags.data_ptr()) == sb.ERR_INVALID_ARG
    assert L.sentinel_verify(None, x.data_ptr(), 0, 2, 4, 16, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_INVALID_ARG
    assert L.sentinel_update_reference(h, x.data_ptr(), 0, 3, 4, 16, s, None) == sb.ERR_SHAPE_MISMATCH
    assert L.sentinel_replace_if_flagged(h, x.data_ptr(), 0, 2, 4, 16, 2, s, None) == sb.ERR_INVALID_ARG
    assert L.sentinel_replace_if_flagged(h, x.data_ptr() + 2, 0, 2, 4, 16, 0, s, None) == sb.ERR_UNALIGNED
    assert L.sentinel_replace_if_flagged(h, x.data_ptr(), 0, 2, 4, 8, 0, s, None) == sb.ERR_SHAPE_MISMATCH
    assert L.sentinel_export_state(h, bytes(8), 8, s) == sb.ERR_STATE_SIZE
    junk = bytearray(before)
    junk[0] ^= 0xFF
    assert L.sentinel_import_state(h, bytes(junk), len(junk), s) == sb.ERR_STATE_SIZE
    assert L.sentinel_distance(x.data_ptr(), None, 2, 4, 16, 0, s, scores.data_ptr(), None) == sb.ERR_INVALID_ARG
    assert L.sentinel_distance(x.data_ptr(), scores.data_ptr(), 2, 4, 12, 0, s, scores.data_ptr(), None) == sb.ERR_UNALIGNED
    torch.cuda.synchronize()
    assert bytes(v.sentinel_export_state()) == before      # none of the above touched the state
    v.close()


# ---------------------------------------------------------------------------------------------
# the reference stored as bf16 (ema_bf16 = 1)

def reference_bits_equal(gv, ov, params):
    """With a bf16 reference both sides round the same single-precision value once: the stored
    references agree bit for bit, not merely to a tolerance."""
    st = parse_blob(gv.sentinel_export_state(), params.B, params.T, params.d, params.l)
    for kind in (ACT, GRAD):
        assert np.array_equal(st["kinds"][kind]["m"].astype(np.float64), ov.ema(kind)), kind


@pytest.mark.parametrize("name,shape,steps", [("cfg2", (5, 40, 1024), 50), ("cfg4", (4, 24, 2056), 40),
                                              ("cfg3", (3, 70, 520), 70)], ids=["cfg2", "cfg4", "cfg3"])
def test_streams_in_lockstep_with_a_bf16_reference(sb, oracle_mod, name, shape, steps):
    w = synth.scaled(synth.WORKLOADS[name], name + "_bf16", *shape, corrupt_rate=0.25)
    gv, ov, params = make_pair(sb, oracle_mod, w, ema_bf16=1)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, steps)
    assert rec["corrupted"] >= 4
    compare_state(gv, ov, params)
    reference_bits_equal(gv, ov, params)
    for kind in (ACT, GRAD):
        compare_thresholds(gv, ov, kind)
    assert rec["near"] <= 1 and rec["k_events"] <= 3, rec
    # Alg. 4 hands out the stored bf16 reference as it is
    x, _ = synth.microbatch(w, 0, GRAD, 0, "cuda")
    loud = (x.float() * 64).to(torch.bfloat16)
    _, gf = gv.verify(loud, GRAD)
    ov.verify(synth.bits(loud), GRAD)
    out = loud.clone()
    gv.sentinel_replace_if_flagged(out, GRAD, 0)
    want, did = ov.replace_if_flagged(synth.bits(loud), GRAD)
    torch.cuda.synchronize()
    assert did and np.array_equal(synth.bits(out), want)
    gv.close()


def test_bf16_reference_with_strided_rows(sb, oracle_mod):
    B, T, k, stride = 3, 21, 523, 524
    w = synth.scaled(synth.WORKLOADS["cfg2"], "compressed_bf16", B, T, stride)
    gv = sb.Verifier(B, T, k, ema_bf16=1)
    params = oracle_mod.Params(B=B, T=T, d=k, ema_bf16=1)
    ov = oracle_mod.Verifier(params)
    for t in range(12):
        wide = synth.clean(w, 0, ACT, t, "cuda")
        packed = wide[:, :, :k].contiguous()
        gs = torch.empty(1 + B, 3, device="cuda")
        if t < 8:
            gv.sentinel_update_reference_strided(wide, ACT, gs)
            os_, _ = ov.update_reference(synth.bits(packed), ACT)
        else:
            gf = torch.empty(1 + B, dtype=torch.int32, device="cuda")
            gv.sentinel_verify_strided(wide, ACT, gs, gf)
            os_, of, _ = ov.verify(synth.bits(packed), ACT)
            assert np.array_equal(gf.cpu().numpy().view(np.uint32), of), t
        assert_scores_close(gs.cpu().numpy(), os_, float(packed.float().abs().mean()), "step %d" % t)
    reference_bits_equal(gv, ov, params)
    gv.close()


def test_bf16_reference_restrictions_and_state_round_trip(sb):
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(2, 8, 64, ema_bf16=2)
    assert e.value.code == sb.ERR_INVALID_ARG
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(2, 8, 64, ema_bf16=1, ref_over_batch=1)
    assert e.value.code == sb.ERR_UNSUPPORTED
    gv = sb.Verifier(2, 8, 64, ema_bf16=1)
    w = synth.scaled(synth.WORKLOADS["cfg1"], "bf16_rt", 2, 8, 64)
    for t in range(5):
        gv.update_reference(synth.clean(w, 0, ACT, t, "cuda"), ACT)
    blob = bytes(gv.sentinel_export_state())
    other = sb.Verifier(2, 8, 64, ema_bf16=1)
    other.sentinel_import_state(blob)
    assert bytes(other.sentinel_export_state()) == blob
    x = synth.clean(w, 0, ACT, 5, "cuda")
    a, b = gv.verify(x, ACT), other.verify(x, ACT)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    # a state written by an fp32 verifier goes in rounded to nearest even
    f32 = sb.Verifier(2, 8, 64)
    for t in range(5):
        f32.update_reference(synth.clean(w, 0, ACT, t, "cuda"), ACT)
    st = parse_blob(f32.sentinel_export_state(), 2, 8, 64, 100)
    other.sentinel_import_state(f32.sentinel_export_state())
    got = parse_blob(other.sentinel_export_state(), 2, 8, 64, 100)["kinds"][ACT]["m"]
    want = torch.from_numpy(st["kinds"][ACT]["m"]).to(torch.bfloat16).float().numpy()
    assert np.array_equal(got, want)
    gv.close(); other.close(); f32.close()


def test_verify_calls_replay_from_a_cuda_graph(sb):
    """A verified step is one kernel launch with no allocation and no host decision, so a sequence
    of calls can be captured once and replayed: every replay is the next step on whatever the
    input buffers hold, and leaves the same scores, flags and state as the same calls made one
    by one."""
    w = synth.scaled(synth.WORKLOADS["cfg1"], "graph", 8, 128, 512)
    eager, graphed = sb.Verifier(w.B, w.T, w.d), sb.Verifier(w.B, w.T, w.d)
    for t in range(8):
        for kind in (ACT, GRAD):
            x = synth.clean(w, 0, kind, t, "cuda")
            eager.update_reference(x, kind)
            graphed.update_reference(x, kind)
    buf = [torch.empty(w.B, w.T, w.d, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    scores = torch.zeros(2, 1 + w.B, 3, device="cuda")
    flags = torch.zeros(2, 1 + w.B, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for kind in (ACT, GRAD):
            graphed.sentinel_verify(buf[kind], kind, scores[kind], flags[kind])
    for t in range(8, 14):
        xs = [synth.clean(w, 0, kind, t, "cuda") for kind in (ACT, GRAD)]
        if t == 11:
            xs[ACT] = synth.corrupt(w, xs[ACT], "scale_sample3", 0, ACT, t)
        for kind in (ACT, GRAD):
            buf[kind].copy_(xs[kind])
        graph.replay()
        torch.cuda.synchronize()
        for kind in (ACT, GRAD):
            es, ef = eager.verify(xs[kind], kind)
            assert torch.equal(es, scores[kind]) and torch.equal(ef, flags[kind]), (t, kind)
        if t == 11:
            assert int(flags[ACT, 4]) & sb.FLAG_L1 and not int(flags[ACT, 0]) & sb.FLAG_COMMITTED
    assert bytes(eager.sentinel_export_state()) == bytes(graphed.sentinel_export_state())
    eager.close(); graphed.close()


# ---------------------------------------------------------------------------------------------
# one [T,d] reference shared by the B samples (ref_over_batch = 1)

@pytest.mark.parametrize("name,shape,steps", [("cfg2", (6, 40, 1024), 50), ("cfg4", (4, 24, 2056), 40),
                                              ("cfg3", (16, 30, 520), 60), ("cfg2", (1, 37, 264), 40)],
                         ids=["cfg2_B6", "cfg4_B4", "cfg3_B16", "cfg2_B1"])
def test_streams_in_lockstep_with_a_shared_reference(sb, oracle_mod, name, shape, steps):
    w = synth.scaled(synth.WORKLOADS[name], name + "_shared", *shape, corrupt_rate=0.25)
    gv, ov, params = make_pair(sb, oracle_mod, w, ref_over_batch=1)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, steps)
    assert rec["corrupted"] >= 3
    compare_state(gv, ov, params)
    for kind in (ACT, GRAD):
        compare_thresholds(gv, ov, kind)
        st = gv.sentinel_get_stats(kind).cpu().numpy()
        x, _ = synth.microbatch(w, 0, kind, steps - 1, "cuda")
        assert_stats_close(st, ov.last_stats(kind), max(float(x.float().std()), 1e-30),
                           max(float(np.abs(ov.last_stats(kind)[0, 4])) ** 0.5, 1e-30), "stats kind %d" % kind)
    assert rec["near"] <= 2 and rec["k_events"] <= 4, rec
    # Alg. 4: every sample receives the one reference
    x, _ = synth.microbatch(w, 0, GRAD, 0, "cuda")
    loud = (x.float() * 64).to(torch.bfloat16)
    gv.verify(loud, GRAD)
    ov.verify(synth.bits(loud), GRAD)
    out = loud.clone()
    gv.sentinel_replace_if_flagged(out, GRAD, 0)
    want, did = ov.replace_if_flagged(synth.bits(loud), GRAD)
    torch.cuda.synchronize()
    assert did
    got = synth.bits(out)
    gv_, rv_ = oracle_mod.bf16_to_f64(got), oracle_mod.bf16_to_f64(want)
    assert np.mean(got != want) <= 1e-3 and np.all(np.abs(gv_ - rv_) <= 2.0 ** -7 * np.abs(rv_) + 1e-6 * float(np.std(rv_)))
    gv.close()


def test_shared_reference_restrictions_and_state_round_trip(sb):
    for kw in ({"n_workers": 2}, {"ema_bf16": 1}):
        with pytest.raises(sb.SentinelError) as e:
            sb.Verifier(2, 8, 64, ref_over_batch=1, **kw)
        assert e.value.code == sb.ERR_UNSUPPORTED
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(17, 8, 64, ref_over_batch=1)
    assert e.value.code == sb.ERR_UNSUPPORTED
    gv = sb.Verifier(3, 8, 64, ref_over_batch=1)
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_set_directions(synth.directions(4, 64, 1, "cuda"))
    assert e.value.code == sb.ERR_UNSUPPORTED
    s, f = torch.zeros(4, 3, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_verify_strided(torch.zeros(3, 8, 65, dtype=torch.bfloat16, device="cuda"), ACT, s, f)
    assert e.value.code == sb.ERR_UNSUPPORTED
    w = synth.scaled(synth.WORKLOADS["cfg1"], "shared_rt", 3, 8, 64)
    for t in range(5):
        gv.update_reference(synth.clean(w, 0, ACT, t, "cuda"), ACT)
    blob = bytes(gv.sentinel_export_state())
    assert len(blob) < len(bytes(sb.Verifier(3, 8, 64).sentinel_export_state()))   # T*d reference values per kind
    other = sb.Verifier(3, 8, 64, ref_over_batch=1)
    other.sentinel_import_state(blob)
    assert bytes(other.sentinel_export_state()) == blob
    x = synth.clean(w, 0, ACT, 5, "cuda")
    a, b = gv.verify(x, ACT), other.verify(x, ACT)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(3, 8, 64).sentinel_import_state(blob)                          # another reference shape
    assert e.value.code == sb.ERR_STATE_SIZE
    gv.close(); other.close()


# ---------------------------------------------------------------------------------------------
# one [d] reference shared by all B*T tokens (ref_over_batch = 1 and ref_over_tokens = 1)

@pytest.mark.parametrize("name,shape,steps", [("cfg2", (6, 40, 1024), 50), ("cfg4", (4, 24, 2056), 40),
                                              ("cfg3", (16, 30, 520), 60), ("cfg2", (1, 37, 264), 40),
                                              ("cfg2", (3, 5, 11000), 30), ("cfg4", (39, 3, 512), 30)],
                         ids=["cfg2_B6", "cfg4_B4", "cfg3_B16", "cfg2_B1", "cfg2_wide", "cfg4_B39"])
def test_streams_in_lockstep_with_a_channel_reference(sb, oracle_mod, name, shape, steps):
    w = synth.scaled(synth.WORKLOADS[name], name + "_channel", *shape, corrupt_rate=0.25)
    gv, ov, params = make_pair(sb, oracle_mod, w, ref_over_batch=1, ref_over_tokens=1)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, steps)
    assert rec["corrupted"] >= 3
    compare_state(gv, ov, params)
    for kind in (ACT, GRAD):
        compare_thresholds(gv, ov, kind)
        st = gv.sentinel_get_stats(kind).cpu().numpy()
        x, _ = synth.microbatch(w, 0, kind, steps - 1, "cuda")
        assert_stats_close(st, ov.last_stats(kind), max(float(x.float().std()), 1e-30),
                           max(float(np.abs(ov.last_stats(kind)[0, 4])) ** 0.5, 1e-30), "stats kind %d" % kind)
    assert rec["near"] <= 2 and rec["k_events"] <= 4, rec
    # Alg. 4: every token receives the one vector
    x, _ = synth.microbatch(w, 0, GRAD, 0, "cuda")
    loud = (x.float() * 64).to(torch.bfloat16)
    gv.verify(loud, GRAD)
    ov.verify(synth.bits(loud), GRAD)
    out = loud.clone()
    gv.sentinel_replace_if_flagged(out, GRAD, 0)
    want, did = ov.replace_if_flagged(synth.bits(loud), GRAD)
    torch.cuda.synchronize()
    assert did
    got = synth.bits(out)
    gv_, rv_ = oracle_mod.bf16_to_f64(got), oracle_mod.bf16_to_f64(want)
    assert np.mean(got != want) <= 1e-3 and np.all(np.abs(gv_ - rv_) <= 2.0 ** -7 * np.abs(rv_) + 1e-6 * float(np.std(rv_)))
    gv.close()


@pytest.mark.parametrize("name,shape,steps", [("cfg2", (6, 40, 1024), 50), ("cfg4", (4, 24, 2056), 40),
                                              ("cfg3", (16, 30, 520), 60), ("cfg2", (1, 37, 264), 40),
                                              ("cfg4", (39, 8, 512), 30), ("cfg2", (5, 200, 264), 30)],
                         ids=["cfg2_B6", "cfg4_B4", "cfg3_B16", "cfg2_B1", "cfg4_B39", "cfg2_T200"])
def test_streams_in_lockstep_with_a_channel_reference_per_sample(sb, oracle_mod, name, shape, steps):
    """[B,d]: one vector per sample (ref_over_tokens = 1 alone).  B = 39 with T = 8 gives CTAs two
    or three rows each and samples that several CTAs share; T = 200 gives CTAs that straddle two
    samples.  (Samples are kept at 4096 elements or more: with fewer, a single sign decided by
    rounding where the reference is all but zero moves the sign-flip ratio by more than 1e-3.)"""
    w = synth.scaled(synth.WORKLOADS[name], name + "_channel_ps", *shape, corrupt_rate=0.25)
    gv, ov, params = make_pair(sb, oracle_mod, w, ref_over_tokens=1)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, steps)
    assert rec["corrupted"] >= 3
    compare_state(gv, ov, params)
    for kind in (ACT, GRAD):
        compare_thresholds(gv, ov, kind)
        st = gv.sentinel_get_stats(kind).cpu().numpy()
        x, _ = synth.microbatch(w, 0, kind, steps - 1, "cuda")
        assert_stats_close(st, ov.last_stats(kind), max(float(x.float().std()), 1e-30),
                           max(float(np.abs(ov.last_stats(kind)[0, 4])) ** 0.5, 1e-30), "stats kind %d" % kind)
    assert rec["near"] <= 2 and rec["k_events"] <= 4, rec
    x, _ = synth.microbatch(w, 0, GRAD, 0, "cuda")
    loud = (x.float() * 64).to(torch.bfloat16)
    gv.verify(loud, GRAD)
    ov.verify(synth.bits(loud), GRAD)
    out = loud.clone()
    gv.sentinel_replace_if_flagged(out, GRAD, 0)
    want, did = ov.replace_if_flagged(synth.bits(loud), GRAD)
    torch.cuda.synchronize()
    assert did
    got = synth.bits(out)
    gv_, rv_ = oracle_mod.bf16_to_f64(got), oracle_mod.bf16_to_f64(want)
    assert np.mean(got != want) <= 1e-3 and np.all(np.abs(gv_ - rv_) <= 2.0 ** -7 * np.abs(rv_) + 1e-6 * float(np.std(rv_)))
    blob = bytes(gv.sentinel_export_state())                                       # round trip, another shape refused
    other = sb.Verifier(w.B, w.T, w.d, ref_over_tokens=1)
    other.sentinel_import_state(blob)
    assert bytes(other.sentinel_export_state()) == blob
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(w.B, w.T, w.d, ref_over_batch=1, ref_over_tokens=1).sentinel_import_state(blob)
    assert e.value.code == sb.ERR_STATE_SIZE
    gv.close(); other.close()


def test_channel_reference_restrictions_and_state_round_trip(sb):
    for kw in ({"n_workers": 2}, {"ema_bf16": 1}):
        with pytest.raises(sb.SentinelError) as e:
            sb.Verifier(2, 8, 64, ref_over_tokens=1, **kw)
        assert e.value.code == sb.ERR_UNSUPPORTED
    for kw in ({"n_workers": 2}, {"ema_bf16": 1}):
        with pytest.raises(sb.SentinelError) as e:
            sb.Verifier(2, 8, 64, ref_over_batch=1, ref_over_tokens=1, **kw)
        assert e.value.code == sb.ERR_UNSUPPORTED
    gv = sb.Verifier(3, 8, 64, ref_over_batch=1, ref_over_tokens=1)
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_set_directions(synth.directions(4, 64, 1, "cuda"))
    assert e.value.code == sb.ERR_UNSUPPORTED
    s, f = torch.zeros(4, 3, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_verify_strided(torch.zeros(3, 8, 65, dtype=torch.bfloat16, device="cuda"), ACT, s, f)
    assert e.value.code == sb.ERR_UNSUPPORTED
    w = synth.scaled(synth.WORKLOADS["cfg1"], "channel_rt", 3, 8, 64)
    for t in range(5):
        gv.update_reference(synth.clean(w, 0, ACT, t, "cuda"), ACT)
    blob = bytes(gv.sentinel_export_state())
    assert len(blob) < len(bytes(sb.Verifier(3, 8, 64, ref_over_batch=1).sentinel_export_state()))   # d values per kind
    other = sb.Verifier(3, 8, 64, ref_over_batch=1, ref_over_tokens=1)
    other.sentinel_import_state(blob)
    assert bytes(other.sentinel_export_state()) == blob
    x = synth.clean(w, 0, ACT, 5, "cuda")
    a, b = gv.verify(x, ACT), other.verify(x, ACT)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    for kw in ({}, {"ref_over_batch": 1}):
        with pytest.raises(sb.SentinelError) as e:
            sb.Verifier(3, 8, 64, **kw).sentinel_import_state(blob)               # another reference shape
        assert e.value.code == sb.ERR_STATE_SIZE
    gv.close(); other.close()


def test_channel_reference_runs_are_bit_reproducible_and_non_finite_input_changes_nothing(sb):
    w = synth.scaled(synth.WORKLOADS["cfg2"], "channel_rep", 5, 33, 1544)
    blobs = []
    for rep in range(2):
        gv = sb.Verifier(w.B, w.T, w.d, ref_over_batch=1, ref_over_tokens=1)
        for t in range(8):
            gv.update_reference(synth.clean(w, 0, GRAD, t, "cuda"), GRAD)
        before = bytes(gv.sentinel_export_state())
        bad = synth.clean(w, 0, GRAD, 8, "cuda").clone()
        bad[2, 7, 100] = float("inf")
        s, f = gv.verify(bad, GRAD)
        torch.cuda.synchronize()
        f = f.cpu().numpy().view(np.uint32)
        assert f[0] & sb.FLAG_NONFINITE and f[3] & sb.FLAG_NONFINITE and not (f[0] & sb.FLAG_COMMITTED)
        st = parse_blob(gv.sentinel_export_state(), w.B, w.T, w.d, 100)
        st0 = parse_blob(before, w.B, w.T, w.d, 100)
        assert np.array_equal(st["kinds"][GRAD]["m"], st0["kinds"][GRAD]["m"])     # the reference did not move
        blobs.append(bytes(gv.sentinel_export_state()))
        gv.close()
    assert blobs[0] == blobs[1]
