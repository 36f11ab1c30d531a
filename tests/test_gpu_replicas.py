"""GPU parity of the multi-worker iteration (worker loop of Alg. 2 / Alg. 3, pooled history,
>50% rule, Eq. 1 with the mean over the clean workers) against the float64 oracle."""
import numpy as np
import pytest
import torch

from helpers import (UNIT_BITS, assert_scores_close, near_threshold, oracle_to_blob, parse_blob,
                     whole_step_k_events)
from paper_2603_03592_b200 import synth

pytestmark = pytest.mark.gpu
ACT, GRAD = 0, 1


@pytest.fixture(scope="module")
def sb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_03592_b200 import binding
    binding.lib()
    return binding


def pair(sb, oracle_mod, w, R, **kw):
    names = {"l": "window_steps", "c": "ban_violations", "t_forgiveness": "forgiveness_steps"}
    gv = sb.Verifier(w.B, w.T, w.d, n_workers=R, **{names.get(k, k): v for k, v in kw.items()})
    params = oracle_mod.Params(B=w.B, T=w.T, d=w.d, R=R, **kw)
    return gv, oracle_mod.Verifier(params), params


def inputs(w, R, kind, t, scale=None):
    xs = [synth.clean(w, r, kind, t, "cuda") for r in range(R)]
    for r, c in (scale or {}).items():
        xs[r] = (xs[r].float() * c).to(torch.bfloat16)
    return xs


def step_both(gv, ov, xs, kind, warmup=False):
    gs, gf = gv.step_replicas(xs, kind, warmup)
    os_, of, n = ov.step_replicas([synth.bits(x) for x in xs], kind, warmup)
    torch.cuda.synchronize()
    return gs.cpu().numpy(), gf.cpu().numpy().view(np.uint32), os_, of, n


def check_state(gv, ov, params, kinds=(ACT, GRAD)):
    st = parse_blob(gv.sentinel_export_state(), params.B, params.T, params.d, params.l, params.R)
    for r in range(params.R):
        assert tuple(int(v) for v in st["workers"][:, r]) == ov.worker_counters(r), r
        assert gv.sentinel_get_worker_counters(r) == ov.worker_counters(r)
    for kind in kinds:
        ks = st["kinds"][kind]
        m_ref = ov.ema(kind)
        assert np.max(np.abs(ks["m"].astype(np.float64) - m_ref)) <= 1e-5 * max(float(np.abs(m_ref).max()), 1e-30)
        assert ks["steps"] == ov.steps(kind)
        for L in range(2):
            for i in range(ov.nm):
                href = ov.history(kind, L, i)
                assert ks["hist"][L][i].size == href.size
                floor = 1e-3 * (np.abs(href).mean() if i in (0, 3) and href.size else 1.0)
                assert np.all(np.abs(ks["hist"][L][i] - href) <= 1e-3 * np.maximum(np.abs(href), floor))
        gt, gvalid = gv.sentinel_get_thresholds(kind)
        ot, ovalid = ov.thresholds(kind)
        assert np.array_equal(gvalid, ovalid)
        for L in range(2):
            for i in range(ov.nm):
                if ovalid[L, i]:
                    assert gt[L, i, 3] == pytest.approx(ot[L, i, 3], rel=1e-12)


@pytest.mark.parametrize("shape,R", [((3, 12, 264), 4), ((2, 40, 1024), 5), ((4, 6, 64), 16)],
                         ids=["3x12x264_R4", "2x40x1024_R5", "4x6x64_R16"])
def test_iterations_in_lockstep(sb, oracle_mod, shape, R):
    """Warm-up, clean iterations, one tainted worker, a majority of flagged workers, a worker
    that gets banned and is then skipped -- scores, flags, counters, histories, multipliers and
    the reference after every phase."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "replicas", *shape)
    gv, ov, params = pair(sb, oracle_mod, w, R, l=5, c=2)
    script = [("warm", {})] * 8 + [("verify", {})] * 3 + [("verify", {1: 6.0})] + [("verify", {})] + \
             [("verify", {r: 3.0 for r in range(R // 2 + 1)})] + [("verify", {1: 6.0})] + [("verify", {})] * 2
    k_events, near_events = 0, 0
    for kind in (ACT, GRAD):
        for t, (what, scale) in enumerate(script):
            xs = inputs(w, R, kind, t, scale)
            thr, valid = ov.thresholds(kind)
            gs, gf, os_, of, n = step_both(gv, ov, xs, kind, warmup=(what == "warm"))
            for r in range(R):
                x_scale = float(xs[r].float().abs().mean())
                assert_scores_close(gs[r], os_[r], x_scale, "kind %d step %d worker %d" % (kind, t, r))
            if what == "warm":
                assert np.array_equal(gf & ~np.uint32(UNIT_BITS), of & ~np.uint32(UNIT_BITS))
                continue
            if not np.array_equal(gf, of):
                for r in range(R):
                    near = near_threshold(os_[r], thr, valid, w.B)
                    assert np.all(near[((gf[r] ^ of[r]) & UNIT_BITS) != 0]), (t, r, gf[r], of[r])
                near_events += 1
                gv.sentinel_import_state(oracle_to_blob(ov, params))
            if scale and len(scale) > 1:
                assert np.all(of[:, 0] & sb.FLAG_NATURAL_SHIFT)
            ev = whole_step_k_events(*gv.sentinel_get_thresholds(kind), *ov.thresholds(kind), params, kind)
            if ev:                                          # an entry sat on a fence: re-align
                k_events += ev
                gv.sentinel_import_state(oracle_to_blob(ov, params))
        check_state(gv, ov, params, kinds=(kind,))
    assert ov.worker_counters(1)[2] == 1                    # worker 1 ended up banned
    print("re-alignments: %d near a bound, %d multiplier events" % (near_events, k_events))
    assert near_events <= 2 and k_events <= 4, (near_events, k_events)
    gv.close()


def test_full_width_rows(sb, oracle_mod):
    """Two workers at a stage-traffic width (d = 4096, several tiles per row)."""
    w = synth.scaled(synth.WORKLOADS["cfg3"], "replicas_wide", 2, 96, 4096)
    gv, ov, params = pair(sb, oracle_mod, w, 2)
    for t in range(6):
        xs = inputs(w, 2, ACT, t, {0: 5.0} if t == 5 else None)
        gs, gf, os_, of, n = step_both(gv, ov, xs, ACT, warmup=t < 4)
        for r in range(2):
            assert_scores_close(gs[r], os_[r], float(xs[r].float().abs().mean()), "wide %d %d" % (t, r))
        if t >= 4:
            assert np.array_equal(gf, of)
    check_state(gv, ov, params, kinds=(ACT,))
    gv.close()


def test_argument_checks(sb):
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(2, 4, 16, n_workers=17)
    assert e.value.code == sb.ERR_INVALID_ARG
    with pytest.raises(sb.SentinelError) as e:
        sb.Verifier(8, 4, 16, n_workers=8)                  # 100 * 8 * 9 > 4096
    assert e.value.code == sb.ERR_UNSUPPORTED
    v = sb.Verifier(2, 4, 16, n_workers=2)
    x = torch.zeros(2, 4, 16, dtype=torch.bfloat16, device="cuda")
    scores = torch.zeros(2, 3, 3, device="cuda")
    flags = torch.zeros(2, 3, dtype=torch.int32, device="cuda")
    L, s = sb.lib(), torch.cuda.current_stream().cuda_stream
    import ctypes as C
    good = (C.c_void_p * 2)(x.data_ptr(), x.data_ptr())
    bad = (C.c_void_p * 2)(x.data_ptr(), None)
    assert L.sentinel_verify_replicas(v._h, bad, 0, 2, 4, 16, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_INVALID_ARG
    assert L.sentinel_verify_replicas(v._h, None, 0, 2, 4, 16, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_INVALID_ARG
    assert L.sentinel_verify_replicas(v._h, good, 0, 2, 4, 8, s, scores.data_ptr(), flags.data_ptr()) == sb.ERR_SHAPE_MISMATCH
    assert L.sentinel_verify_replicas(v._h, good, 0, 2, 4, 16, s, scores.data_ptr(), None) == sb.ERR_INVALID_ARG
    assert L.sentinel_reset_worker(v._h, 2, s) == sb.ERR_INVALID_ARG
    assert L.sentinel_verify_replicas(v._h, good, 0, 2, 4, 16, s, scores.data_ptr(), flags.data_ptr()) == sb.OK
    torch.cuda.synchronize()
    v.close()


# ---------------------------------------------------------------------------------------------
# workers tainted at another stage (Sec. 3.1, cascading effects; Alg. 2 / Alg. 3)

def step_both_tainted(gv, ov, xs, kind, mask):
    gx = [None if (mask >> r) & 1 else x for r, x in enumerate(xs)]
    gs, gf = gv.step_replicas(gx, kind, False, tainted_in=mask)
    os_, of, n = ov.step_replicas([None if x is None else synth.bits(x) for x in gx], kind, False, tainted_in=mask)
    torch.cuda.synchronize()
    return gs.cpu().numpy(), gf.cpu().numpy().view(np.uint32), os_, of, n


@pytest.mark.parametrize("kind", [ACT, GRAD], ids=["act", "grad"])
def test_workers_tainted_elsewhere(sb, oracle_mod, kind):
    """Not collected, reported, out of the mean; for gradients part of the stage's tainted set
    (majority rule, verdict for Alg. 4), for activations not."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "tainted_in", 3, 24, 264)
    R = 4
    gv, ov, params = pair(sb, oracle_mod, w, R, l=6, c=2)
    for t in range(10):
        step_both(gv, ov, inputs(w, R, kind, t), kind, warmup=True)
    plan = [(0b0000, {}), (0b0010, {}), (0b1100, {0: 6.0}), (0b0001, {}), (0b0000, {3: 6.0}), (0b0000, {3: 6.0}),
            (0b1000, {}), (0b1111, {}), (0b0000, {})]
    near_events, k_events = 0, 0
    for t, (mask, scale) in enumerate(plan, start=10):
        xs = inputs(w, R, kind, t, scale)
        thr, valid = ov.thresholds(kind)
        gs, gf, os_, of, n = step_both_tainted(gv, ov, xs, kind, mask)
        for r in range(R):
            assert_scores_close(gs[r], os_[r], float(xs[r].float().abs().mean()), "step %d worker %d" % (t, r))
        if not np.array_equal(gf, of):
            for r in range(R):
                near = near_threshold(os_[r], thr, valid, w.B)
                assert np.all(near[((gf[r] ^ of[r]) & UNIT_BITS) != 0]), (t, r, gf[r], of[r])
            near_events += 1
            gv.sentinel_import_state(oracle_to_blob(ov, params))
        ev = whole_step_k_events(*gv.sentinel_get_thresholds(kind), *ov.thresholds(kind), params, kind)
        if ev:
            k_events += ev
            gv.sentinel_import_state(oracle_to_blob(ov, params))
        # the verdict Alg. 4 acts on
        probe = xs[0].clone()
        replaced = torch.zeros(1, dtype=torch.int32, device="cuda")
        gv.sentinel_replace_if_flagged(probe, kind, 0, replaced)
        torch.cuda.synchronize()
        assert bool(replaced.item()) == ov.replace_if_flagged(synth.bits(xs[0]), kind)[1], (t, mask)
        check_state(gv, ov, params, kinds=(kind,))
    assert ov.worker_counters(3)[2] == 1                    # banned on the way; its bit then changes nothing
    print("re-alignments: %d near a bound, %d multiplier events" % (near_events, k_events))
    assert near_events <= 2 and k_events <= 4, (near_events, k_events)
    gv.close()


def test_tainted_in_argument_checks(sb):
    gv = sb.Verifier(2, 8, 64, n_workers=3)
    x = torch.zeros(2, 8, 64, dtype=torch.bfloat16, device="cuda")
    s, f = torch.zeros(3, 3, 3, device="cuda"), torch.zeros(3, 3, dtype=torch.int32, device="cuda")
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_verify_replicas_tainted([x, x, x], ACT, 0b1000, s, f)     # worker 3 does not exist
    assert e.value.code == sb.ERR_INVALID_ARG
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_verify_replicas_tainted([x, None, x], ACT, 0b0000, s, f)  # collected, but no tensor
    assert e.value.code == sb.ERR_INVALID_ARG
    gv.sentinel_verify_replicas_tainted([x, None, x], ACT, 0b0010, s, f)
    torch.cuda.synchronize()
    assert int(f[1, 0].item()) & sb.FLAG_TAINTED_ELSEWHERE
    gv.close()


def test_skip_tainted_single_submission(sb, oracle_mod):
    w = synth.scaled(synth.WORKLOADS["cfg1"], "skip", 2, 16, 128)
    gv = sb.Verifier(w.B, w.T, w.d)
    ov = oracle_mod.Verifier(oracle_mod.Params(B=w.B, T=w.T, d=w.d))
    for t in range(14):
        x = synth.clean(w, 0, GRAD, t, "cuda")
        gv.update_reference(x, GRAD)
        ov.update_reference(synth.bits(x), GRAD)
    before = bytes(gv.sentinel_export_state())
    gv.sentinel_skip_tainted(GRAD)
    ov.skip_tainted(GRAD)
    st0 = parse_blob(before, w.B, w.T, w.d, 100)
    st1 = parse_blob(gv.sentinel_export_state(), w.B, w.T, w.d, 100)
    assert st1["kinds"][GRAD]["steps"] == st0["kinds"][GRAD]["steps"] + 1 == ov.steps(GRAD)
    assert np.array_equal(st1["kinds"][GRAD]["m"], st0["kinds"][GRAD]["m"])
    assert all(np.array_equal(a, b) for a, b in zip(st1["kinds"][GRAD]["hist"][0], st0["kinds"][GRAD]["hist"][0]))
    assert (st1["violations"], st1["clean_streak"], st1["banned"]) == ov.counters()
    g = synth.clean(w, 0, GRAD, 15, "cuda")
    out = g.clone()
    replaced = torch.zeros(1, dtype=torch.int32, device="cuda")
    gv.sentinel_replace_if_flagged(out, GRAD, 0, replaced)
    torch.cuda.synchronize()
    want, did = ov.replace_if_flagged(synth.bits(g), GRAD)
    assert did and replaced.item() == 1
    got = synth.bits(out)
    assert np.mean(got != want) <= 1e-3                     # fp32 reference vs float64, then one rounding
    gs, gf = gv.verify(g, GRAD)
    assert int(gf[0].item()) & sb.FLAG_COMMITTED
    gv.sentinel_replace_if_flagged(out, GRAD, 0, replaced)
    torch.cuda.synchronize()
    assert replaced.item() == 0
    gv.close()


@pytest.mark.parametrize("shape,R", [((3, 12, 264), 4), ((2, 20, 1024), 2), ((4, 6, 64), 7)],
                         ids=["3x12x264_R4", "2x20x1024_R2", "4x6x64_R7"])
def test_iterations_in_lockstep_with_a_bf16_reference(sb, oracle_mod, shape, R):
    """The fixed-mesh verifier (several workers per iteration) with the reference stored as bf16:
    warm-up, clean iterations (the mean written by the scoring launch), a tainted worker (the mean
    over the clean ones taken afterwards), a flagged majority; the stored reference agrees with the
    oracle's bit for bit after every iteration."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "replicas_bf16", *shape)
    gv, ov, params = pair(sb, oracle_mod, w, R, l=5, c=3, ema_bf16=1)
    script = [("warm", {})] * 6 + [("verify", {})] * 2 + [("verify", {1: 6.0})] + [("verify", {})] + \
             [("verify", {r: 3.0 for r in range(R // 2 + 1)})] + [("verify", {})]
    near_events, k_events = 0, 0
    for t, (what, scale) in enumerate(script):
        xs = inputs(w, R, ACT, t, scale)
        thr, valid = ov.thresholds(ACT)
        gs, gf, os_, of, n = step_both(gv, ov, xs, ACT, warmup=(what == "warm"))
        for r in range(R):
            assert_scores_close(gs[r], os_[r], float(xs[r].float().abs().mean()), "step %d worker %d" % (t, r))
        if what != "warm" and not np.array_equal(gf, of):
            for r in range(R):
                near = near_threshold(os_[r], thr, valid, w.B)
                assert np.all(near[((gf[r] ^ of[r]) & UNIT_BITS) != 0]), (t, r, gf[r], of[r])
            near_events += 1
            gv.sentinel_import_state(oracle_to_blob(ov, params))
        ev = whole_step_k_events(*gv.sentinel_get_thresholds(ACT), *ov.thresholds(ACT), params, ACT)
        if ev:
            k_events += ev
            gv.sentinel_import_state(oracle_to_blob(ov, params))
        st = parse_blob(gv.sentinel_export_state(), w.B, w.T, w.d, params.l, R)
        assert np.array_equal(st["kinds"][ACT]["m"].astype(np.float64), ov.ema(ACT)), t
    print("re-alignments: %d near a bound, %d multiplier events" % (near_events, k_events))
    assert near_events <= 2 and k_events <= 4, (near_events, k_events)
    gv.close()
