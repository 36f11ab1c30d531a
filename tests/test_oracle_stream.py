"""Pins for the oracle's stateful part: Eq. (1), the warm-up loop of Alg. 1, the per-submission
body of Alg. 2 / Alg. 3 and the violation counter of Sec. 3.1.  Expected values are closed
forms, hand-scripted sequences, or library routines applied to the recorded history."""
import numpy as np
import pytest
import torch

from paper_2603_03592_b200 import synth
from test_oracle_pins import from_bits, to_bits

ACT, GRAD = 0, 1


def make(oracle_mod, B=2, T=4, d=8, **kw):
    return oracle_mod.Verifier(oracle_mod.Params(B=B, T=T, d=d, **kw))


def test_ema_closed_form_for_identical_inputs(oracle_mod):
    """m_0 = 0 and t identical submissions x give m_t = (1 - beta^t) x (Eq. 1)."""
    rs = np.random.default_rng(1)
    v = make(oracle_mod)
    xb = to_bits(rs.normal(0, 1, (2, 4, 8)))
    x = from_bits(xb)
    assert np.all(v.ema(ACT) == 0.0)
    for t in range(1, 8):
        v.update_reference(xb, ACT)
        v.update_reference(xb, GRAD)
        assert v.ema(ACT) == pytest.approx((1 - 0.9 ** t) * x, rel=1e-13)
        assert v.ema(GRAD) == pytest.approx((1 - 0.8 ** t) * x, rel=1e-13)


def test_ema_is_the_weighted_sum_of_past_inputs(oracle_mod):
    rs = np.random.default_rng(2)
    v = make(oracle_mod, beta=(0.5, 0.25))
    xs = [to_bits(rs.normal(0, 1, (2, 4, 8))) for _ in range(5)]
    for xb in xs:
        v.update_reference(xb, GRAD)
    want = sum(0.75 * 0.25 ** (4 - i) * from_bits(xb) for i, xb in enumerate(xs))
    assert v.ema(GRAD) == pytest.approx(want, rel=1e-13, abs=1e-16)
    assert np.all(v.ema(ACT) == 0.0)                  # the two kinds have separate references


def test_beta_zero_keeps_the_last_submission(oracle_mod):
    rs = np.random.default_rng(3)
    v = make(oracle_mod, beta=(0.0, 0.0))
    for _ in range(3):
        xb = to_bits(rs.normal(0, 1, (2, 4, 8)))
        v.update_reference(xb, ACT)
        assert np.array_equal(v.ema(ACT), from_bits(xb))


def test_first_warmup_step_scores_against_the_zero_reference(oracle_mod):
    """m_0 = 0: L1 = mean|x|, L2 = 1 (z-score of a constant is zero), SFR = fraction non-zero."""
    rs = np.random.default_rng(4)
    v = make(oracle_mod)
    x = from_bits(to_bits(rs.normal(0, 1, (2, 4, 8))))
    x[0, 0, :3] = 0.0
    scores, bad = v.update_reference(to_bits(x), ACT)
    assert not bad
    units = [x] + [x[b] for b in range(2)]
    for r, u in enumerate(units):
        assert scores[r, 0] == pytest.approx(np.mean(np.abs(u)), rel=1e-13)
        assert scores[r, 1] == pytest.approx(1.0, rel=1e-12)
        assert scores[r, 2] == np.count_nonzero(u) / u.size
    # scores of a step are measured against the reference *before* that step's update
    scores2, _ = v.update_reference(to_bits(x), ACT)
    assert scores2[0, 0] == pytest.approx(np.mean(np.abs(x - 0.1 * x)), rel=1e-12)
    assert scores2[0, 2] == 0.0


def test_tensor_level_is_the_mean_of_equal_sized_samples(oracle_mod):
    rs = np.random.default_rng(5)
    v = make(oracle_mod, B=4, T=8, d=16)
    v.update_reference(to_bits(rs.normal(0, 1, (4, 8, 16))), ACT)
    scores, _ = v.update_reference(to_bits(rs.normal(0, 1, (4, 8, 16))), ACT)
    assert scores[0, 0] == pytest.approx(scores[1:, 0].mean(), rel=1e-13)
    assert scores[0, 2] == pytest.approx(scores[1:, 2].mean(), rel=1e-13)
    s = v.last_stats(ACT)
    assert s[0, 0] == pytest.approx(s[1:, 0].mean(), rel=1e-12, abs=1e-16)
    assert s[0, 2] ** 2 == pytest.approx(np.sum(s[1:, 2] ** 2), rel=1e-13)


def test_warmup_history_and_thresholds(oracle_mod):
    """Every warm-up deviation joins the window (oldest leaves after l entries per unit) and the
    stored thresholds are Alg. 5 applied to that window with the multiplier carried over."""
    rs = np.random.default_rng(6)
    B, l = 3, 5
    v = make(oracle_mod, B=B, T=4, d=8, l=l)
    rec = [[], []]
    k = [[1.5] * 3, [1.5] * 3]
    for t in range(9):
        scores, _ = v.update_reference(to_bits(rs.normal(0, 1, (B, 4, 8))), ACT)
        rec[0].append(scores[0])
        rec[1].extend(scores[1:])
        thr, valid = v.thresholds(ACT)
        assert valid.all()
        for L, cap in ((0, l), (1, l * B)):
            for i in range(3):
                want_hist = np.array(rec[L])[-cap:, i]
                assert np.array_equal(v.history(ACT, L, i), want_hist)
                want, _ = oracle_mod.adaptive_iqr(want_hist, k[L][i], 1e-4, 10, 1.1, 0.9, 0.15, 1e-3)
                assert np.array_equal(thr[L, i], want)
                q = np.percentile(want_hist, [25, 50, 75])
                assert thr[L, i, :3] == pytest.approx(q, rel=1e-13)
                k[L][i] = want[3]
    tg, vg = v.thresholds(GRAD)
    assert not vg.any() and np.all(tg[:, :, 3] == 3.0)     # untouched kind keeps k0


def _warm(oracle_mod, w, n, **kw):
    v = oracle_mod.Verifier(oracle_mod.Params(B=w.B, T=w.T, d=w.d, **kw))
    for t in range(n):
        for kind in (ACT, GRAD):
            v.update_reference(synth.bits(synth.clean(w, 0, kind, t)), kind)
    return v


@pytest.fixture(scope="module")
def small():
    return synth.scaled(synth.WORKLOADS["cfg1"], "cfg1_small", 8, 32, 128)


def test_clean_stream_raises_no_flags(oracle_mod, small):
    v = _warm(oracle_mod, small, 16)
    for t in range(16, 56):
        for kind in (ACT, GRAD):
            scores, flags, commit = v.verify(synth.bits(synth.clean(small, 0, kind, t)), kind)
            assert commit
            assert np.all((flags & 0xFFFF) == 0)
            assert flags[0] == oracle_mod.FLAG_COMMITTED
    assert v.counters() == (0, 40 * 2, 0)


def test_scaled_sample_is_flagged_and_reference_is_kept(oracle_mod, small):
    """Config-1 scenario: sample 3 multiplied by 10 after 16 clean warm-up microbatches."""
    v = _warm(oracle_mod, small, 16)
    clean = synth.clean(small, 0, ACT, 16)
    bad = synth.corrupt(small, clean, "scale_sample3", 0, ACT, 16)
    m_before = v.ema(ACT)
    hist_before = [v.history(ACT, L, 0).size for L in (0, 1)]
    clean_scores, _ = oracle_mod.distance(synth.bits(clean)[3], m_before[3])[:2]
    scores, flags, commit = v.verify(synth.bits(bad), ACT)
    assert not commit and not (flags[0] & oracle_mod.FLAG_COMMITTED)
    assert flags[4] & oracle_mod.FLAG_L1                      # row 1+3
    assert scores[4, 0] > 5 * clean_scores[0]                 # L1 grows about tenfold
    others = [r for r in range(1, 9) if r != 4]
    assert np.all(flags[others] == 0)
    assert np.array_equal(v.ema(ACT), m_before)               # flagged => EMA not updated
    # flagged units stay out of the history, clean samples still join it
    n_flagged = int(np.count_nonzero(flags[1:] & 0xFFFF))
    assert v.history(ACT, 1, 0).size == min(hist_before[1] + 8 - n_flagged, 100 * 8)
    level0_flagged = bool(flags[0] & 0xFFFF)
    assert v.history(ACT, 0, 0).size == hist_before[0] + (0 if level0_flagged else 1)
    assert v.counters()[0] == 1


def test_gradient_sign_flip_is_statistically_invisible(oracle_mod, small):
    """The paper's tables show a 0% detection of gradients multiplied by -1: against an EMA of
    independent zero-mean gradients, -g has the same three scores up to sampling noise."""
    v = _warm(oracle_mod, small, 16)
    g = synth.clean(small, 0, GRAD, 16)
    m = v.ema(GRAD)
    a, _, _ = oracle_mod.distance(synth.bits(g), m)
    b, _, _ = oracle_mod.distance(synth.bits(-g), m)
    assert b == pytest.approx(a, rel=0.02)
    _, flags, commit = v.verify(synth.bits(-g), GRAD)
    assert commit and np.all((flags & 0xFFFF) == 0)


def test_violation_counter_ban_and_forgiveness(oracle_mod, small):
    v = _warm(oracle_mod, small, 16, c=3, t_forgiveness=4)
    step = [16]

    def send(corrupt):
        x = synth.clean(small, 0, ACT, step[0])
        if corrupt:
            x = (x.float() * 3.0).to(torch.bfloat16)         # mild: caught, far from severe
        step[0] += 1
        return v.verify(synth.bits(x), ACT)

    _, f, c = send(True)
    assert not c and v.counters() == (1, 0, 0) and not (f[0] & oracle_mod.FLAG_SEVERE)
    for i in range(3):
        _, f, c = send(False)
        assert c and v.counters() == (1, i + 1, 0)
    send(False)                                               # 4th clean step: forgiven
    assert v.counters() == (0, 0, 0)
    for i in range(4):
        send(False)
    assert v.counters() == (0, 0, 0)                          # never below zero
    send(True); send(False); send(True)
    assert v.counters() == (2, 0, 0)                          # a clean step does not reset v
    _, f, _ = send(True)
    assert v.counters() == (3, 0, 1) and (f[0] & oracle_mod.FLAG_BANNED)
    _, f, c = send(False)
    assert c and (f[0] & oracle_mod.FLAG_BANNED)              # the ban is sticky ...
    v.reset_worker()
    _, f, _ = send(False)
    assert not (f[0] & oracle_mod.FLAG_BANNED) and v.counters() == (0, 1, 0)   # ... until reset


def test_severe_deviation_bans_at_once(oracle_mod, small):
    v = _warm(oracle_mod, small, 16)
    x = (synth.clean(small, 0, ACT, 16).float() * 4096.0).to(torch.bfloat16)
    thr, _ = v.thresholds(ACT)
    scores, flags, commit = v.verify(synth.bits(x), ACT)
    assert abs(scores[0, 0] - thr[0, 0, 1]) >= 100 * (thr[0, 0, 5] - thr[0, 0, 1])
    assert (flags[0] & oracle_mod.FLAG_SEVERE) and (flags[0] & oracle_mod.FLAG_BANNED)
    assert v.counters() == (1, 0, 1)


def test_verify_without_warmup_flags_nothing(oracle_mod):
    rs = np.random.default_rng(8)
    v = make(oracle_mod)
    xb = to_bits(rs.normal(0, 1, (2, 4, 8)))
    scores, flags, commit = v.verify(xb, ACT)
    assert commit
    assert flags[0] == (oracle_mod.FLAG_COMMITTED | oracle_mod.FLAG_NO_THRESHOLDS)
    assert np.all(flags[1:] == 0)
    assert v.history(ACT, 0, 0).size == 1 and v.history(ACT, 1, 0).size == 2
    assert v.ema(ACT) == pytest.approx(0.1 * from_bits(xb), rel=1e-13)
    _, flags, _ = v.verify(xb, ACT)
    assert not (flags[0] & oracle_mod.FLAG_NO_THRESHOLDS)


def test_non_finite_submission_is_a_violation_and_changes_nothing(oracle_mod, small):
    v = _warm(oracle_mod, small, 4)
    x = synth.clean(small, 0, ACT, 4).float()
    x[2, 1, 5] = float("nan")
    m0, h0 = v.ema(ACT), v.history(ACT, 1, 0).size
    scores, flags, commit = v.verify(synth.bits(x.to(torch.bfloat16)), ACT)
    assert not commit
    assert flags[0] & oracle_mod.FLAG_NONFINITE and flags[3] & oracle_mod.FLAG_NONFINITE
    assert np.all(np.isnan(scores[0])) and np.all(np.isnan(scores[3]))
    assert np.all(np.isfinite(scores[[1, 2, 4, 5, 6, 7, 8]]))
    assert np.array_equal(v.ema(ACT), m0)
    assert v.history(ACT, 1, 0).size == h0 + 7 and v.counters()[0] == 1
    # warm-up refuses it outright
    s, bad = v.update_reference(synth.bits(x.to(torch.bfloat16)), ACT)
    assert bad and np.array_equal(v.ema(ACT), m0) and v.history(ACT, 1, 0).size == h0 + 7


def test_metric_mask_limits_which_metrics_may_flag(oracle_mod, small):
    x = (synth.clean(small, 0, ACT, 16).float() * 3.0).to(torch.bfloat16)
    v = _warm(oracle_mod, small, 16)
    _, f_all, _ = v.verify(synth.bits(x), ACT)
    assert f_all[0] & oracle_mod.FLAG_L1
    v = _warm(oracle_mod, small, 16, metric_mask=0b110)       # L1 switched off
    scores, f, commit = v.verify(synth.bits(x), ACT)
    assert not np.any(f & oracle_mod.FLAG_L1)
    # scaling by 3 leaves the z-scored distance and the signs alone, so nothing else fires
    assert commit and np.all((f & 0xFFFF) == 0)


def test_gradient_replacement_follows_the_last_verdict(oracle_mod, small):
    """Alg. 4: a flagged submission is replaced by the reference m_{t-1} (or zeros); a clean one
    is forwarded untouched."""
    v = _warm(oracle_mod, small, 16)
    g = synth.clean(small, 0, GRAD, 16)
    _, flags, commit = v.verify(synth.bits(g), GRAD)
    assert commit
    out, did = v.replace_if_flagged(synth.bits(g), GRAD)
    assert not did and np.array_equal(out, synth.bits(g))
    bad = (synth.clean(small, 0, GRAD, 17).float() * 50.0).to(torch.bfloat16)
    m_before = v.ema(GRAD)
    _, flags, commit = v.verify(synth.bits(bad), GRAD)
    assert not commit
    out, did = v.replace_if_flagged(synth.bits(bad), GRAD)
    assert did
    got = from_bits(out)
    assert np.all(np.abs(got - m_before) <= 2.0 ** -8 * np.abs(m_before) + 1e-45)   # half an ulp of bf16
    zeros, did = v.replace_if_flagged(synth.bits(bad), GRAD, fill=1)
    assert did and not zeros.any()
    # the verdict is per kind: the activation side was never flagged
    a = synth.clean(small, 0, ACT, 16)
    out, did = v.replace_if_flagged(synth.bits(a), ACT)
    assert not did


# ---------------------------------------------------------------- several workers per stage

def _replica_inputs(w, R, step, kind=ACT):
    return [synth.clean(w, r, kind, step) for r in range(R)]      # boundary index = worker index


def test_replica_warmup_is_the_mean_over_workers(oracle_mod, small):
    """Eq. 1: m_t = beta m_{t-1} + (1-beta) * (1/d_s) sum_r x^(r); the pooled window holds the
    deviations of all workers (l*R entries per level-0 metric)."""
    R = 3
    v = oracle_mod.Verifier(oracle_mod.Params(B=small.B, T=small.T, d=small.d, R=R, l=4))
    xs = _replica_inputs(small, R, 0)
    scores, flags, n = v.step_replicas([synth.bits(x) for x in xs], ACT, warmup=True)
    assert n == R and np.all(flags == oracle_mod.FLAG_COMMITTED * (np.arange(1 + small.B) == 0))
    mean = sum(from_bits(synth.bits(x)) for x in xs) / R
    assert v.ema(ACT) == pytest.approx(0.1 * mean, rel=1e-13, abs=1e-15)
    for r in range(R):                       # every worker is scored against the same m_{t-1} = 0
        assert scores[r, 0, 0] == pytest.approx(np.mean(np.abs(from_bits(synth.bits(xs[r])))), rel=1e-13)
    assert v.history(ACT, 0, 0).size == R and v.history(ACT, 1, 0).size == R * small.B
    for t in range(1, 7):
        v.step_replicas([synth.bits(x) for x in _replica_inputs(small, R, t)], ACT, warmup=True)
    assert v.history(ACT, 0, 0).size == 4 * R and v.history(ACT, 1, 0).size == 4 * R * small.B


def test_one_worker_is_the_single_submission_path(oracle_mod, small):
    """On clean traffic the worker loop with one worker is the single-submission call.  (On a
    flagged step it is not: one flagged worker out of one is a majority, so the >50% rule of
    Alg. 2 clears the taint, whereas the per-trainer form has no such rule.)"""
    a = oracle_mod.Verifier(oracle_mod.Params(B=small.B, T=small.T, d=small.d))
    b = oracle_mod.Verifier(oracle_mod.Params(B=small.B, T=small.T, d=small.d, R=1))
    for t in range(12):
        xb = synth.bits(synth.clean(small, 0, GRAD, t))
        if t < 6:
            sa, _ = a.update_reference(xb, GRAD)
            sb_, fb, _ = b.step_replicas([xb], GRAD, warmup=True)
        else:
            sa, fa, _ = a.verify(xb, GRAD)
            sb_, fb, _ = b.step_replicas([xb], GRAD)
            assert np.array_equal(fa, fb[0])
        assert np.array_equal(sa, sb_[0])
        assert np.array_equal(a.ema(GRAD), b.ema(GRAD))
        assert a.counters() == b.worker_counters(0)
        ta, tb = a.thresholds(GRAD), b.thresholds(GRAD)
        assert np.array_equal(ta[0], tb[0])


def _warm_replicas(oracle_mod, w, R, n, **kw):
    v = oracle_mod.Verifier(oracle_mod.Params(B=w.B, T=w.T, d=w.d, R=R, **kw))
    for t in range(n):
        v.step_replicas([synth.bits(x) for x in _replica_inputs(w, R, t)], ACT, warmup=True)
    return v


def test_tainted_worker_is_left_out_of_the_mean(oracle_mod, small):
    R = 4
    v = _warm_replicas(oracle_mod, small, R, 12)
    xs = _replica_inputs(small, R, 12)
    xs[2] = (xs[2].float() * 6).to(torch.bfloat16)
    m0 = v.ema(ACT)
    scores, flags, n = v.step_replicas([synth.bits(x) for x in xs], ACT)
    assert n == 3
    assert flags[2, 0] & 0xFFFF and not (flags[2, 0] & oracle_mod.FLAG_COMMITTED)
    for r in (0, 1, 3):
        assert flags[r, 0] == oracle_mod.FLAG_COMMITTED and not np.any(flags[r, 1:])
    mean = sum(from_bits(synth.bits(xs[r])) for r in (0, 1, 3)) / 3
    assert v.ema(ACT) == pytest.approx(0.9 * m0 + 0.1 * mean, rel=1e-12, abs=1e-15)
    assert [v.worker_counters(r)[0] for r in range(R)] == [0, 0, 1, 0]


def test_majority_flagged_is_a_natural_shift(oracle_mod, small):
    """More than half of the workers flagged: the taint set is cleared, every submission enters
    the EMA, but the violation counters have already moved (Alg. 2)."""
    R = 4
    v = _warm_replicas(oracle_mod, small, R, 12)
    xs = _replica_inputs(small, R, 12)
    for r in (0, 1, 3):
        xs[r] = (xs[r].float() * 3).to(torch.bfloat16)
    m0 = v.ema(ACT)
    h0 = v.history(ACT, 0, 0).size
    scores, flags, n = v.step_replicas([synth.bits(x) for x in xs], ACT)
    assert n == 4 and np.all(flags[:, 0] & oracle_mod.FLAG_NATURAL_SHIFT)
    assert np.all(flags[:, 0] & oracle_mod.FLAG_COMMITTED)
    mean = sum(from_bits(synth.bits(x)) for x in xs) / 4
    assert v.ema(ACT) == pytest.approx(0.9 * m0 + 0.1 * mean, rel=1e-12, abs=1e-15)
    assert [v.worker_counters(r)[0] for r in range(R)] == [1, 1, 0, 1]
    assert v.history(ACT, 0, 0).size == h0 + 1          # only the unflagged worker's deviation joined
    # exactly half flagged is not a majority
    v = _warm_replicas(oracle_mod, small, R, 12)
    xs = _replica_inputs(small, R, 12)
    for r in (0, 1):
        xs[r] = (xs[r].float() * 3).to(torch.bfloat16)
    _, flags, n = v.step_replicas([synth.bits(x) for x in xs], ACT)
    assert n == 2 and not np.any(flags[:, 0] & oracle_mod.FLAG_NATURAL_SHIFT)


def test_banned_worker_is_no_longer_collected(oracle_mod, small):
    R = 3
    v = _warm_replicas(oracle_mod, small, R, 12, c=2)
    for t in range(12, 14):
        xs = _replica_inputs(small, R, t)
        xs[1] = (xs[1].float() * 6).to(torch.bfloat16)
        _, flags, n = v.step_replicas([synth.bits(x) for x in xs], ACT)
        assert n == 2
    assert v.worker_counters(1) == (2, 0, 1) and flags[1, 0] & oracle_mod.FLAG_BANNED
    xs = _replica_inputs(small, R, 14)
    m0 = v.ema(ACT)
    scores, flags, n = v.step_replicas([synth.bits(x) for x in xs], ACT)
    assert n == 2 and np.all(np.isnan(scores[1])) and flags[1, 0] == oracle_mod.FLAG_BANNED
    mean = sum(from_bits(synth.bits(xs[r])) for r in (0, 2)) / 2
    assert v.ema(ACT) == pytest.approx(0.9 * m0 + 0.1 * mean, rel=1e-12, abs=1e-15)
    # with one of three banned, one flagged worker of the remaining two is exactly half: no shift
    xs = _replica_inputs(small, R, 15)
    xs[0] = (xs[0].float() * 6).to(torch.bfloat16)
    _, flags, n = v.step_replicas([synth.bits(x) for x in xs], ACT)
    assert n == 1 and not (flags[0, 0] & oracle_mod.FLAG_NATURAL_SHIFT)


def _warm_replicas_kind(oracle_mod, w, R, n, kind, **kw):
    v = oracle_mod.Verifier(oracle_mod.Params(B=w.B, T=w.T, d=w.d, R=R, **kw))
    for t in range(n):
        v.step_replicas([synth.bits(x) for x in _replica_inputs(w, R, t, kind)], kind, warmup=True)
    return v


@pytest.mark.parametrize("kind", [ACT, GRAD])
def test_worker_tainted_at_another_stage_is_not_collected(oracle_mod, small, kind):
    """Sec. 3.1 (cascading effects), Alg. 2 / Alg. 3: no metrics, no counter, no history entry for
    such a worker, and the mean of Eq. 1 runs over the others; its tensor is never touched."""
    R = 4
    v = _warm_replicas_kind(oracle_mod, small, R, 12, kind)
    xs = _replica_inputs(small, R, 12, kind)
    m0 = v.ema(kind)
    h0 = [v.history(kind, L, 0).size for L in (0, 1)]
    bits = [synth.bits(x) for x in xs]
    bits[1] = None                                          # not even supplied
    scores, flags, n = v.step_replicas(bits, kind, tainted_in=0b0010)
    assert n == 3 and np.all(np.isnan(scores[1]))
    assert flags[1, 0] == oracle_mod.FLAG_TAINTED_ELSEWHERE and not np.any(flags[1, 1:])
    for r in (0, 2, 3):
        assert flags[r, 0] == oracle_mod.FLAG_COMMITTED
    mean = sum(from_bits(synth.bits(xs[r])) for r in (0, 2, 3)) / 3
    assert v.ema(kind) == pytest.approx((0.9 if kind == ACT else 0.8) * m0 + (0.1 if kind == ACT else 0.2) * mean,
                                        rel=1e-12, abs=1e-15 if kind == ACT else 1e-18)
    assert v.worker_counters(1) == (0, 0, 0)                # neither a violation nor a clean step
    assert v.worker_counters(0) == (0, 1, 0)
    assert [v.history(kind, L, 0).size for L in (0, 1)] == [min(h0[0] + 3, 100 * R), min(h0[1] + 3 * small.B, 100 * R * small.B)]
    # Alg. 4 needs the verdict: for gradients the stage's tainted set holds the worker (Alg. 3)
    out, did = v.replace_if_flagged(synth.bits(xs[1]), kind)
    assert did == (kind == GRAD)


def test_workers_tainted_elsewhere_count_towards_the_majority_for_gradients_only(oracle_mod, small):
    """Alg. 3 adds a worker tainted downstream to the stage's tainted set, Alg. 2 leaves a worker
    tainted upstream out of its loop: with 2 of 4 workers tainted elsewhere and a third flagged
    here, the gradient side sees 3 of 4 (a natural shift: the flagged submission enters the EMA
    after all), the activation side 1 of 4."""
    R = 4
    for kind, beta in ((GRAD, 0.8), (ACT, 0.9)):
        v = _warm_replicas_kind(oracle_mod, small, R, 12, kind)
        xs = _replica_inputs(small, R, 12, kind)
        xs[0] = (xs[0].float() * 6).to(torch.bfloat16)
        m0 = v.ema(kind)
        scores, flags, n = v.step_replicas([synth.bits(x) for x in xs], kind, tainted_in=0b1100)
        assert flags[0, 0] & 0xFFFF and v.worker_counters(0)[0] == 1
        natural = bool(flags[0, 0] & oracle_mod.FLAG_NATURAL_SHIFT)
        assert natural == (kind == GRAD)
        clean = (0, 1) if natural else (1,)
        assert n == len(clean)
        mean = sum(from_bits(synth.bits(xs[r])) for r in clean) / len(clean)
        assert v.ema(kind) == pytest.approx(beta * m0 + (1 - beta) * mean, rel=1e-12, abs=1e-15 if kind == ACT else 1e-18)
        for r in (2, 3):                                    # never part of the mean, shift or not
            assert flags[r, 0] & oracle_mod.FLAG_TAINTED_ELSEWHERE and not (flags[r, 0] & oracle_mod.FLAG_COMMITTED)


def test_tainted_elsewhere_is_ignored_for_banned_workers_and_in_warmup(oracle_mod, small):
    R = 3
    v = _warm_replicas(oracle_mod, small, R, 12, c=1)
    xs = _replica_inputs(small, R, 12)
    xs[1] = (xs[1].float() * 6).to(torch.bfloat16)
    v.step_replicas([synth.bits(x) for x in xs], ACT)
    assert v.worker_counters(1)[2] == 1
    _, flags, n = v.step_replicas([synth.bits(x) for x in _replica_inputs(small, R, 13)], ACT, tainted_in=0b010)
    assert flags[1, 0] == oracle_mod.FLAG_BANNED and n == 2
    _, flags, n = v.step_replicas([synth.bits(x) for x in _replica_inputs(small, R, 14)], ACT, warmup=True,
                                  tainted_in=0b001)
    assert n == 3 and not np.any(flags & oracle_mod.FLAG_TAINTED_ELSEWHERE)


def test_skip_tainted_counts_the_step_and_asks_for_replacement(oracle_mod, small):
    v = _warm(oracle_mod, small, 2)
    for t in range(14):
        v.update_reference(synth.bits(synth.clean(small, 0, GRAD, t)), GRAD)
    m0, h0, c0, s0 = v.ema(GRAD), v.history(GRAD, 0, 0).copy(), v.counters(), v.steps(GRAD)
    v.skip_tainted(GRAD)
    assert v.steps(GRAD) == s0 + 1 and v.counters() == c0
    assert np.array_equal(v.ema(GRAD), m0) and np.array_equal(v.history(GRAD, 0, 0), h0)
    g = synth.clean(small, 0, GRAD, 15)
    out, did = v.replace_if_flagged(synth.bits(g), GRAD)
    assert did and np.all(np.abs(from_bits(out) - m0) <= 2.0 ** -8 * np.abs(m0) + 1e-45)
    assert v.verify(synth.bits(g), GRAD)[2]                 # a clean step clears the verdict
    assert not v.replace_if_flagged(synth.bits(g), GRAD)[1]


# ---------------------------------------------------------------------------------------------
# the sliced Wasserstein distance as a fourth member of the metric set M (Sec. 3.1)

def _directions(rs, L, d):
    u = rs.normal(0, 1, (L, d))
    return to_bits(u / np.linalg.norm(u, axis=1, keepdims=True))


def _sw_numpy(x, m, u):
    """mean over directions of W1 between the projected token clouds, from scipy's 1-D W1."""
    import scipy.stats
    return float(np.mean([scipy.stats.wasserstein_distance(x @ ul, m @ ul) for ul in u]))


def test_fourth_metric_is_the_sliced_wasserstein_distance_of_every_unit(oracle_mod):
    """With directions set, column 3 of the scores is SW(unit, m_{t-1}): B*T tokens for the whole
    tensor, T tokens for a sample; the other three columns are what they were without it."""
    rs = np.random.default_rng(21)
    B, T, d, L = 3, 6, 8, 4
    ub = _directions(rs, L, d)
    u = from_bits(ub)
    v, v3 = make(oracle_mod, B=B, T=T, d=d), make(oracle_mod, B=B, T=T, d=d)
    v.set_directions(ub)
    for t in range(6):
        xb = to_bits(rs.normal(0.3, 1, (B, T, d)))
        m = v.ema(ACT).copy()
        if t < 4:
            scores, _ = v.update_reference(xb, ACT)
            scores3, _ = v3.update_reference(xb, ACT)
        else:
            scores, _, _ = v.verify(xb, ACT)
            scores3, _, _ = v3.verify(xb, ACT)
        assert scores.shape == (1 + B, 4) and scores3.shape == (1 + B, 3)
        assert np.array_equal(scores[:, :3], scores3)
        x = from_bits(xb)
        assert scores[0, 3] == pytest.approx(_sw_numpy(x.reshape(-1, d), m.reshape(-1, d), u), rel=1e-12)
        for b in range(B):
            assert scores[1 + b, 3] == pytest.approx(_sw_numpy(x[b], m[b], u), rel=1e-12)


def test_fourth_metric_has_its_own_history_and_thresholds(oracle_mod):
    rs = np.random.default_rng(22)
    B, l = 2, 4
    v = make(oracle_mod, B=B, T=5, d=8, l=l)
    v.set_directions(_directions(rs, 4, 8))
    rec = [[], []]
    k = [1.5, 1.5]
    for t in range(7):
        scores, _ = v.update_reference(to_bits(rs.normal(0, 1, (B, 5, 8))), ACT)
        rec[0].append(scores[0, 3])
        rec[1].extend(scores[1:, 3])
        thr, valid = v.thresholds(ACT)
        assert thr.shape == (2, 4, 6) and valid.all()
        for L, cap in ((0, l), (1, l * B)):
            want_hist = np.array(rec[L])[-cap:]
            assert np.array_equal(v.history(ACT, L, 3), want_hist)
            want, _ = oracle_mod.adaptive_iqr(want_hist, k[L], 1e-4, 10, 1.1, 0.9, 0.15, 1e-3)
            assert np.array_equal(thr[L, 3], want)
            k[L] = want[3]


def test_a_shift_seen_only_by_the_sliced_wasserstein_distance_is_flagged(oracle_mod):
    """A verifier that may flag on SW alone (metric_mask = 8): a submission whose tokens are
    spread three times as wide along every direction moves SW far outside its window and raises bit 3,
    nothing else; the EMA stays.  The same verifier without directions sees no metric at all."""
    rs = np.random.default_rng(23)
    B, T, d = 2, 32, 16
    v = make(oracle_mod, B=B, T=T, d=d, metric_mask=8)
    v.set_directions(_directions(rs, 8, d))
    base = rs.normal(0, 1, (B, T, d))
    for t in range(12):
        v.update_reference(to_bits(base + 0.05 * rs.normal(0, 1, (B, T, d))), ACT)
    ok, f_ok, commit = v.verify(to_bits(base + 0.05 * rs.normal(0, 1, (B, T, d))), ACT)
    assert commit and not (f_ok & oracle_mod.METRIC_BITS).any()
    m0 = v.ema(ACT).copy()
    scores, flags, commit = v.verify(to_bits(3.0 * base), ACT)
    assert not commit and np.array_equal(v.ema(ACT), m0)
    assert np.all(flags & oracle_mod.METRIC_BITS == oracle_mod.FLAG_SW)
    assert np.all(scores[:, 3] > 5 * ok[:, 3])
    thr, _ = v.thresholds(ACT)
    assert np.all(scores[0, 3] > thr[0, 3, 5]) and np.all(scores[1:, 3] > thr[1, 3, 5])


def test_directions_are_refused_after_the_first_step(oracle_mod):
    rs = np.random.default_rng(24)
    v = make(oracle_mod)
    v.update_reference(to_bits(rs.normal(0, 1, (2, 4, 8))), GRAD)
    with pytest.raises(RuntimeError):
        v.set_directions(_directions(rs, 4, 8))


# ---------------------------------------------------------------------------------------------
# the reference stored as bf16

def _as_bf16_f32(a32):
    """float32 -> nearest bf16 (ties to even) -> float32, by torch's conversion."""
    return torch.from_numpy(np.ascontiguousarray(a32, dtype=np.float32)).to(torch.bfloat16).float().numpy()


def test_bf16_reference_is_the_single_precision_update_rounded_once(oracle_mod):
    """m_t = bf16(fma(beta, m_{t-1}, (1-beta)*x)) in float32.  Expected values: the product and
    the fused sum formed exactly in float64 (24-bit times 8-bit and 24-bit operands) and rounded
    to float32, then torch's float32 -> bfloat16 conversion."""
    rs = np.random.default_rng(31)
    v = make(oracle_mod, B=2, T=6, d=16, ema_bf16=1)
    beta32, omb32 = np.float32(0.9), np.float32(1.0 - 0.9)
    m = np.zeros((2, 6, 16), dtype=np.float32)
    for t in range(12):
        xb = to_bits(rs.normal(0.2, 1.5, (2, 6, 16)))
        x32 = from_bits(xb).astype(np.float32)
        v.update_reference(xb, ACT)
        prod = (omb32.astype(np.float64) * x32.astype(np.float64)).astype(np.float32)
        fused = (np.float64(beta32) * m.astype(np.float64) + prod.astype(np.float64)).astype(np.float32)
        m = _as_bf16_f32(fused)
        got = v.ema(ACT)
        assert np.array_equal(got, m.astype(np.float64)), t
    assert np.all(v.ema(GRAD) == 0.0)


def test_bf16_reference_scores_use_the_rounded_reference(oracle_mod):
    rs = np.random.default_rng(32)
    v = make(oracle_mod, B=2, T=4, d=8, ema_bf16=1)
    for t in range(5):
        v.update_reference(to_bits(rs.normal(0, 1, (2, 4, 8))), GRAD)
    m = v.ema(GRAD).copy()
    assert np.array_equal(from_bits(to_bits(m)), m)          # every entry is a bf16 value
    xb = to_bits(rs.normal(0, 1, (2, 4, 8)))
    scores, _, _ = v.verify(xb, GRAD)
    want, _, _ = oracle_mod.distance(xb, m)
    assert np.array_equal(scores[0], want)


def test_bf16_reference_settles_within_a_few_ulps_of_a_constant_input(oracle_mod):
    """With x fixed the update stalls once (1-beta)|x - m| drops below half a bf16 ulp of m:
    the reference ends within 1/(2(1-beta)) = 5 ulps (each at most 2^-7 relative) of x."""
    rs = np.random.default_rng(33)
    v = make(oracle_mod, B=1, T=8, d=16, ema_bf16=1)
    xb = to_bits(rs.normal(0, 1, (1, 8, 16)) + 3.0)
    x = from_bits(xb)
    for t in range(200):
        v.update_reference(xb, ACT)
    m1 = v.ema(ACT).copy()
    v.update_reference(xb, ACT)
    assert np.array_equal(v.ema(ACT), m1)                    # a fixed point
    assert np.all(np.abs(m1 - x) <= 5.5 * 2.0 ** -7 * np.abs(x))
    assert np.any(m1 != x)                                   # and it is not x itself everywhere


def test_bf16_reference_stores_rounded_values(oracle_mod):
    v = make(oracle_mod, ema_bf16=1)
    rs = np.random.default_rng(34)
    m = rs.normal(0, 1, (2, 4, 8))
    v.set_ema(ACT, m)
    assert np.array_equal(v.ema(ACT), from_bits(to_bits(m)))  # stored rounded


def test_bf16_reference_with_several_workers_is_the_single_precision_mean_rounded_once(oracle_mod):
    """m_t = bf16(fma(beta, m_{t-1}, (1-beta)/n * sum_r x^(r))) in float32, the sum in worker
    order.  Expected values: every float32 step formed exactly in float64 (operands of 24 bits or
    fewer) and rounded to float32, then torch's float32 -> bfloat16 conversion."""
    rs = np.random.default_rng(35)
    R = 3
    v = make(oracle_mod, B=2, T=5, d=16, ema_bf16=1, R=R)
    beta32 = np.float32(0.8)
    w32 = np.float32(np.float32(1.0 - 0.8) / np.float32(R))
    m = np.zeros((2, 5, 16), dtype=np.float32)
    for t in range(8):
        xbs = [to_bits(rs.normal(-0.3, 1.2, (2, 5, 16))) for _ in range(R)]
        v.step_replicas(xbs, GRAD, True)
        total = np.zeros_like(m)
        for xb in xbs:                                           # float32 adds, in worker order
            total = (total.astype(np.float64) + from_bits(xb)).astype(np.float32)
        prod = (np.float64(w32) * total.astype(np.float64)).astype(np.float32)
        fused = (np.float64(beta32) * m.astype(np.float64) + prod.astype(np.float64)).astype(np.float32)
        m = _as_bf16_f32(fused)
        assert np.array_equal(v.ema(GRAD), m.astype(np.float64)), t
    assert np.all(v.ema(ACT) == 0.0)


def test_bf16_reference_takes_directions(oracle_mod):
    """The sliced Wasserstein column of a bf16-reference verifier is the stateless distance against
    the stored (rounded) reference."""
    rs = np.random.default_rng(36)
    B, T, d = 2, 6, 16
    v = make(oracle_mod, B=B, T=T, d=d, ema_bf16=1)
    u = _directions(rs, 4, d)
    v.set_directions(u)
    for t in range(4):
        v.update_reference(to_bits(rs.normal(0, 1, (B, T, d))), ACT)
    m = v.ema(ACT).copy()
    xb = to_bits(rs.normal(0, 1, (B, T, d)))
    scores, _, _ = v.verify(xb, ACT)
    assert scores.shape[1] == 4
    assert scores[0, 3] == pytest.approx(oracle_mod.sliced_wasserstein(xb.reshape(B * T, d), m.reshape(B * T, d), u)[0], rel=1e-13)
    assert scores[2, 3] == pytest.approx(oracle_mod.sliced_wasserstein(xb[1], m[1], u)[0], rel=1e-13)


# ---------------------------------------------------------------------------------------------
# one [T,d] reference shared by the B samples

def test_shared_reference_is_the_full_reference_of_the_batch_mean(oracle_mod):
    """Eq. 1 with the mean over the samples as the submission: the [T,d] reference follows the
    batch mean exactly as a full reference of a one-sample verifier fed that mean would, and the
    closed form from m_0 = 0 holds."""
    rs = np.random.default_rng(41)
    B, T, d = 4, 5, 8
    v = make(oracle_mod, B=B, T=T, d=d, ref_over_batch=1)
    want = np.zeros((T, d))
    for t in range(6):
        xb = to_bits(rs.normal(0.5, 1, (B, T, d)))
        v.update_reference(xb, ACT)
        want = 0.9 * want + 0.1 * from_bits(xb).mean(axis=0)
        assert v.ema(ACT).shape == (T, d)
        assert v.ema(ACT) == pytest.approx(want, rel=1e-13, abs=1e-16)


def test_shared_reference_scores_are_those_against_the_tiled_reference(oracle_mod):
    """Every unit is compared with the same [T,d] tensor: sample b against m, the whole tensor
    against B copies of m -- the stateless distances say the same."""
    rs = np.random.default_rng(42)
    B, T, d = 3, 4, 8
    v = make(oracle_mod, B=B, T=T, d=d, ref_over_batch=1)
    for t in range(5):
        v.update_reference(to_bits(rs.normal(0, 1, (B, T, d)) + np.arange(d)), GRAD)
    m = v.ema(GRAD)
    xb = to_bits(rs.normal(0, 1, (B, T, d)) + np.arange(d))
    scores, flags, _ = v.verify(xb, GRAD)
    g0, s0, _ = oracle_mod.distance(xb, np.tile(m, (B, 1, 1)))
    assert np.array_equal(scores[0], g0) and np.array_equal(v.last_stats(GRAD)[0], s0)
    for b in range(B):
        gb, _, _ = oracle_mod.distance(xb[b], m)
        assert np.array_equal(scores[1 + b], gb)


def test_shared_reference_flags_commit_and_replacement(oracle_mod, small):
    v = oracle_mod.Verifier(oracle_mod.Params(B=small.B, T=small.T, d=small.d, ref_over_batch=1))
    for t in range(14):
        v.update_reference(synth.bits(synth.clean(small, 0, GRAD, t)), GRAD)
    g = synth.clean(small, 0, GRAD, 14)
    _, flags, commit = v.verify(synth.bits(g), GRAD)
    assert commit and not (flags & 0xFFFF).any()
    m0 = v.ema(GRAD)
    loud = (g.float() * 50).to(torch.bfloat16)
    _, flags, commit = v.verify(synth.bits(loud), GRAD)
    assert not commit and (flags[0] & 0xFFFF) and np.array_equal(v.ema(GRAD), m0)
    out, did = v.replace_if_flagged(synth.bits(loud), GRAD)
    assert did
    got = from_bits(out)
    for b in range(small.B):                                 # every sample receives the one reference
        assert np.all(np.abs(got[b] - m0) <= 2.0 ** -8 * np.abs(m0) + 1e-45)
    with pytest.raises(ValueError):
        oracle_mod.Verifier(oracle_mod.Params(B=2, T=4, d=8, ref_over_batch=1, R=2))
    with pytest.raises(ValueError):
        oracle_mod.Verifier(oracle_mod.Params(B=2, T=4, d=8, ref_over_batch=1, ema_bf16=1))


# ---------------------------------------------------------------------------------------------
# one [d] reference shared by all B*T tokens

def test_channel_reference_is_the_full_reference_of_the_token_mean(oracle_mod):
    """Eq. 1 with the mean over all B*T token rows as the submission: closed form from m_0 = 0,
    and rows that all equal one vector r give m_t = (1 - beta^t) r."""
    rs = np.random.default_rng(51)
    B, T, d = 3, 5, 8
    v = make(oracle_mod, B=B, T=T, d=d, ref_over_batch=1, ref_over_tokens=1)
    want = np.zeros(d)
    for t in range(6):
        xb = to_bits(rs.normal(0.5, 1, (B, T, d)))
        v.update_reference(xb, ACT)
        want = 0.9 * want + 0.1 * from_bits(xb).reshape(B * T, d).mean(axis=0)
        assert v.ema(ACT).shape == (d,)
        assert v.ema(ACT) == pytest.approx(want, rel=1e-13, abs=1e-16)
    r = from_bits(to_bits(rs.normal(0, 1, d)))
    v = make(oracle_mod, B=B, T=T, d=d, ref_over_batch=1, ref_over_tokens=1)
    for t in range(1, 5):
        v.update_reference(to_bits(np.tile(r, (B, T, 1))), GRAD)
        assert v.ema(GRAD) == pytest.approx((1 - 0.8 ** t) * r, rel=1e-13, abs=1e-16)


def test_channel_reference_scores_are_those_against_the_tiled_reference(oracle_mod):
    """Every token is compared with the same vector: sample b against T copies of m, the whole
    tensor against B*T copies -- the stateless distances say the same."""
    rs = np.random.default_rng(52)
    B, T, d = 3, 4, 8
    v = make(oracle_mod, B=B, T=T, d=d, ref_over_batch=1, ref_over_tokens=1)
    for t in range(5):
        v.update_reference(to_bits(rs.normal(0, 1, (B, T, d)) + np.arange(d)), GRAD)
    m = v.ema(GRAD)
    xb = to_bits(rs.normal(0, 1, (B, T, d)) + np.arange(d))
    scores, flags, _ = v.verify(xb, GRAD)
    g0, s0, _ = oracle_mod.distance(xb, np.tile(m, (B, T, 1)))
    assert np.array_equal(scores[0], g0) and np.array_equal(v.last_stats(GRAD)[0], s0)
    for b in range(B):
        gb, _, _ = oracle_mod.distance(xb[b], np.tile(m, (T, 1)))
        assert np.array_equal(scores[1 + b], gb)
    # a unit's statistics of the reference are those of the vector itself
    st = v.last_stats(GRAD)
    assert st[:, 3] == pytest.approx(m.mean(), rel=1e-12) and st[:, 4] == pytest.approx(m.var(), rel=1e-12)


def test_channel_reference_flags_commit_and_replacement(oracle_mod, small):
    v = oracle_mod.Verifier(oracle_mod.Params(B=small.B, T=small.T, d=small.d, ref_over_batch=1, ref_over_tokens=1))
    for t in range(14):
        v.update_reference(synth.bits(synth.clean(small, 0, ACT, t)), ACT)
    h = synth.clean(small, 0, ACT, 14)
    _, flags, commit = v.verify(synth.bits(h), ACT)
    assert commit and not (flags & 0xFFFF).any()
    m0 = v.ema(ACT)
    loud = (h.float() * 50).to(torch.bfloat16)
    _, flags, commit = v.verify(synth.bits(loud), ACT)
    assert not commit and (flags[0] & 0xFFFF) and np.array_equal(v.ema(ACT), m0)
    out, did = v.replace_if_flagged(synth.bits(loud), ACT)
    assert did
    got = from_bits(out)
    assert np.all(np.abs(got - m0) <= 2.0 ** -8 * np.abs(m0) + 1e-45)      # every token receives the one vector
    with pytest.raises(ValueError):
        oracle_mod.Verifier(oracle_mod.Params(B=2, T=4, d=8, ref_over_batch=1, ref_over_tokens=1, R=2))


# ---------------------------------------------------------------------------------------------
# one [B,d] reference: a vector per sample, shared by the sample's T tokens

def test_per_sample_channel_reference_follows_each_samples_token_mean(oracle_mod):
    """Eq. 1 with the mean over the T token rows of every sample: closed form from m_0 = 0, and
    the samples do not mix (changing sample 1 leaves the reference of sample 0 alone)."""
    rs = np.random.default_rng(61)
    B, T, d = 3, 5, 8
    v = make(oracle_mod, B=B, T=T, d=d, ref_over_tokens=1)
    u = make(oracle_mod, B=B, T=T, d=d, ref_over_tokens=1)
    want = np.zeros((B, d))
    for t in range(6):
        x = rs.normal(0.5, 1, (B, T, d))
        xb = to_bits(x)
        v.update_reference(xb, ACT)
        y = x.copy(); y[1] += 3.0
        u.update_reference(to_bits(y), ACT)
        want = 0.9 * want + 0.1 * from_bits(xb).mean(axis=1)
        assert v.ema(ACT).shape == (B, d)
        assert v.ema(ACT) == pytest.approx(want, rel=1e-13, abs=1e-16)
        assert np.array_equal(u.ema(ACT)[[0, 2]], v.ema(ACT)[[0, 2]]) and not np.allclose(u.ema(ACT)[1], v.ema(ACT)[1])


def test_per_sample_channel_reference_scores_are_those_against_the_tiled_reference(oracle_mod):
    rs = np.random.default_rng(62)
    B, T, d = 3, 4, 8
    v = make(oracle_mod, B=B, T=T, d=d, ref_over_tokens=1)
    for t in range(5):
        v.update_reference(to_bits(rs.normal(0, 1, (B, T, d)) + np.arange(d) + np.arange(B)[:, None, None]), GRAD)
    m = v.ema(GRAD)                                                      # [B, d]
    xb = to_bits(rs.normal(0, 1, (B, T, d)) + np.arange(d))
    scores, flags, _ = v.verify(xb, GRAD)
    tiled = np.repeat(m[:, None, :], T, axis=1)                          # [B, T, d]
    g0, s0, _ = oracle_mod.distance(xb, tiled)
    assert np.array_equal(scores[0], g0) and np.array_equal(v.last_stats(GRAD)[0], s0)
    for b in range(B):
        gb, _, _ = oracle_mod.distance(xb[b], tiled[b])
        assert np.array_equal(scores[1 + b], gb)


def test_per_sample_channel_reference_commit_and_replacement(oracle_mod, small):
    v = oracle_mod.Verifier(oracle_mod.Params(B=small.B, T=small.T, d=small.d, ref_over_tokens=1))
    for t in range(14):
        v.update_reference(synth.bits(synth.clean(small, 0, ACT, t)), ACT)
    h = synth.clean(small, 0, ACT, 14)
    _, flags, commit = v.verify(synth.bits(h), ACT)
    assert commit and not (flags & 0xFFFF).any()
    m0 = v.ema(ACT)
    loud = (h.float() * 50).to(torch.bfloat16)
    _, flags, commit = v.verify(synth.bits(loud), ACT)
    assert not commit and (flags[0] & 0xFFFF) and np.array_equal(v.ema(ACT), m0)
    out, did = v.replace_if_flagged(synth.bits(loud), ACT)
    assert did
    got = from_bits(out)
    for b in range(small.B):                                 # every token of sample b receives that sample's vector
        assert np.all(np.abs(got[b] - m0[b]) <= 2.0 ** -8 * np.abs(m0[b]) + 1e-45)
    with pytest.raises(ValueError):
        oracle_mod.Verifier(oracle_mod.Params(B=2, T=4, d=8, ref_over_tokens=1, ema_bf16=1))


def test_a_constant_history_does_not_make_clean_steps_severe(oracle_mod):
    """With iqr_eps = 0 and lambda = 0 a window of identical deviations gives tau_upper = q2.  A
    clean step on the median then has |gamma - q2| = 0 >= 100 * 0: the severe rule must not fire
    for it (it speaks of a deviation that broke the threshold), while a flagged step at any
    distance from such a window does."""
    v = make(oracle_mod, B=1, T=2, d=8, eps=(0.0, 0.0), lam=(0.0, 0.0))
    xb = to_bits(np.tile(np.array([1.0, -2.0, 3.0, 0.5, -1.5, 2.5, -0.25, 4.0]), (1, 2, 1)))
    v.set_ema(ACT, np.zeros((1, 2, 8)))
    for _ in range(6):                                   # beta irrelevant: keep the reference at 0
        v.update_reference(xb, ACT)
        v.set_ema(ACT, np.zeros((1, 2, 8)))
    thr, valid = v.thresholds(ACT)
    assert valid.all() and np.all(thr[:, :, 5] == thr[:, :, 1])          # tau_upper == q2 everywhere
    scores, flags, commit = v.verify(xb, ACT)
    assert commit and not (flags[0] & oracle_mod.FLAG_SEVERE) and not (flags[0] & 0xFFFF)
    assert v.counters() == (0, 1, 0)
    v.set_ema(ACT, np.zeros((1, 2, 8)))
    scores, flags, commit = v.verify(to_bits(2.0 * from_bits(xb)), ACT)  # L1 doubles: off the single point
    assert not commit and (flags[0] & oracle_mod.FLAG_L1) and (flags[0] & oracle_mod.FLAG_SEVERE)
    assert v.counters() == (1, 0, 1)
