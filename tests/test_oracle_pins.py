"""Pins for the float64 CPU oracle: it is checked against what the paper and the mathematics
fix (closed forms, library routines, exact rational brute force, hand-worked Alg. 5 cases),
never against itself and never against the CUDA path."""
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.stats
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def to_bits(a) -> np.ndarray:
    """float array -> bf16 bit patterns (round to nearest even)."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def from_bits(b) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


@pytest.fixture(scope="module")
def rng():
    return np.random.default_rng(20260303)


# ---------------------------------------------------------------- element conversion

def test_bf16_conversion_is_exact(oracle_mod):
    for bits, val in [(0x3F80, 1.0), (0xBF80, -1.0), (0x4000, 2.0), (0x3F00, 0.5), (0x0000, 0.0),
                      (0x8000, -0.0), (0x4049, 3.140625), (0x0001, 2.0 ** -133)]:
        assert oracle_mod.lib().so_bf16(bits) == val
    assert np.isinf(oracle_mod.lib().so_bf16(0x7F80))
    assert np.isnan(oracle_mod.lib().so_bf16(0x7FC0))
    b = np.arange(0, 65536, 7, dtype=np.uint16)
    assert np.array_equal(oracle_mod.bf16_to_f64(b), from_bits(b), equal_nan=True)


# ---------------------------------------------------------------- Sec. 3.1 metrics

def test_metrics_against_library_routines(oracle_mod, rng):
    """L1 = mean |x-m|; L2 = mean squared difference of scipy z-scores = 2 - 2*Pearson rho;
    SFR = mean(sign(x) != sign(m))."""
    for n, loc, scale in [(64, 0.0, 1.0), (1000, 3.0, 0.25), (4096, -0.5, 7.0)]:
        xb = to_bits(rng.normal(loc, scale, n))
        x = from_bits(xb)
        m = rng.normal(loc * 0.9, scale * 1.3, n)
        g, s, nf = oracle_mod.distance(xb, m)
        assert not nf
        assert g[0] == pytest.approx(np.mean(np.abs(x - m)), rel=1e-13)
        zx, zm = scipy.stats.zscore(x, ddof=0), scipy.stats.zscore(m, ddof=0)
        assert g[1] == pytest.approx(np.mean((zx - zm) ** 2), rel=1e-12)
        rho = np.corrcoef(x, m)[0, 1]
        assert g[1] == pytest.approx(2.0 - 2.0 * rho, rel=1e-11, abs=1e-13)
        assert g[2] == pytest.approx(np.mean(np.sign(x) != np.sign(m)), abs=0)
        assert s[0] == pytest.approx(x.mean(), rel=1e-12, abs=1e-15)
        assert s[1] == pytest.approx(x.var(), rel=1e-12)
        assert s[2] == pytest.approx(np.linalg.norm(x), rel=1e-12)
        assert s[3] == pytest.approx(m.mean(), rel=1e-12, abs=1e-15)
        assert s[4] == pytest.approx(m.var(), rel=1e-12)
        assert s[5] == pytest.approx(np.cov(x, m, ddof=0)[0, 1], rel=1e-11, abs=1e-15)
        assert s[6] == pytest.approx(np.linalg.norm(m), rel=1e-12)
        assert s[7] == pytest.approx(rho, rel=1e-11, abs=1e-14)


def test_metric_closed_forms(oracle_mod, rng):
    n = 2048
    xb = to_bits(rng.normal(0.3, 1.0, n))
    x = from_bits(xb)
    m = 0.7 * x + rng.normal(0, 0.5, n)
    g, _, _ = oracle_mod.distance(xb, m)
    # negating x: rho -> -rho, so L2 -> 4 - L2; every sign flips, so SFR -> 1 - SFR (no zeros)
    assert np.all(x != 0) and np.all(m != 0)
    gn, _, _ = oracle_mod.distance(to_bits(-x), m)
    assert gn[1] == pytest.approx(4.0 - g[1], rel=1e-12)
    assert gn[2] == pytest.approx(1.0 - g[2], abs=1e-15)
    # positive affine maps of x leave the z-scored distance alone (2x and x+1 stay in bf16
    # only approximately, so apply them to m, which is float64)
    ga, _, _ = oracle_mod.distance(xb, 3.0 * m + 11.0)
    assert ga[1] == pytest.approx(g[1], rel=1e-11)
    # L1 against the zero reference is the mean magnitude; L1 is absolutely homogeneous
    g0, _, _ = oracle_mod.distance(xb, np.zeros(n))
    assert g0[0] == pytest.approx(np.mean(np.abs(x)), rel=1e-13)
    g4, _, _ = oracle_mod.distance(to_bits(-4.0 * x), -4.0 * m)   # x*4 is exact in bf16
    assert g4[0] == pytest.approx(4.0 * g[0], rel=1e-13)
    # identical vectors are at distance zero in every metric
    gs, ss, _ = oracle_mod.distance(xb, x)
    assert gs[0] == 0.0 and gs[2] == 0.0 and abs(gs[1]) < 1e-13
    assert ss[7] == pytest.approx(1.0, abs=1e-13)


def test_constant_and_degenerate_vectors(oracle_mod, rng):
    n = 512
    m = rng.normal(0, 1, n)
    # constant x: variance exactly 0, z-score is the zero vector, so L2 = mean(zm^2) = 1
    for c in (0.0, -1.0, 0.1, 37.5):
        xb = to_bits(np.full(n, c))
        g, s, _ = oracle_mod.distance(xb, m)
        assert s[1] == 0.0
        assert g[1] == pytest.approx(1.0, rel=1e-12)
        assert s[7] == 0.0
    # both constant: L2 = 0; constant reference that is no round number: var_m exactly 0
    g, s, _ = oracle_mod.distance(to_bits(np.full(n, 2.0)), np.full(n, 0.1 * 0.3))
    assert g[1] == 0.0 and s[1] == 0.0 and s[4] == 0.0
    assert g[0] == pytest.approx(2.0 - 0.03, rel=1e-13)
    # sign of zero is zero: against m = 0, SFR is the fraction of non-zero x
    x = rng.normal(0, 1, n)
    x[::4] = 0.0
    x[1::8] = -0.0
    g, _, _ = oracle_mod.distance(to_bits(x), np.zeros(n))
    assert g[2] == np.count_nonzero(x) / n
    # zero against zero is no flip
    g, _, _ = oracle_mod.distance(to_bits(np.zeros(n)), np.zeros(n))
    assert tuple(g) == (0.0, 0.0, 0.0)


def test_non_finite_input_is_reported(oracle_mod):
    x = np.ones(16, dtype=np.float32)
    for bad in (np.nan, np.inf, -np.inf):
        y = x.copy()
        y[5] = bad
        g, s, nf = oracle_mod.distance(to_bits(y), np.zeros(16))
        assert nf and np.all(np.isnan(g)) and np.all(np.isnan(s))


def test_brute_force_exact_rationals(oracle_mod):
    """Tiny [2,3,8] tensors: L1 and SFR in exact rational arithmetic with Python loops; the
    z-scored distance from exactly accumulated moments."""
    rs = np.random.default_rng(7)
    B, T, d = 2, 3, 8
    xb = to_bits(rs.integers(-8, 9, size=(B, T, d)) / 4.0)
    m = rs.integers(-8, 9, size=(B, T, d)) / 8.0
    x = from_bits(xb)
    x[0, 0, 0] = 0.0
    xb = to_bits(x)
    for sl in (np.s_[:], np.s_[0], np.s_[1]):
        xs, ms = x[sl].reshape(-1), m[sl].reshape(-1)
        n = xs.size
        fx = [Fraction(float(v)) for v in xs]
        fm = [Fraction(float(v)) for v in ms]
        l1 = sum(abs(a - b) for a, b in zip(fx, fm)) / n
        sgn = lambda v: (v > 0) - (v < 0)
        sfr = Fraction(sum(sgn(a) != sgn(b) for a, b in zip(fx, fm)), n)
        mx, mm = sum(fx) / n, sum(fm) / n
        vx = sum((a - mx) ** 2 for a in fx) / n
        vm = sum((b - mm) ** 2 for b in fm) / n
        cov = sum((a - mx) * (b - mm) for a, b in zip(fx, fm)) / n
        l2 = 2.0 - 2.0 * float(cov) / (float(vx) ** 0.5 * float(vm) ** 0.5)
        g, s, _ = oracle_mod.distance(xb[sl], ms)
        assert g[0] == pytest.approx(float(l1), rel=1e-14)
        assert g[2] == float(sfr)
        assert g[1] == pytest.approx(l2, rel=1e-12)
        assert s[1] == pytest.approx(float(vx), rel=1e-13)
        assert s[5] == pytest.approx(float(cov), rel=1e-12, abs=1e-15)


def test_hand_made_tiny_cases(oracle_mod):
    # one element flipped out of 8
    x = np.array([1, 2, 3, 4, 5, 6, 7, 8], dtype=np.float64)
    m = x.copy()
    m[2] = -3.0
    g, _, _ = oracle_mod.distance(to_bits(x), m)
    assert g[2] == 1 / 8
    assert g[0] == 6 / 8
    # x = 2*m + 1 exactly: rho = 1, L2 = 0, L1 = mean|m + 1|
    m = np.array([-2.0, -1.0, 0.0, 1.0, 2.0, 3.0, 0.5, -0.5])
    g, s, _ = oracle_mod.distance(to_bits(2 * m + 1), m)
    assert abs(g[1]) < 1e-14 and s[7] == pytest.approx(1.0, abs=1e-14)
    assert g[0] == pytest.approx(np.mean(np.abs(m + 1)), rel=1e-14)


def test_invariants_scaling_and_permutation(oracle_mod, rng):
    B, T, d = 3, 16, 32
    x = from_bits(to_bits(rng.normal(0, 1, (B, T, d))))
    m = rng.normal(0, 1, (B, T, d))
    g, s, _ = oracle_mod.distance(to_bits(x[1]), m[1])
    # scaling by c = -8 (exact in bf16): norm and |mean| scale by |c|, variance by c^2
    g8, s8, _ = oracle_mod.distance(to_bits(-8.0 * x[1]), m[1])
    assert s8[2] == pytest.approx(8.0 * s[2], rel=1e-13)
    assert s8[0] == pytest.approx(-8.0 * s[0], rel=1e-12)
    assert s8[1] == pytest.approx(64.0 * s[1], rel=1e-12)
    # permuting tokens of x and m jointly changes nothing; permuting x alone keeps x's moments
    perm = rng.permutation(T)
    gp, sp, _ = oracle_mod.distance(to_bits(x[1][perm]), m[1][perm])
    assert gp == pytest.approx(g, rel=1e-12)
    _, sq, _ = oracle_mod.distance(to_bits(x[1][perm]), m[1])
    assert sq[:3] == pytest.approx(s[:3], rel=1e-12)


# ---------------------------------------------------------------- Alg. 5

def test_percentile_matches_numpy_linear(oracle_mod, rng):
    for n in (1, 2, 3, 4, 5, 10, 99, 100, 101, 1600):
        a = np.sort(rng.normal(0, 1, n))
        for p in (0.0, 0.25, 0.5, 0.75, 1.0, 0.1, 0.9):
            want = np.percentile(a, 100 * p, method="linear")
            assert oracle_mod.percentile(a, p) == pytest.approx(want, rel=1e-13, abs=1e-15)


def _parse_window(spec):
    tok = spec.split()
    if tok[0] == "range":
        return np.arange(int(tok[1]), int(tok[2]) + 1, dtype=np.float64)
    if tok[0] == "const":
        return np.full(int(tok[2]), float(tok[1]))
    return np.array([float(t) for t in tok[1:]])


def _hand_cases():
    cases = []
    with open(os.path.join(GOLDEN, "alg5_hand_cases.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            name, win, par, exp, its = [f.strip() for f in line.split("|")]
            cases.append((name, _parse_window(win), [float(v) for v in par.split()],
                          [float(v) for v in exp.split()], [int(v) for v in its.split()]))
    return cases


@pytest.mark.parametrize("case", _hand_cases(), ids=lambda c: c[0])
def test_alg5_hand_worked_cases(oracle_mod, case, rng):
    _, window, par, exp, its = case
    k_prev, alpha, n_max, gg, gs, lam, eps, ratio = par
    for w in (window, rng.permutation(window)):          # the order of the window is immaterial
        thr, iters = oracle_mod.adaptive_iqr(w, k_prev, alpha, int(n_max), gg, gs, lam, eps, ratio)
        assert thr == pytest.approx(exp, rel=1e-11, abs=1e-12)
        assert list(iters) == its


def test_alg5_reduces_to_plain_tukey_rule(oracle_mod, rng):
    """With no iterations allowed, no floor and no clamp, the thresholds are median -+ k*IQR."""
    w = rng.lognormal(0, 1, 257)
    q1, q2, q3 = np.percentile(w, [25, 50, 75])
    thr, iters = oracle_mod.adaptive_iqr(w, 1.5, 0.01, 0, 1.1, 0.9, 0.0, 0.0)
    assert iters == (0, 0)
    assert thr == pytest.approx([q1, q2, q3, 1.5, q2 - 1.5 * (q3 - q1), q2 + 1.5 * (q3 - q1)], rel=1e-12)


def test_alg5_properties(oracle_mod, rng):
    w = rng.normal(5.0, 1.0, 400)
    # empty window: nothing to compute
    thr, _ = oracle_mod.adaptive_iqr(np.zeros(0), 1.5, 0.01, 10, 1.1, 0.9, 0.1, 1e-3)
    assert thr is None
    # the multiplier only moves by whole powers of the two factors
    thr, (gi, si) = oracle_mod.adaptive_iqr(w, 0.2, 0.01, 10, 1.1, 0.9, 0.0, 0.0)
    assert thr[3] == pytest.approx(0.2 * 1.1 ** gi * 0.9 ** si, rel=1e-13)
    assert gi == 10                       # far too narrow: widening runs out of iterations
    # after widening stops early the window's FP-rate is at most alpha
    thr, (gi, si) = oracle_mod.adaptive_iqr(w, 1.0, 0.05, 50, 1.1, 0.9, 0.0, 0.0, shrink_ratio=0.0)
    assert gi < 50 and si == 0
    assert np.mean((w < thr[4]) | (w > thr[5])) <= 0.05
    # the clamp keeps both bounds at least |q2|*lambda from the median
    thr, _ = oracle_mod.adaptive_iqr(w, 0.01, 1.0, 10, 1.1, 0.9, 0.3, 0.0)
    assert thr[4] <= thr[1] - 0.3 * abs(thr[1]) + 1e-15 and thr[5] >= thr[1] + 0.3 * abs(thr[1]) - 1e-15


def test_default_hyperparameters_match_the_paper_table(oracle_mod):
    want = {}
    with open(os.path.join(GOLDEN, "hyperparams_table.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            tok = line.split()
            want[tok[0]] = tuple(float(v) for v in tok[1:])
    got = oracle_mod.default_params_from_c()
    py = oracle_mod.Params()
    for key, cname, pyname in [("beta", "beta", "beta"), ("k0", "k0", "k0"), ("alpha", "alpha", "alpha"),
                               ("n_max", "n_max", "n_max"), ("gamma_g", "gamma_g", "gamma_g"),
                               ("gamma_s", "gamma_s", "gamma_s"), ("lambda", "lam", "lam"),
                               ("eps", "eps", "eps")]:
        assert tuple(got[cname]) == want[key]
        assert tuple(getattr(py, pyname)) == want[key]
    for key, cname in [("c", "c"), ("t_forgiveness", "t_forgiveness"), ("l", "l"), ("severe_mult", "severe_mult")]:
        assert float(got[cname]) == want[key][0]
        assert float(getattr(py, cname)) == want[key][0]


# ---------------------------------------------------------------- bf16 rounding (Alg. 4 output)

def test_bf16_rounding_matches_the_library_on_floats_and_rounds_once(oracle_mod, rng):
    """For values a float holds exactly, round-to-nearest-even to bf16 is torch's conversion; a
    double just above a tie must go up although its float image sits on the tie."""
    vals = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-4, 2000), rng.normal(0, 1e4, 2000),
                           [0.0, -0.0, 1.0, -1.0, 65504.0, 3.3e38, 1e-40, -1e-40]]).astype(np.float32)
    want = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle_mod.bf16_round(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, want)
    # ties to even, by hand: 1 + 2^-8 is halfway between 1 (even) and 1 + 2^-7
    assert oracle_mod.bf16_round(1 + 2.0 ** -8) == 0x3F80
    assert oracle_mod.bf16_round(1 + 3 * 2.0 ** -8) == 0x3F82
    assert oracle_mod.bf16_round(1 + 2.0 ** -8 + 2.0 ** -40) == 0x3F81      # one rounding, not two
    assert oracle_mod.bf16_round(1 + 2.0 ** -8 - 2.0 ** -40) == 0x3F80
    assert oracle_mod.bf16_round(float("inf")) == 0x7F80 and oracle_mod.bf16_round(-1e39) == 0xFF80
    assert oracle_mod.bf16_round(float("nan")) & 0x7FC0 == 0x7FC0
    # rounding is the identity on bf16 values
    b = np.arange(0, 0x7F80, 37, dtype=np.uint16)
    assert all(oracle_mod.bf16_round(float(v)) == int(u) for u, v in zip(b, from_bits(b)))


# ---------------------------------------------------------------- sliced Wasserstein (Sec. 3.1)

def _directions(rng, L, d):
    u = rng.normal(0, 1, (L, d))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    ub = to_bits(u)
    return ub, from_bits(ub)


def test_sliced_wasserstein_against_scipy_and_closed_forms(oracle_mod, rng):
    tokens, d, L = 96, 40, 5
    ub, u = _directions(rng, L, d)
    xb = to_bits(rng.normal(0.2, 1.0, (tokens, d)))
    x = from_bits(xb)
    m = rng.normal(-0.1, 1.5, (tokens, d))
    val, w1 = oracle_mod.sliced_wasserstein(xb, m, ub)
    for l in range(L):                     # 1-D W1 of equal-size samples is scipy's routine
        want = scipy.stats.wasserstein_distance(x @ u[l], m @ u[l])
        assert w1[l] == pytest.approx(want, rel=1e-11)
    assert val == pytest.approx(w1.mean(), rel=1e-14)
    # identical clouds: zero; a cloud shifted by one vector v: every projection moves by u.v
    assert oracle_mod.sliced_wasserstein(xb, x, ub)[0] == 0.0
    v = rng.normal(0, 1, d)
    val_s, w1_s = oracle_mod.sliced_wasserstein(xb, x + v, ub)
    assert w1_s == pytest.approx(np.abs(u @ v), rel=1e-11)
    # the order of the tokens is immaterial, separately for the two clouds
    p1, p2 = rng.permutation(tokens), rng.permutation(tokens)
    assert oracle_mod.sliced_wasserstein(xb[p1], m[p2], ub)[0] == pytest.approx(val, rel=1e-12)
    # absolutely homogeneous: scaling both clouds by -4 (exact in bf16) scales the distance by 4
    assert oracle_mod.sliced_wasserstein(to_bits(-4 * x), -4 * m, ub)[0] == pytest.approx(4 * val, rel=1e-12)
    # two point masses per cloud, by hand: x projects to {0, 2}, m to {1, 5} along e1 -> (1 + 3)/2
    e1 = to_bits(np.array([[1.0, 0.0]]))
    val2, _ = oracle_mod.sliced_wasserstein(to_bits(np.array([[2.0, 7.0], [0.0, -3.0]])),
                                            np.array([[5.0, 0.0], [1.0, 9.0]]), e1)
    assert val2 == 2.0
    bad = x.copy()
    bad[3, 4] = np.inf
    assert np.isnan(oracle_mod.sliced_wasserstein(to_bits(bad), m, ub)[0])


# ---------------------------------------------------------------- decision rules, token sums

def test_out_of_bounds_is_the_negated_closed_interval(oracle_mod):
    """Eq. 3 / Alg. 5: flagged iff outside [tau_lower, tau_upper]; the bounds themselves are inside,
    and a deviation that is not a number is outside."""
    ob = oracle_mod.out_of_bounds
    assert not ob(1.0, 1.0, 2.0) and not ob(2.0, 1.0, 2.0) and not ob(1.5, 1.0, 2.0)
    assert ob(np.nextafter(1.0, 0.0), 1.0, 2.0) and ob(np.nextafter(2.0, 3.0), 1.0, 2.0)
    assert ob(float("nan"), 1.0, 2.0) and ob(float("inf"), 1.0, 2.0) and ob(-float("inf"), 1.0, 2.0)
    assert not ob(0.0, 0.0, 0.0)                      # a degenerate interval still holds its point


def test_severe_rule_needs_a_flag(oracle_mod):
    """Sec. 3.1: 'x100 above the threshold' is said of a deviation that broke the threshold."""
    sv = oracle_mod.severe
    assert sv(True, 1.0 + 100 * 0.5, 1.0, 1.5, 100.0)            # exactly 100 allowed deviations
    assert not sv(True, 1.0 + 99.9 * 0.5, 1.0, 1.5, 100.0)
    assert sv(True, 1.0 - 100 * 0.5, 1.0, 1.5, 100.0)            # two-sided
    assert not sv(False, 1e9, 1.0, 1.5, 100.0)                   # not flagged: never severe
    assert not sv(False, 1.0, 1.0, 1.0, 100.0)                   # tau_upper == q2, clean step on the median
    assert sv(True, 2.0, 1.0, 1.0, 100.0)                        # zero allowed deviation, flagged
    assert not sv(True, float("nan"), 1.0, 1.5, 100.0)           # not a number: flagged, but no distance


def test_token_sums_by_hand_and_against_the_unit_measures(oracle_mod, rng):
    """Hand-written rows (small integers and halves are exact in bf16), then the identity that ties
    the token sums to the pinned unit measures: summed over the rows of a unit and divided by its
    size they are the L1 distance and the sign-flip ratio of so_distance."""
    x = np.array([[1.0, -2.0, 0.0, 3.0, -0.0, 0.5, -4.0, 8.0]])
    m = np.array([[1.0, 2.0, 0.0, -1.0, 1.0, 0.25, -4.0, 0.0]])
    got = oracle_mod.token_sums(to_bits(x), m)
    #  sum x = 6.5; sum x^2 = 1+4+0+9+0+0.25+16+64 = 94.25; |x-m| = 0+4+0+4+1+0.25+0+8 = 17.25
    #  sign mismatches: (-2,2) (3,-1) (-0,1) (8,0) -> 4
    assert got.tolist() == [[6.5, 94.25, 17.25, 4.0]]
    xb = to_bits(rng.normal(0.2, 1.3, (5, 24)))
    mm = rng.normal(0.0, 1.0, (5, 24))
    ts = oracle_mod.token_sums(xb, mm)
    gam, stat, _ = oracle_mod.distance(xb, mm)
    assert ts[:, 2].sum() / xb.size == pytest.approx(gam[0], rel=1e-13)
    assert ts[:, 3].sum() / xb.size == pytest.approx(gam[2], rel=1e-13)
    assert ts[:, 0].sum() / xb.size == pytest.approx(stat[0], rel=1e-12, abs=1e-15)
    assert np.sqrt(ts[:, 1].sum()) == pytest.approx(stat[2], rel=1e-13)
