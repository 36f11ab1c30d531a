"""GPU parity of the sliced Wasserstein distance (Sec. 3.1) against the float64 oracle."""
import numpy as np
import pytest
import torch

from paper_2603_03592_b200 import synth

pytestmark = pytest.mark.gpu
REL = 1e-3


@pytest.fixture(scope="module")
def sb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_03592_b200 import binding
    binding.lib()
    return binding


def directions(L, d, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    u = torch.randn(L, d, generator=g, device="cuda")
    return (u / u.norm(dim=1, keepdim=True)).to(torch.bfloat16).contiguous()


def oracle_all_units(oracle_mod, x, m, u):
    xb, ub = synth.bits(x), synth.bits(u)
    m64 = m.double().cpu().numpy()
    B = x.shape[0]
    out = np.empty(1 + B)
    out[0] = oracle_mod.sliced_wasserstein(xb.reshape(-1, x.shape[2]), m64.reshape(-1, x.shape[2]), ub)[0]
    for b in range(B):
        out[1 + b] = oracle_mod.sliced_wasserstein(xb[b], m64[b], ub)[0]
    return out


def run(sb, x, m, u):
    out = torch.full((1 + x.shape[0],), -7.0, dtype=torch.float32, device="cuda")
    sb.sentinel_sliced_wasserstein(x, m, u, out)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


CASES = [((1, 1, 8), 4), ((2, 3, 16), 4), ((3, 37, 520), 8), ((5, 100, 1024), 16), ((4, 128, 2048), 8),
         ((8, 64, 512), 4), ((7, 33, 264), 16), ((1, 700, 136), 8),
         # long lists that are few: each sample's list is sorted as two halves (T even, at least 1024) and merged
         ((2, 1536, 264), 8), ((1, 2048, 136), 8), ((3, 1024, 72), 4), ((5, 1030, 40), 4), ((2, 1025, 64), 4)]


@pytest.mark.parametrize("shape,L", CASES, ids=["%dx%dx%d_L%d" % (*s, l) for s, l in CASES])
def test_matches_oracle_over_shapes(sb, oracle_mod, shape, L):
    """Odd sample counts (unpaired runs in the merge), token counts that are no power of two,
    ragged d, a single token."""
    B, T, d = shape
    g = torch.Generator(device="cuda").manual_seed(77 + B + T + d)
    x = (torch.randn(B, T, d, generator=g, device="cuda") * 1.3 + 0.1).to(torch.bfloat16)
    m = (0.4 * x.float() + torch.randn(B, T, d, generator=g, device="cuda") * 0.7 - 0.2).contiguous()
    u = directions(L, d, 5 + L)
    got = run(sb, x, m, u)
    want = oracle_all_units(oracle_mod, x, m, u)
    scale = float(x.float().std())
    assert np.all(np.abs(got - want) <= REL * np.maximum(np.abs(want), 1e-3 * scale)), (got, want)


def test_an_entry_that_is_not_finite_spoils_its_sample_and_the_whole_tensor(sb):
    B, T, d, L = 3, 1200, 64, 8
    g = torch.Generator(device="cuda").manual_seed(21)
    x = torch.randn(B, T, d, generator=g, device="cuda").to(torch.bfloat16)
    m = torch.randn(B, T, d, generator=g, device="cuda")
    u = directions(L, d, 2)
    for bad in (float("inf"), float("nan")):
        y = x.clone()
        y[1, 700, 5] = bad
        got = run(sb, y, m, u)
        assert np.isfinite(got[1]) and np.isfinite(got[3]), got
        assert not np.isfinite(got[0]) and not np.isfinite(got[2]), got


def test_closed_forms_on_gpu(sb):
    B, T, d, L = 3, 50, 256, 8
    g = torch.Generator(device="cuda").manual_seed(3)
    x = torch.randn(B, T, d, generator=g, device="cuda").to(torch.bfloat16)
    u = directions(L, d, 9)
    # identical clouds are at distance zero
    assert np.all(run(sb, x, x.float().contiguous(), u) == 0.0)
    # a cloud shifted by one vector v moves every projection by u.v
    v = torch.randn(d, generator=g, device="cuda")
    want = float((u.float() @ v).abs().mean())
    got = run(sb, x, (x.float() + v).contiguous(), u)
    assert got == pytest.approx(np.full(1 + B, want), rel=1e-4)
    # permuting the tokens of a sample changes nothing
    perm = torch.randperm(T, generator=g, device="cuda")
    m = torch.randn(B, T, d, generator=g, device="cuda")
    a = run(sb, x, m, u)
    b = run(sb, x[:, perm].contiguous(), m, u)
    assert b == pytest.approx(a, rel=1e-5)


def test_stage_traffic_shape(sb, oracle_mod):
    """The small-LM stage shape (16 x 1024 x 2048) with the recipe's activations against an EMA of
    earlier microbatches; the oracle checks the whole tensor and three samples."""
    w = synth.WORKLOADS["cfg2"]
    m = torch.zeros(w.B, w.T, w.d, device="cuda")
    for t in range(4):
        m = 0.9 * m + 0.1 * synth.clean(w, 0, 0, t, "cuda").float()
    x = synth.clean(w, 0, 0, 4, "cuda")
    u = directions(8, w.d, 1)
    got = run(sb, x, m.contiguous(), u)
    xb, ub, m64 = synth.bits(x), synth.bits(u), m.double().cpu().numpy()
    for row in (0, 1, 7, 16):
        if row == 0:
            want = oracle_mod.sliced_wasserstein(xb.reshape(-1, w.d), m64.reshape(-1, w.d), ub)[0]
        else:
            want = oracle_mod.sliced_wasserstein(xb[row - 1], m64[row - 1], ub)[0]
        assert got[row] == pytest.approx(want, rel=REL)


def test_argument_checks(sb):
    x = torch.zeros(2, 4, 16, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(2, 4, 16, device="cuda")
    u = torch.zeros(8, 16, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(3, device="cuda")
    L, s = sb.lib(), torch.cuda.current_stream().cuda_stream
    f = L.sentinel_sliced_wasserstein
    assert f(x.data_ptr(), m.data_ptr(), u.data_ptr(), 5, 2, 4, 16, 0, s, o.data_ptr()) == sb.ERR_UNSUPPORTED
    assert f(x.data_ptr(), m.data_ptr(), None, 8, 2, 4, 16, 0, s, o.data_ptr()) == sb.ERR_INVALID_ARG
    assert f(x.data_ptr(), m.data_ptr(), u.data_ptr() + 2, 8, 2, 4, 16, 0, s, o.data_ptr()) == sb.ERR_UNALIGNED
    assert f(x.data_ptr(), m.data_ptr(), u.data_ptr(), 8, 2, 20000, 16, 0, s, o.data_ptr()) == sb.ERR_UNSUPPORTED
    assert f(x.data_ptr(), m.data_ptr(), u.data_ptr(), 16, 2, 4, 8192, 0, s, o.data_ptr()) == sb.ERR_UNSUPPORTED
    assert f(x.data_ptr(), m.data_ptr(), u.data_ptr(), 8, 2, 4, 12, 0, s, o.data_ptr()) == sb.ERR_UNALIGNED


# ---------------------------------------------------------------------------------------------
# the distance as the fourth metric of a verifier (sentinel_set_directions)

from helpers import UNIT_BITS, assert_scores_close, near_threshold, oracle_to_blob, parse_blob  # noqa: E402
from test_gpu_parity import compare_state, compare_thresholds, lockstep, make_pair  # noqa: E402
import test_gpu_replicas as rep  # noqa: E402

ACT, GRAD = 0, 1


def with_directions(gv, ov, L, d, seed=3):
    u = synth.directions(L, d, seed, "cuda")
    gv.sentinel_set_directions(u)
    ov.set_directions(synth.bits(u))
    assert gv.sentinel_num_metrics() == 4 and gv.M == 4
    return u


@pytest.mark.parametrize("name,shape,L,steps", [("cfg2", (4, 40, 264), 8, 50), ("cfg4", (3, 24, 1024), 4, 40),
                                                ("cfg3", (5, 33, 520), 16, 60)],
                         ids=["cfg2_L8", "cfg4_L4", "cfg3_L16"])
def test_streams_in_lockstep_with_four_metrics(sb, oracle_mod, name, shape, L, steps):
    """The benchmark recipes at oracle size with the sliced Wasserstein distance switched on:
    four score columns, four flag bits, four histories and sets of bounds, step by step."""
    w = synth.scaled(synth.WORKLOADS[name], name + "_sw", *shape, corrupt_rate=0.25)
    gv, ov, params = make_pair(sb, oracle_mod, w)
    with_directions(gv, ov, L, w.d)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, steps)
    assert rec["corrupted"] >= 4
    compare_state(gv, ov, params)
    for kind in (ACT, GRAD):
        compare_thresholds(gv, ov, kind)
        gt, gvalid = gv.sentinel_get_thresholds(kind)
        assert gt.shape == (2, 4, 6) and gvalid.all()
    assert rec["near"] <= 2 and rec["k_events"] <= 4, rec
    gv.close()


def test_fourth_column_equals_the_stateless_distance(sb, oracle_mod):
    """Column 3 of a verified step is sentinel_sliced_wasserstein of the same tensor against the
    reference the step was tested with (exported just before).  Not bit for bit: the verifier
    carries the reference's projections along (float64 recursion of Eq. 1 on the projections)
    where the stateless call projects the fp32 reference afresh.  Right after a state import the
    verifier projects the reference afresh too, and the two agree exactly."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "sw_col", 3, 50, 512)
    gv, ov, params = make_pair(sb, oracle_mod, w)
    u = with_directions(gv, ov, 8, w.d)
    for t in range(5):
        gv.update_reference(synth.clean(w, 0, ACT, t, "cuda"), ACT)
    m = torch.from_numpy(parse_blob(gv.sentinel_export_state(), w.B, w.T, w.d, params.l)["kinds"][ACT]["m"]).cuda()
    x = synth.clean(w, 0, ACT, 5, "cuda")
    gs, gf = gv.verify(x, ACT)
    torch.cuda.synchronize()
    want = torch.empty(1 + w.B, device="cuda")
    sb.sentinel_sliced_wasserstein(x, m, u, want)
    torch.cuda.synchronize()
    assert torch.allclose(gs[:, 3], want, rtol=2e-5, atol=0)
    # a state import invalidates the carried projections: the next step recomputes them from m
    blob = gv.sentinel_export_state()
    m2 = torch.from_numpy(parse_blob(blob, w.B, w.T, w.d, params.l)["kinds"][ACT]["m"]).cuda()
    gv.sentinel_import_state(blob)
    x2 = synth.clean(w, 0, ACT, 6, "cuda")
    gs2, _ = gv.verify(x2, ACT)
    sb.sentinel_sliced_wasserstein(x2, m2, u, want)
    torch.cuda.synchronize()
    assert torch.equal(gs2[:, 3], want)
    # ... and the steps after that carry them along again
    m3 = torch.from_numpy(parse_blob(gv.sentinel_export_state(), w.B, w.T, w.d, params.l)["kinds"][ACT]["m"]).cuda()
    x3 = synth.clean(w, 0, ACT, 7, "cuda")
    gs3, _ = gv.verify(x3, ACT)
    sb.sentinel_sliced_wasserstein(x3, m3, u, want)
    torch.cuda.synchronize()
    assert torch.allclose(gs3[:, 3], want, rtol=2e-5, atol=0)
    gv.close()


def test_only_the_sliced_wasserstein_bit_with_mask_8(sb, oracle_mod):
    w = synth.scaled(synth.WORKLOADS["cfg1"], "sw_mask", 2, 32, 64)
    gv, ov, params = make_pair(sb, oracle_mod, w, metric_mask=8)
    with_directions(gv, ov, 4, w.d)
    for t in range(12):
        x = synth.clean(w, 0, ACT, t, "cuda")
        gv.update_reference(x, ACT)
        ov.update_reference(synth.bits(x), ACT)
    x = (synth.clean(w, 0, ACT, 12, "cuda").float() * 4.0).to(torch.bfloat16)
    gs, gf = gv.verify(x, ACT)
    os_, of, commit = ov.verify(synth.bits(x), ACT)
    gf = gf.cpu().numpy().view(np.uint32)
    assert np.array_equal(gf, of) and not commit
    assert np.all(gf & UNIT_BITS == sb.FLAG_SWD)
    assert_scores_close(gs.cpu().numpy(), os_, float(x.float().abs().mean()), "mask 8")
    gv.close()


def test_worker_iterations_with_four_metrics(sb, oracle_mod):
    """The multi-worker iteration with directions: every worker's launch is preceded by its own
    projection / sort chain; a banned worker's chain is skipped on the device."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "replicas_sw", 3, 20, 264)
    R = 4
    gv, ov, params = rep.pair(sb, oracle_mod, w, R, l=5, c=2)
    with_directions(gv, ov, 8, w.d)
    script = [("warm", {})] * 8 + [("verify", {})] * 2 + [("verify", {1: 6.0})] + [("verify", {})] + \
             [("verify", {1: 6.0})] + [("verify", {})] * 2
    near_events, k_events = 0, 0
    for t, (what, scale) in enumerate(script):
        xs = rep.inputs(w, R, ACT, t, scale)
        thr, valid = ov.thresholds(ACT)
        gs, gf, os_, of, n = rep.step_both(gv, ov, xs, ACT, warmup=(what == "warm"))
        assert gs.shape == (R, 1 + w.B, 4)
        for r in range(R):
            assert_scores_close(gs[r], os_[r], float(xs[r].float().abs().mean()), "step %d worker %d" % (t, r))
        if what != "warm" and not np.array_equal(gf, of):
            for r in range(R):
                near = near_threshold(os_[r], thr, valid, w.B)
                assert np.all(near[((gf[r] ^ of[r]) & UNIT_BITS) != 0]), (t, r, gf[r], of[r])
            near_events += 1
            gv.sentinel_import_state(oracle_to_blob(ov, params))
        ev = rep.whole_step_k_events(*gv.sentinel_get_thresholds(ACT), *ov.thresholds(ACT), params, ACT)
        if ev:
            k_events += ev
            gv.sentinel_import_state(oracle_to_blob(ov, params))
    print("re-alignments: %d near a bound, %d multiplier events" % (near_events, k_events))
    assert near_events <= 2 and k_events <= 4, (near_events, k_events)
    assert ov.worker_counters(1)[2] == 1                    # banned, then skipped
    rep.check_state(gv, ov, params, kinds=(ACT,))
    gv.close()


def test_directions_argument_checks(sb):
    gv = sb.Verifier(2, 8, 64)
    u = synth.directions(8, 64, 1, "cuda")
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_set_directions(synth.directions(5, 64, 1, "cuda"))      # L not 4, 8 or 16
    assert e.value.code == sb.ERR_UNSUPPORTED
    gv.sentinel_set_directions(u)
    gv.sentinel_set_directions(u)                                           # again, before any step: fine
    blob3 = sb.Verifier(2, 8, 64).sentinel_export_state()
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_import_state(blob3)                                     # a three-metric state
    assert e.value.code == sb.ERR_STATE_SIZE
    x = torch.zeros(2, 8, 64, dtype=torch.bfloat16, device="cuda")
    gv.update_reference(x, ACT)
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_set_directions(u)                                       # after the first step
    assert e.value.code == sb.ERR_INVALID_ARG
    wide = torch.zeros(2, 8, 65, dtype=torch.bfloat16, device="cuda")
    s, f = torch.zeros(3, 4, device="cuda"), torch.zeros(3, dtype=torch.int32, device="cuda")
    with pytest.raises(sb.SentinelError) as e:
        gv.sentinel_verify_strided(wide, ACT, s, f)                         # dense rows only
    assert e.value.code == sb.ERR_UNSUPPORTED
    gv.close()
    big = sb.Verifier(31, 8, 64)                                            # 100 * 32 = 3200 entries
    with pytest.raises(sb.SentinelError) as e:
        big.sentinel_set_directions(u)                                      # four windows' copies do not fit
    assert e.value.code == sb.ERR_UNSUPPORTED
    big.close()


def test_streams_in_lockstep_with_four_metrics_and_a_bf16_reference(sb, oracle_mod):
    """Directions on a verifier whose reference is stored as bf16: the reference is projected
    afresh every step (its stored values are rounded, so its projections do not follow Eq. 1's
    recursion); four columns in lockstep, the stored reference bit for bit."""
    w = synth.scaled(synth.WORKLOADS["cfg2"], "cfg2_sw_bf16", 4, 40, 264, corrupt_rate=0.25)
    gv, ov, params = make_pair(sb, oracle_mod, w, ema_bf16=1)
    with_directions(gv, ov, 8, w.d)
    rec = lockstep(sb, oracle_mod, w, gv, ov, params, 40)
    assert rec["corrupted"] >= 3
    st = parse_blob(gv.sentinel_export_state(), w.B, w.T, w.d, params.l)
    for kind in (ACT, GRAD):
        assert np.array_equal(st["kinds"][kind]["m"].astype(np.float64), ov.ema(kind))
        compare_thresholds(gv, ov, kind)
    assert rec["near"] <= 2 and rec["k_events"] <= 4, rec
    gv.close()
