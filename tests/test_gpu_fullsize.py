"""GPU parity at the benchmark's full sizes, in the launch configuration ``bench.py`` times
(same entry points, same shapes): every score of every unit and every flag against the float64
oracle run on the same tensors.  Here: the variants (several workers, the storage forms of the
reference, the sliced Wasserstein distance), a few steps each."""
import numpy as np
import pytest
import torch

from helpers import UNIT_BITS, assert_scores_close, assert_stats_close, near_threshold
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


def run_steps(sb, oracle_mod, w, kind, n_warm, corruption, directions=0, **variant):
    gv = sb.Verifier(w.B, w.T, w.d, **variant)
    ov = oracle_mod.Verifier(oracle_mod.Params(B=w.B, T=w.T, d=w.d, **variant))
    if directions:                                          # the sliced Wasserstein distance as a fourth metric
        u = synth.directions(directions, w.d, 7, "cuda")
        gv.sentinel_set_directions(u)
        ov.set_directions(synth.bits(u))
    for t in range(n_warm):
        x = synth.clean(w, 0, kind, t, "cuda")
        gs = gv.update_reference(x, kind)
        os_, _ = ov.update_reference(synth.bits(x), kind)
        assert_scores_close(gs.cpu().numpy(), os_, float(x.float().abs().mean()), "%s warm-up %d" % (w.name, t))
        st = gv.sentinel_get_stats(kind).cpu().numpy()
        assert_stats_close(st, ov.last_stats(kind), float(x.float().std()),
                           max(float(np.abs(ov.last_stats(kind)[0, 4])) ** 0.5, 1e-30), "%s stats %d" % (w.name, t))
    # a clean verified step, then a corrupted one
    near_events = 0
    for t, name in ((n_warm, None), (n_warm + 1, corruption)):
        x = synth.clean(w, 0, kind, t, "cuda")
        if name:
            x = synth.corrupt(w, x, name, 0, kind, t)
        thr, valid = ov.thresholds(kind)
        gs, gf = gv.verify(x, kind)
        os_, of, commit = ov.verify(synth.bits(x), kind)
        gs, gf = gs.cpu().numpy(), gf.cpu().numpy().view(np.uint32)
        assert_scores_close(gs, os_, float(x.float().abs().mean()), "%s verify (%s)" % (w.name, name))
        if not np.array_equal(gf, of):
            near = near_threshold(os_, thr, valid, w.B)
            assert np.all(near[((gf ^ of) & UNIT_BITS) != 0]), (gf, of)
            near_events += 1
        assert bool(gf[0] & sb.FLAG_COMMITTED) == commit
    assert near_events <= 1, near_events
    c = gv.sentinel_get_counters()
    assert (c["violations"], c["clean_streak"], c["banned"]) == ov.counters()
    gv.close()


# (The plain verifier at the full shapes of configurations 2 to 5 -- whole streams, both kinds, in
# lockstep with oracle processes -- is test_gpu_streams_as_stated.py.)


# ---------------------------------------------------------------------------------------------
# the variants at full size, through properties that hold at any size

def test_cfg4_identical_workers_reduce_to_one_submission(sb):
    """Four workers handing in the same 4 x 8192 x 8192 tensor: every worker's scores are those of
    the single-submission call (other summation order: 1e-5), and the mean over four equal
    tensors is that tensor, so the reference moves exactly (bit for bit) as it does for one
    submission -- through the one-launch kernel and its speculative mean."""
    w = synth.WORKLOADS["cfg4"]
    R = 4
    one = sb.Verifier(w.B, w.T, w.d)
    many = sb.Verifier(w.B, w.T, w.d, n_workers=R, window_steps=50)
    n = 4 * w.B * w.T * w.d

    def act_reference(verifier):        # the reference is the tail of the first kind block of the blob
        blob = verifier.sentinel_export_state()
        per_kind = (verifier.sentinel_state_bytes() - 64 - 192) // 2
        return np.frombuffer(blob, dtype=np.uint8, count=n, offset=64 + 192 + per_kind - n)

    for t in range(5):
        x = synth.clean(w, 0, ACT, t, "cuda")
        warm = t < 4
        if warm:
            s1, committed = one.update_reference(x, ACT), True
        else:
            s1, f1 = one.verify(x, ACT)
            committed = bool(int(f1[0]) & sb.FLAG_COMMITTED)
        sr, fr = many.step_replicas([x] * R, ACT, warmup=warm)
        torch.cuda.synchronize()
        for r in range(R):
            assert torch.allclose(sr[r], s1, rtol=1e-5, atol=1e-7), (t, r)
        if committed:                   # (a flagged step: four of four is a majority, another rule applies)
            assert all(int(fr[r, 0]) & sb.FLAG_COMMITTED for r in range(R))
            assert np.array_equal(act_reference(one), act_reference(many)), t
    one.close(); many.close()


def test_cfg3_two_workers_against_the_oracle(sb, oracle_mod):
    """8 x 4096 x 4096, two workers per iteration: two warm-up iterations, a clean verified one and
    one in which worker 1 submits a tensor five times too large -- every worker's scores, flags
    and counters, and a sample of the reference after the mean over the clean workers."""
    w = synth.WORKLOADS["cfg3"]
    R = 2
    gv = sb.Verifier(w.B, w.T, w.d, n_workers=R)
    ov = oracle_mod.Verifier(oracle_mod.Params(B=w.B, T=w.T, d=w.d, R=R))
    near_events = 0
    for t in range(4):
        xs = [synth.clean(w, r, GRAD, t, "cuda") for r in range(R)]
        if t == 3:
            xs[1] = (xs[1].float() * 5).to(torch.bfloat16)
        thr, valid = ov.thresholds(GRAD)
        gs, gf = gv.step_replicas(xs, GRAD, t < 2)
        os_, of, n_clean = ov.step_replicas([synth.bits(x) for x in xs], GRAD, t < 2)
        torch.cuda.synchronize()
        gs, gf = gs.cpu().numpy(), gf.cpu().numpy().view(np.uint32)
        for r in range(R):
            assert_scores_close(gs[r], os_[r], float(xs[r].float().abs().mean()), "iteration %d worker %d" % (t, r))
        if t >= 2 and not np.array_equal(gf, of):
            for r in range(R):
                near = near_threshold(os_[r], thr, valid, w.B)
                assert np.all(near[((gf[r] ^ of[r]) & UNIT_BITS) != 0]), (t, r, gf[r], of[r])
            near_events += 1
        if t == 3:
            assert of[1, 0] & UNIT_BITS and not (of[0, 0] & UNIT_BITS) and n_clean == 1
    assert near_events == 0, near_events                    # (the counters below would differ otherwise)
    for r in range(R):
        assert gv.sentinel_get_worker_counters(r) == ov.worker_counters(r)
    blob = gv.sentinel_export_state()
    per_kind = (gv.sentinel_state_bytes() - 64 - 192) // 2
    n = w.B * w.T * w.d
    m_gpu = np.frombuffer(blob, dtype="<f4", count=n, offset=64 + 192 + 2 * per_kind - 4 * n)   # the gradients' reference
    m_ref = ov.ema(GRAD).reshape(-1)
    idx = np.random.default_rng(0).integers(0, n, 200000)
    assert np.max(np.abs(m_gpu[idx] - m_ref[idx])) <= 1e-5 * float(np.abs(m_ref[idx]).max())
    gv.close()


def test_cfg4_bf16_reference_first_update(sb):
    """From m_0 = 0 one update leaves bf16((1-beta) x) in single precision, here checked on the
    whole 4 x 8192 x 8192 tensor against torch's multiply and conversion."""
    w = synth.WORKLOADS["cfg4"]
    gv = sb.Verifier(w.B, w.T, w.d, ema_bf16=1)
    x = synth.clean(w, 0, ACT, 0, "cuda")
    gs = gv.update_reference(x, ACT)
    blob = gv.sentinel_export_state()
    per_kind = (gv.sentinel_state_bytes() - 64 - 192) // 2
    n = w.B * w.T * w.d
    m = torch.from_numpy(np.frombuffer(blob, dtype=np.float32, count=n, offset=64 + 192 + per_kind - 4 * n).copy())
    want = (x.float() * float(np.float32(1.0 - 0.9))).to(torch.bfloat16).float().cpu().reshape(-1)
    assert torch.equal(m, want)
    # the first warm-up step runs against m = 0: L1 = mean |x|, sign flips = share of non-zero x
    assert float(gs[0, 0]) == pytest.approx(float(x.float().abs().mean()), rel=1e-5)
    assert float(gs[0, 2]) == pytest.approx(float((x != 0).float().mean()), rel=1e-6)
    gv.close()


def test_cfg4_shared_reference_of_identical_samples(sb):
    """4 x 8192 x 8192 with one [T,d] reference: when all samples of every tensor are the same
    [T,d] slice, the mean over the samples is that slice, so the reference and every sample's
    scores are those of a one-sample verifier fed the slice (the reference bit for bit)."""
    w = synth.WORKLOADS["cfg4"]
    one = sb.Verifier(1, w.T, w.d)
    shared = sb.Verifier(w.B, w.T, w.d, ref_over_batch=1)
    for t in range(4):
        sl = synth.clean(w, 0, ACT, t, "cuda")[:1].contiguous()
        x = sl.expand(w.B, w.T, w.d).contiguous()
        s1 = one.update_reference(sl, ACT)
        ss = shared.update_reference(x, ACT)
        torch.cuda.synchronize()
        for r in range(1 + w.B):                 # the whole tensor is B copies of the slice: same scores again
            assert torch.allclose(ss[r], s1[1], rtol=1e-5, atol=1e-7), (t, r)
    n = 4 * w.T * w.d
    def act_reference(v):
        blob = v.sentinel_export_state()
        per_kind = (v.sentinel_state_bytes() - 64 - 192) // 2
        return np.frombuffer(blob, dtype=np.uint8, count=n, offset=64 + 192 + per_kind - n)
    assert np.array_equal(act_reference(one), act_reference(shared))
    one.close(); shared.close()


def test_cfg4_compressed_layout_equals_the_dense_call_bit_for_bit(sb):
    """4 x 8192 x 8192 inside a [4, 8192, 8193] tensor (rows on every 2-byte boundary): the
    funnel-shifted loads hand the arithmetic the same words as the dense call gets, so scores,
    flags and the whole exported state are the same bits."""
    w = synth.WORKLOADS["cfg4"]
    dense, wide_v = sb.Verifier(w.B, w.T, w.d), sb.Verifier(w.B, w.T, w.d)
    for t in range(4):
        x = synth.clean(w, 0, GRAD, t, "cuda")
        if t == 3:
            x = synth.corrupt(w, x, "add_uniform_sample", 0, GRAD, t)
        wide = torch.nn.functional.pad(x, (0, 1), value=77.0).contiguous()
        s2 = torch.empty(1 + w.B, 3, device="cuda")
        if t < 2:
            s1 = dense.update_reference(x, GRAD)
            wide_v.sentinel_update_reference_strided(wide, GRAD, s2)
        else:
            s1, f1 = dense.verify(x, GRAD)
            f2 = torch.empty(1 + w.B, dtype=torch.int32, device="cuda")
            wide_v.sentinel_verify_strided(wide, GRAD, s2, f2)
            assert torch.equal(f1, f2), t
        torch.cuda.synchronize()
        assert torch.equal(s1, s2), t
        del wide
    assert bytes(dense.sentinel_export_state()) == bytes(wide_v.sentinel_export_state())
    dense.close(); wide_v.close()


def test_cfg4_channel_reference_against_the_oracle(sb, oracle_mod):
    """4 x 8192 x 8192 with one [d] reference for all tokens: two warm-up steps, a clean and a
    corrupted verified step, every score, statistic, flag and counter against the oracle."""
    run_steps(sb, oracle_mod, synth.WORKLOADS["cfg4"], ACT, 2, "add_uniform_sample", ref_over_batch=1, ref_over_tokens=1)


def test_cfg4_channel_reference_per_sample_against_the_oracle(sb, oracle_mod):
    """The same with a vector per sample ([B,d])."""
    run_steps(sb, oracle_mod, synth.WORKLOADS["cfg4"], GRAD, 2, "add_uniform_sample", ref_over_tokens=1)


def test_cfg4_steps_with_four_metrics_against_the_oracle(sb, oracle_mod):
    """4 x 8192 x 8192 with 8 directions as the verifier's fourth metric: two warm-up steps (the second
    one takes the reference's projections from the recursion), a clean verified step and one with
    uniform noise on a sample -- all four scores of every unit, flags and counters."""
    run_steps(sb, oracle_mod, synth.WORKLOADS["cfg4"], ACT, 2, "add_uniform_sample", directions=8)


def test_cfg4_sliced_wasserstein_units(sb, oracle_mod):
    """4 x 8192 x 8192, 8 directions.  Two samples against the float64 oracle (projections of
    8192 tokens in R^8192 each); and the whole-tensor unit through a property: a tensor made of
    four copies of one sample, against a reference made of four copies of one slice, has the
    same empirical distributions along every direction as the single sample, hence the same
    distance."""
    w = synth.WORKLOADS["cfg4"]
    u = synth.directions(8, w.d, 5, "cuda")
    x = synth.clean(w, 0, ACT, 0, "cuda")
    m = (0.7 * synth.clean(w, 0, ACT, 1, "cuda").float() + 0.05).contiguous()
    out = torch.empty(1 + w.B, device="cuda")
    sb.sentinel_sliced_wasserstein(x, m, u, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    ub = synth.bits(u)
    for b in (0, 3):
        want = oracle_mod.sliced_wasserstein(synth.bits(x[b]), m[b].double().cpu().numpy(), ub)[0]
        assert abs(got[1 + b] - want) <= 1e-3 * want, (b, got[1 + b], want)
    assert np.all(np.isfinite(got)) and got[0] > 0
    xs = x[:1].expand(w.B, w.T, w.d).contiguous()
    ms = m[:1].expand(w.B, w.T, w.d).contiguous()
    sb.sentinel_sliced_wasserstein(xs, ms, u, out)
    torch.cuda.synchronize()
    tiled = out.cpu().numpy().astype(np.float64)
    assert np.allclose(tiled[1:], got[1], rtol=1e-6)
    assert tiled[0] == pytest.approx(got[1], rel=1e-5)
