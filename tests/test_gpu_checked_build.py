"""The checked build of the library (the same sources compiled with -DSENTINEL_CHECK_BOUNDS):
every index its kernels derive from the shape is compared with the buffer's extent before the
access, and an access that would leave the buffer is skipped and counted.  The cases whose index
arithmetic is the most delicate -- ragged shapes, rows on every 2-byte misalignment with the
tensor ending where its allocation ends, the largest sizes, windows that wrap, the staged
kernels -- run through it here; the count must stay at zero, the error word of every handle too,
and the results must be those of the normal build.  Nothing here provokes a violation."""
import numpy as np
import pytest
import torch

from paper_2603_03592_b200 import synth

pytestmark = pytest.mark.gpu
ACT, GRAD = 0, 1


@pytest.fixture(scope="module")
def builds():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_03592_b200 import _build, binding
    checked = _build.build_checked()
    binding.use_library(None)
    binding.lib()
    yield binding, checked
    binding.use_library(None)


def on_both(binding, checked, fn):
    """fn(binding) with the normal build, then with the checked one; returns the two results."""
    out = []
    for path in (None, checked):
        binding.use_library(path)
        out.append(fn(binding))
        torch.cuda.synchronize()
    assert binding.sentinel_bounds_violations() == (0, 0)          # (asked of the checked build)
    binding.use_library(None)
    return out


def same(a, b):
    for x, y in zip(a, b):
        assert np.array_equal(np.asarray(x), np.asarray(y), equal_nan=True)


SHAPES = [(1, 1, 8), (2, 3, 8), (3, 5, 520), (4, 33, 1024), (2, 19, 4104), (64, 2, 64), (1, 2, 65536),
          (2, 5000, 8), (64, 1, 8), (5, 67, 1032)]


def test_stateless_distance_over_ragged_and_largest_shapes(builds):
    binding, checked = builds

    def run(sb):
        res = []
        for B, T, d in SHAPES:
            g = torch.Generator(device="cuda").manual_seed(B * 7 + T * 13 + d)
            x = (torch.randn(B, T, d, generator=g, device="cuda") * 1.7 + 0.3).to(torch.bfloat16)
            m = torch.randn(B, T, d, generator=g, device="cuda")
            s = torch.empty(1 + B, 3, device="cuda")
            st = torch.empty(1 + B, 8, device="cuda")
            sb.sentinel_distance(x, m, s, st)
            sb.sentinel_distance_noalloc(x, m, s, st)
            res += [s.cpu().numpy(), st.cpu().numpy()]
        return res

    same(*on_both(binding, checked, run))


@pytest.mark.parametrize("k,stride,offset", [(1024, 1025, 0), (512, 515, 3), (2056, 2057, 5), (264, 272, 7),
                                             (8, 9, 1), (1528, 1536, 2), (520, 521, 6), (72, 73, 4), (41, 57, 1)],
                         ids=lambda v: str(v))
def test_rows_on_every_misalignment_ending_with_the_allocation(builds, k, stride, offset):
    """Strided rows through the funnel-shift kernel (k a multiple of 8) and the scalar one, base
    offsets and strides that walk through all residues mod 16 bytes, both reference formats, the
    last row ending exactly where the allocation ends."""
    binding, checked = builds
    B, T = 3, 29
    w = synth.scaled(synth.WORKLOADS["cfg2"], "checked_shift", B, T, stride)
    n = B * T * stride

    def run(sb):
        res = []
        for bf16 in (0, 1):
            gv = sb.Verifier(B, T, k, ema_bf16=bf16, window_steps=4)
            for t in range(9):
                flat = torch.empty(offset + n, dtype=torch.bfloat16, device="cuda")
                wide = flat[offset:].view(B, T, stride)
                wide.copy_(synth.clean(w, 0, GRAD, t, "cuda"))
                gs = torch.empty(1 + B, 3, device="cuda")
                gf = torch.zeros(1 + B, dtype=torch.int32, device="cuda")
                if t < 4:
                    gv.sentinel_update_reference_strided(wide, GRAD, gs)
                else:
                    gv.sentinel_verify_strided(wide, GRAD, gs, gf)
                res += [gs.cpu().numpy(), gf.cpu().numpy()]
            assert gv.sentinel_get_counters()["error"] == 0
            gv.close()
        return res

    same(*on_both(binding, checked, run))


@pytest.mark.parametrize("variant", [dict(), dict(ema_bf16=1), dict(ref_over_batch=1), dict(ref_over_tokens=1),
                                     dict(ref_over_batch=1, ref_over_tokens=1)],
                         ids=["full", "bf16", "shared", "per_sample_vector", "one_vector"])
@pytest.mark.parametrize("shape", [(4, 33, 1032), (3, 70, 520), (2, 9, 4096)], ids=lambda s: "x".join(map(str, s)))
def test_streams_with_wrapping_windows(builds, variant, shape):
    """Warm-up and verified steps with a window of three steps (the rings wrap, entries are pushed
    out, the ascending copies are merged), the per-token buffer, gradient replacement and a state
    round trip, in every storage variant."""
    binding, checked = builds
    B, T, d = shape
    w = synth.scaled(synth.WORKLOADS["cfg3"], "checked_stream", B, T, d, corrupt_rate=0.3, warmup=4)

    def run(sb):
        res = []
        gv = sb.Verifier(B, T, d, window_steps=3, **variant)
        tok = None
        if not variant or variant == dict(ema_bf16=1):
            tok = torch.zeros(B, T, 4, device="cuda")
            gv.sentinel_set_token_stats_buffer(tok)
        for t in range(14):
            for kind in (ACT, GRAD):
                x, _ = synth.microbatch(w, 0, kind, t, "cuda")
                if t < w.warmup:
                    res.append(gv.update_reference(x, kind).cpu().numpy())
                else:
                    gs, gf = gv.verify(x, kind)
                    out = x.clone()
                    gv.sentinel_replace_if_flagged(out, kind, 0)
                    res += [gs.cpu().numpy(), gf.cpu().numpy(), out.view(torch.int16).cpu().numpy()]
        if tok is not None:
            res.append(tok.cpu().numpy())
        blob = gv.sentinel_export_state()
        gv.sentinel_import_state(blob)
        res.append(np.frombuffer(blob, dtype=np.uint8))
        assert gv.sentinel_get_counters()["error"] == 0
        gv.close()
        return res

    same(*on_both(binding, checked, run))


@pytest.mark.parametrize("shape,R", [((3, 12, 264), 4), ((2, 40, 1024), 3), ((4, 6, 64), 9)], ids=["R4", "R3", "R9"])
def test_iterations_with_several_workers(builds, shape, R):
    binding, checked = builds
    w = synth.scaled(synth.WORKLOADS["cfg2"], "checked_workers", *shape)

    def run(sb):
        res = []
        gv = sb.Verifier(w.B, w.T, w.d, n_workers=R, window_steps=3, ban_violations=2)
        for t in range(10):
            xs = [synth.clean(w, r, ACT, t, "cuda") for r in range(R)]
            if t in (6, 7, 8):
                xs[1] = (xs[1].float() * 6).to(torch.bfloat16)          # flagged, then banned and skipped
            gs, gf = gv.step_replicas(xs, ACT, warmup=t < 4)
            res += [gs.cpu().numpy(), gf.cpu().numpy()]
        assert gv.sentinel_get_counters()["error"] == 0
        gv.close()
        return res

    same(*on_both(binding, checked, run))


SWD_SHAPES = [((1, 1, 8), 4), ((3, 37, 520), 8), ((5, 100, 1024), 16), ((2, 1536, 264), 8), ((1, 2048, 136), 8),
              ((5, 1030, 40), 4), ((2, 1025, 64), 4)]


def test_sliced_wasserstein_sort_merge_and_w1_launches(builds):
    """The launches that follow the projections (sort per sample, whole and in halves; merge rounds with
    odd sample counts and token counts that are no multiple of the span; the last round with the
    W1 sums): stateless calls over ragged shapes, and a verifier with directions over a short stream."""
    binding, checked = builds

    def run(sb):
        res = []
        for (B, T, d), L in SWD_SHAPES:
            g = torch.Generator(device="cuda").manual_seed(B * 5 + T * 3 + d)
            x = (torch.randn(B, T, d, generator=g, device="cuda") * 1.1).to(torch.bfloat16)
            m = torch.randn(B, T, d, generator=g, device="cuda")
            out = torch.empty(1 + B, device="cuda")
            sb.sentinel_sliced_wasserstein(x, m, synth.directions(L, d, 3, "cuda"), out)
            res.append(out.cpu().numpy())
        w = synth.scaled(synth.WORKLOADS["cfg2"], "checked_swd", 3, 40, 264)
        gv = sb.Verifier(w.B, w.T, w.d, window_steps=4)
        gv.sentinel_set_directions(synth.directions(8, w.d, 1, "cuda"))
        for t in range(9):
            x = synth.clean(w, 0, ACT, t, "cuda")
            if t < 4:
                res.append(gv.update_reference(x, ACT).cpu().numpy())
            else:
                gs, gf = gv.verify(x, ACT)
                res += [gs.cpu().numpy(), gf.cpu().numpy()]
        assert gv.sentinel_get_counters()["error"] == 0
        gv.close()
        return res

    same(*on_both(binding, checked, run))
