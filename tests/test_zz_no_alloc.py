"""The no-allocation entry point (``sentinel_distance_noalloc``) against ``sentinel_distance``.

Some callers cannot let a library allocate device memory while it runs: they froze their memory
pool, were given a fixed device-memory budget, or sit in a loop where an allocator call of
unbounded duration is not acceptable.  For them the library keeps the kernel's scratch in a fixed
array of its own.  This file is collected last so that a failure here cannot hide another test's
result, and it must pass both alone in a fresh process and after the rest of the suite."""
import numpy as np
import pytest
import torch

from helpers import assert_scores_close, assert_stats_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_03592_b200 import binding
    binding.lib()
    return binding


def both(sb, x, m):
    B = x.shape[0]
    out = []
    for fn in (sb.sentinel_distance, sb.sentinel_distance_noalloc):
        scores = torch.full((1 + B, 3), -7.0, dtype=torch.float32, device="cuda")
        stats = torch.full((1 + B, 8), -7.0, dtype=torch.float32, device="cuda")
        fn(x, m, scores, stats)
        torch.cuda.synchronize()
        out.append((scores.cpu().numpy(), stats.cpu().numpy()))
    return out


def test_two_calls_in_a_row_match_the_allocating_entry_point(sb):
    g = torch.Generator(device="cuda").manual_seed(4242)
    # two different problems back to back: the second call finds the first one's leftovers in
    # the shared scratch (partial slots of another shape, a used ticket) and must not care
    for B, T, d in [(5, 67, 1032), (3, 200, 4096)]:
        x = (torch.randn(B, T, d, generator=g, device="cuda") * 1.3 - 0.2).to(torch.bfloat16)
        m = (0.5 * x.float() + torch.randn(B, T, d, generator=g, device="cuda")).contiguous()
        (s_ref, t_ref), (s_new, t_new) = both(sb, x, m)
        assert not np.any(s_new == -7.0) and not np.any(t_new == -7.0)
        scale = float(x.float().abs().mean())
        assert_scores_close(s_new, s_ref, scale, "noalloc scores %s" % ((B, T, d),))
        assert_stats_close(t_new, t_ref, float(x.float().std()), float(m.std()), "noalloc stats")


def test_repeated_calls_on_one_stream_without_synchronising(sb):
    g = torch.Generator(device="cuda").manual_seed(99)
    B, T, d = 4, 128, 2048
    xs = [(torch.randn(B, T, d, generator=g, device="cuda") * (i + 1)).to(torch.bfloat16) for i in range(3)]
    m = torch.randn(B, T, d, generator=g, device="cuda")
    want = []
    for x in xs:
        s = torch.empty(1 + B, 3, device="cuda")
        sb.sentinel_distance(x, m, s)
        want.append(s)
    got = [torch.empty(1 + B, 3, device="cuda") for _ in xs]
    for x, s in zip(xs, got):                       # stream-ordered, no host sync in between
        sb.sentinel_distance_noalloc(x, m, s)
    torch.cuda.synchronize()
    for w, s, x in zip(want, got, xs):
        assert_scores_close(s.cpu().numpy(), w.cpu().numpy(), float(x.float().abs().mean()), "back to back")


def test_invalid_arguments_are_rejected_before_any_launch(sb):
    x = torch.zeros(2, 4, 16, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(2, 4, 16, device="cuda")
    s = torch.zeros(3, 3, device="cuda")
    L = sb.lib()
    st = torch.cuda.current_stream().cuda_stream
    assert L.sentinel_distance_noalloc(x.data_ptr(), None, 2, 4, 16, 0, st, s.data_ptr(), None) == sb.ERR_INVALID_ARG
    assert L.sentinel_distance_noalloc(x.data_ptr(), m.data_ptr(), 2, 4, 12, 0, st, s.data_ptr(), None) == sb.ERR_UNALIGNED
    assert L.sentinel_distance_noalloc(x.data_ptr(), m.data_ptr(), 65, 4, 16, 0, st, s.data_ptr(), None) == sb.ERR_UNSUPPORTED
    assert L.sentinel_distance_noalloc(x.data_ptr(), m.data_ptr(), 2, 4, 16, 99, st, s.data_ptr(), None) == sb.ERR_INVALID_ARG
    assert b"device" in L.sentinel_last_error(None)


def test_calls_after_the_first_take_no_device_memory(sb):
    """What the entry point is for: once its first call on the device has looked up the built-in
    array, further calls leave the device's free memory exactly where it was (cudaMemGetInfo
    before and after, with every tensor of the test created beforehand)."""
    g = torch.Generator(device="cuda").manual_seed(7)
    B, T, d = 6, 96, 1024
    xs = [(torch.randn(B, T, d, generator=g, device="cuda")).to(torch.bfloat16) for _ in range(4)]
    m = torch.randn(B, T, d, generator=g, device="cuda")
    outs = [torch.empty(1 + B, 3, device="cuda") for _ in xs]
    stats = [torch.empty(1 + B, 8, device="cuda") for _ in xs]
    sb.sentinel_distance_noalloc(xs[0], m, outs[0], stats[0])      # the priming call
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(5):
        for x, s, st in zip(xs, outs, stats):
            sb.sentinel_distance_noalloc(x, m, s, st)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    # (the arithmetic of the refusal: 256 bytes of ticket and two 64-byte slots per streaming CTA
    # must fit the array; this device's launch does, with room)
    import re, os
    header = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "sentinel.h")).read()
    size = int(re.search(r"#define\s+SENTINEL_NOALLOC_SCRATCH_BYTES\s+\(?(\d+)", header).group(1))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert 256 + 2 * 64 * sms <= size
