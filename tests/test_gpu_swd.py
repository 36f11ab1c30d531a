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
         ((8, 64, 512), 4), ((7, 33, 264), 16), ((1, 700, 136), 8)]


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
