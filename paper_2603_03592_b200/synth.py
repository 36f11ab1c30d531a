"""Seeded synthetic stage-boundary traffic.

Produces bf16 ``[B, T, d]`` tensors shaped and distributed like the activations ``h`` and
activation-gradients ``g`` that cross a pipeline-stage boundary, plus the corruptions a
malicious worker may apply (Sec. 2.1, "Attack Variants").  Nothing here is part of the
verification method: this module only draws inputs, so both the CUDA library's tests and the
CPU reference used to check it may import it.

Every microbatch is a pure function of ``(workload, boundary, kind, step)`` and the device
type, so any step -- a stale one included -- can be regenerated at will.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

ACT, GRAD = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    T: int
    d: int
    act: str              # "normal" | "lognormal_channel" | "student_t4"
    grad_std: float       # gradients ~ N(0, grad_std^2)
    warmup: int           # clean warm-up microbatches per kind
    steps: int            # verified microbatches per kind
    corrupt_rate: float
    corruptions: tuple    # names drawn uniformly for a corrupted step
    boundaries: int = 1
    uid: int = 0          # enters the seed


WORKLOADS = {
    # tiny single boundary: N(0,1), 16 warm-up microbatches, then sample 3 multiplied by 10
    "cfg1": Workload("cfg1", 8, 128, 512, "normal", 1e-3, 16, 1, 1.0, ("scale_sample3",), 1, 1),
    # small-LM stage traffic
    "cfg2": Workload("cfg2", 16, 1024, 2048, "lognormal_channel", 1e-3, 16, 200, 0.05,
                     ("add_gauss", "sign_flip"), 1, 2),
    # 1B-class stage traffic
    "cfg3": Workload("cfg3", 8, 4096, 4096, "lognormal_channel", 1e-3, 16, 500, 0.04,
                     ("zero_tokens", "stale50"), 1, 3),
    # wide-model stage traffic (512 MiB per tensor)
    "cfg4": Workload("cfg4", 4, 8192, 8192, "student_t4", 1e-4, 16, 100, 0.05,
                     ("add_uniform_sample",), 1, 4),
    # many-boundary sweep
    "cfg5": Workload("cfg5", 16, 2048, 4096, "lognormal_channel", 1e-3, 16, 64, 0.03,
                     ("add_gauss", "sign_flip", "zero_tokens", "stale50", "add_uniform_sample"),
                     8, 5),
}


def scaled(w: Workload, name: str, B: int, T: int, d: int, **kw) -> Workload:
    """The same recipe at another shape (used by tests that need seconds-sized inputs)."""
    fields = dict(w.__dict__)
    fields.update(name=name, B=B, T=T, d=d, **kw)
    return Workload(**fields)


def _seed(w: Workload, boundary: int, kind: int, step: int, salt: int = 0) -> int:
    s = (w.uid * 1_000_003 + boundary * 10_007 + kind * 101 + salt * 7_919) * 1_000_000 + step
    return s % (2 ** 63 - 1)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def channel_scale(w: Workload, boundary: int, device) -> torch.Tensor:
    """Per-channel scale ~ LogNormal(0, 0.5), fixed for the whole stream of a boundary."""
    g = _gen(device, _seed(w, boundary, 0, 0, salt=1))
    return torch.exp(0.5 * torch.randn(w.d, generator=g, device=device, dtype=torch.float32))


def clean(w: Workload, boundary: int, kind: int, step: int, device="cpu") -> torch.Tensor:
    """An honest worker's tensor for this step, fp32 values rounded to bf16 (RNE)."""
    g = _gen(device, _seed(w, boundary, kind, step))
    out = torch.empty(w.B, w.T, w.d, dtype=torch.bfloat16, device=device)
    scale = channel_scale(w, boundary, device) if (kind == ACT and w.act == "lognormal_channel") else None
    for b in range(w.B):  # one sample at a time bounds the fp32 scratch
        z = torch.randn(w.T, w.d, generator=g, device=device, dtype=torch.float32)
        if kind == GRAD:
            z.mul_(w.grad_std)
        elif w.act == "lognormal_channel":
            z.mul_(scale)
        elif w.act == "student_t4":
            chi = torch.zeros_like(z)
            for _ in range(4):
                r = torch.randn(w.T, w.d, generator=g, device=device, dtype=torch.float32)
                chi.addcmul_(r, r)
            z.div_(torch.sqrt(chi.div_(4.0))).mul_(0.5)
        out[b] = z.to(torch.bfloat16)
    return out


def corruption_of(w: Workload, boundary: int, kind: int, step: int) -> str | None:
    """Which corruption (if any) hits verified step ``step`` (0-based after warm-up)."""
    if step < w.warmup:
        return None
    g = _gen("cpu", _seed(w, boundary, kind, step, salt=2))
    u = torch.rand(2, generator=g)
    if float(u[0]) >= w.corrupt_rate:
        return None
    names = [n for n in w.corruptions if not (n == "sign_flip" and kind == ACT)] or list(w.corruptions)
    return names[min(int(float(u[1]) * len(names)), len(names) - 1)]


def corrupt(w: Workload, x: torch.Tensor, name: str, boundary: int, kind: int, step: int) -> torch.Tensor:
    """Apply one named corruption to a clean tensor."""
    device = x.device
    g = _gen(device, _seed(w, boundary, kind, step, salt=3))
    xf = x.float()
    if name == "scale_sample3":
        xf[3] *= 10.0
    elif name == "add_gauss":          # additive noise whose std equals the tensor's std
        xf += torch.randn(xf.shape, generator=g, device=device) * xf.std()
    elif name == "sign_flip":
        xf = -xf
    elif name == "zero_tokens":        # a random 10% of the token rows set to zero
        mask = torch.rand(w.B, w.T, generator=g, device=device) < 0.10
        xf[mask] = 0.0
    elif name == "stale50":            # replay of the tensor sent 50 steps earlier
        return clean(w, boundary, kind, max(step - 50, 0), device)
    elif name == "add_uniform_sample":  # U(-a, a) on one random sample, a = sqrt(3) * std(x)
        b = int(torch.randint(0, w.B, (1,), generator=g, device=device))
        a = float(xf.std()) * 3.0 ** 0.5
        xf[b] += (torch.rand(xf[b].shape, generator=g, device=device) * 2.0 - 1.0) * a
    else:
        raise ValueError(name)
    return xf.to(torch.bfloat16)


def microbatch(w: Workload, boundary: int, kind: int, step: int, device="cpu"):
    """(tensor, corruption name or None) for stream position ``step`` (warm-up steps first)."""
    x = clean(w, boundary, kind, step, device)
    name = corruption_of(w, boundary, kind, step)
    if name is not None:
        x = corrupt(w, x, name, boundary, kind, step)
    return x, name


def bits(x: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns on the host."""
    return x.detach().contiguous().view(torch.int16).cpu().numpy().view("uint16")


def directions(L: int, d: int, seed: int, device="cpu") -> torch.Tensor:
    """L random unit vectors of R^d as bf16 [L, d]: the directions a caller hands to the sliced
    Wasserstein metric (the paper fixes neither their number nor their draw)."""
    g = torch.Generator(device="cpu").manual_seed(0x5EED0000 + seed)
    u = torch.randn(L, d, generator=g, dtype=torch.float64)
    return (u / u.norm(dim=1, keepdim=True)).to(torch.bfloat16).contiguous().to(device)
