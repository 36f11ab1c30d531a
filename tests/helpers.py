"""Shared helpers of the GPU parity tests: tolerances, oracle <-> library state blobs."""
from __future__ import annotations

import struct

import numpy as np

REL = 1e-3            # statistics and scores: relative error allowed against the float64 oracle
MAGIC = 0x4C454E49544E4553
METRIC_MASK = 0xF
UNIT_BITS = 0xFFFF


def assert_scores_close(gpu, ref, x_scale, what=""):
    """|gpu - ref| <= 1e-3 * max(|ref|, floor).  Floors: 1e-3 for the bounded scores (L2z in
    [0,4], SFR in [0,1]: an absolute 1e-6, the resolution fp32 products leave on a
    correlation), 1e-3 * mean|x| for L1 and for the sliced Wasserstein distance (a fourth
    column, present when the verifier has directions)."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    floors = np.array([1e-3 * x_scale, 1e-3, 1e-3, 1e-3 * x_scale])[:gpu.shape[-1]]
    both_nan = np.isnan(gpu) & np.isnan(ref)
    tol = REL * np.maximum(np.abs(ref), floors)
    bad = ~both_nan & ~(np.abs(gpu - ref) <= tol)
    assert not bad.any(), "%s scores differ: gpu=%s ref=%s" % (what, gpu[bad][:6], ref[bad][:6])


def assert_stats_close(gpu, ref, x_scale, m_scale, what=""):
    """Same rule for mean_x var_x |x| mean_m var_m cov |m| rho; floors follow each
    quantity's natural scale (a mean is compared on the scale of the standard deviation)."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    sx, sm = max(x_scale, 1e-30), max(m_scale, 1e-30)
    floors = np.array([sx, sx * sx, sx, sm, sm * sm, sx * sm, sm, 1.0]) * 1e-3
    both_nan = np.isnan(gpu) & np.isnan(ref)
    tol = REL * np.maximum(np.abs(ref), floors)
    bad = ~both_nan & ~(np.abs(gpu - ref) <= tol)
    assert not bad.any(), "%s stats differ: gpu=%s ref=%s" % (what, gpu[bad][:6], ref[bad][:6])


def near_threshold(scores, thr, valid, B, rel=REL):
    """Rows whose score lies within `rel` of a bound it is tested against (oracle values)."""
    near = np.zeros(1 + B, dtype=bool)
    for r in range(1 + B):
        L = 0 if r == 0 else 1
        for i in range(scores.shape[1]):
            if not valid[L, i] or np.isnan(scores[r, i]):
                continue
            for bound in (thr[L, i, 4], thr[L, i, 5]):
                if abs(scores[r, i] - bound) <= rel * max(abs(bound), 1e-30):
                    near[r] = True
    return near


# ---------------------------------------------------------------------------------------------
# state blobs (layout documented in include/sentinel.h)

def oracle_to_blob(v, params) -> bytes:
    """Serialise an oracle verifier into the library's checkpoint format."""
    B, T, d, l, R = params.B, params.T, params.d, params.l, params.R
    M = v.nm                                   # metrics in use; the layout has room for four
    # 0: [B,T,d] reference, 1: one [T,d] reference for all samples, 2: one [d] reference for all
    # tokens, 3: a [B,d] reference, one vector per sample
    over_b, over_t = int(getattr(params, "ref_over_batch", 0)), int(getattr(params, "ref_over_tokens", 0))
    shared = {(0, 0): 0, (1, 0): 1, (1, 1): 2, (0, 1): 3}[(over_b, over_t)]
    out = bytearray(struct.pack("<QI7i", MAGIC, 3, B, T, d, l, R, M, shared))
    out += b"\0" * (64 - len(out))
    workers = np.zeros((3, 16), dtype="<i4")
    for r in range(R):
        workers[:, r] = v.worker_counters(r)
    out += workers.tobytes()
    for kind in (0, 1):
        thr, valid = v.thresholds(kind)
        counts = [v.history(kind, L, 0).size for L in (0, 1)]
        valid4 = np.zeros((2, 4), dtype=int)
        valid4[:, :M] = valid
        thr4 = np.zeros((2, 4, 6))
        thr4[:, :M] = thr
        out += struct.pack("<q2i8i", v.steps(kind), *counts, *valid4.reshape(-1))
        out += thr4.astype("<f8").tobytes()
        for L, cap in ((0, l * R), (1, l * R * B)):
            for i in range(4):
                h = np.zeros(cap)
                if i < M:
                    hv = v.history(kind, L, i)
                    h[:hv.size] = hv
                out += h.astype("<f8").tobytes()
        out += v.ema(kind).astype("<f4").tobytes()
    return bytes(out)


def parse_blob(blob, B, T, d, l, R=1) -> dict:
    """Decode a checkpoint blob into plain numpy pieces."""
    buf = memoryview(bytes(blob))
    magic, version, b, t, dd, ll, rr, M, shared = struct.unpack_from("<QI7i", buf, 0)
    assert magic == MAGIC and version == 3 and (b, t, dd, ll, rr) == (B, T, d, l, R) and M in (3, 4)
    workers = np.frombuffer(buf, dtype="<i4", count=48, offset=64).reshape(3, 16)
    off = 64 + 192
    out = {"violations": int(workers[0, 0]), "clean_streak": int(workers[1, 0]), "banned": int(workers[2, 0]),
           "workers": workers.copy(), "n_metrics": M, "ref_over_batch": shared, "kinds": []}
    ref_shape = {0: (B, T, d), 1: (T, d), 2: (d,), 3: (B, d)}[shared]
    N = int(np.prod(ref_shape))
    for _ in range(2):
        steps, c0, c1 = struct.unpack_from("<q2i", buf, off)
        valid = np.array(struct.unpack_from("<8i", buf, off + 16)).reshape(2, 4).astype(bool)[:, :M]
        off += 48
        thr = np.frombuffer(buf, dtype="<f8", count=48, offset=off).reshape(2, 4, 6)[:, :M].copy()
        off += 384
        hist = [[None] * M, [None] * M]
        for L, cap, cnt in ((0, l * R, c0), (1, l * R * B, c1)):
            for i in range(4):
                if i < M:
                    hist[L][i] = np.frombuffer(buf, dtype="<f8", count=cap, offset=off)[:cnt].copy()
                off += 8 * cap
        m = np.frombuffer(buf, dtype="<f4", count=N, offset=off).reshape(ref_shape).copy()
        off += 4 * N
        out["kinds"].append({"steps": steps, "count": (c0, c1), "valid": valid, "thr": thr,
                             "hist": hist, "m": m})
    assert off == len(buf)
    return out


def whole_step_k_events(gt, gvalid, ot, ovalid, params, kind) -> int:
    """Alg. 5 compares every window entry with a fence; an entry that lies on a fence to within the
    score tolerance may fall on either side, which moves k by whole widen/narrow steps.  Returns
    the number of (level, metric) windows where the two multipliers differ that way; any other
    difference fails."""
    assert np.array_equal(gvalid, ovalid)
    events = 0
    lg, ls = np.log(params.gamma_g[kind]), np.log(params.gamma_s[kind])
    n = params.n_max[kind]
    for L in range(2):
        for i in range(ovalid.shape[1]):
            if not ovalid[L, i] or abs(gt[L, i, 3] / ot[L, i, 3] - 1.0) <= 1e-12:
                continue
            r = np.log(gt[L, i, 3] / ot[L, i, 3])
            whole = any(abs(r - (a * lg + b * ls)) < 1e-9 for a in range(-n, n + 1) for b in range(-n, n + 1))
            assert whole, "k differs by no whole number of steps: %r vs %r" % (gt[L, i, 3], ot[L, i, 3])
            events += 1
    return events


def assert_thresholds_close(gt, ot, valid, params, kind, what=""):
    """Bounds of Alg. 5, library against oracle.  The quartiles are functions of scores that agree
    to 1e-3, so they are compared at 1e-3 on the scale of the median.  tau = q2 -+ k*IQR amplifies
    a difference of the quartiles k-fold (k reaches the hundreds where a window is narrow), so the
    bounds are checked for what they must be: Alg. 5's last lines applied to the library's own
    quartiles and multiplier, to rounding."""
    lam, eps = params.lam[kind], params.eps[kind]
    for L in range(2):
        for i in range(valid.shape[1]):
            if not valid[L, i]:
                continue
            q1, q2, q3, k, lo, hi = gt[L, i]
            tol = REL * np.maximum(np.abs(ot[L, i, :3]), abs(ot[L, i, 1]))
            assert np.all(np.abs(gt[L, i, :3] - ot[L, i, :3]) <= tol), (what, L, i, gt[L, i], ot[L, i])
            iqr = max(q3 - q1, eps)
            want_lo = min(q2 - k * iqr, q2 - lam * abs(q2))
            want_hi = max(q2 + k * iqr, q2 + lam * abs(q2))
            scale = max(abs(q2), k * iqr, 1e-300)
            assert abs(lo - want_lo) <= 1e-12 * scale and abs(hi - want_hi) <= 1e-12 * scale, (what, L, i, gt[L, i])
