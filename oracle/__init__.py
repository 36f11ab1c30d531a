"""Reference oracle for the Sentinel verifier check -- TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper around ``sentinel_oracle.c`` (plain C, float64), which restates the
paper's definitions: the distance measures of Sec. 3.1, the EMA of Eq. (1), the per-submission
body of Alg. 2 / Alg. 3, the warm-up loop of Alg. 1 and the adaptive IQR thresholds of Alg. 5.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and does not import it.

Parity unpinned (conventions the paper leaves open, each a parameter): the reading of
"FP-rate << alpha" (``shrink_ratio``), the severe-deviation multiple (``severe_mult``), the
forgiveness bookkeeping, and the percentile interpolation rule.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sentinel_oracle.c")
_HDR = os.path.join(_HERE, "sentinel_oracle.h")
_LIB = os.path.join(_HERE, "libsentinel_oracle.so")

ACT, GRAD = 0, 1
L1, L2Z, SFR = 0, 1, 2
NMETRIC, NSTAT, NTHR = 4, 8, 6   # room for four metrics; a verifier uses three until directions are set

FLAG_L1, FLAG_L2Z, FLAG_SFR, FLAG_SW = 1 << 0, 1 << 1, 1 << 2, 1 << 3
FLAG_NONFINITE = 1 << 7
FLAG_COMMITTED, FLAG_SEVERE, FLAG_BANNED, FLAG_NO_THRESHOLDS = 1 << 16, 1 << 17, 1 << 18, 1 << 19
FLAG_NATURAL_SHIFT = 1 << 20
FLAG_TAINTED_ELSEWHERE = 1 << 21
METRIC_BITS = FLAG_L1 | FLAG_L2Z | FLAG_SFR | FLAG_SW


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no CUDA involved); returns the library path."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [
        ("beta", C.c_double * 2), ("k0", C.c_double * 2), ("alpha", C.c_double * 2),
        ("n_max", C.c_int * 2), ("gamma_g", C.c_double * 2), ("gamma_s", C.c_double * 2),
        ("lam", C.c_double * 2), ("eps", C.c_double * 2),
        ("shrink_ratio", C.c_double), ("severe_mult", C.c_double),
        ("l", C.c_int), ("c", C.c_int), ("t_forgiveness", C.c_int),
        ("metric_mask", C.c_uint), ("B", C.c_int), ("T", C.c_int), ("d", C.c_int),
        ("R", C.c_int), ("ema_bf16", C.c_int), ("ref_over_batch", C.c_int), ("ref_over_tokens", C.c_int),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        dp, u16p = C.POINTER(C.c_double), C.POINTER(C.c_uint16)
        L.so_default_params.argtypes = [C.POINTER(_Params)]
        L.so_default_params.restype = None
        L.so_bf16.argtypes = [C.c_uint16]
        L.so_bf16.restype = C.c_double
        L.so_distance.argtypes = [u16p, dp, C.c_size_t, dp, dp]
        L.so_distance.restype = C.c_int
        L.so_token_sums.argtypes = [u16p, dp, C.c_size_t, dp]
        L.so_token_sums.restype = None
        L.so_out_of_bounds.argtypes = [C.c_double, C.c_double, C.c_double]
        L.so_out_of_bounds.restype = C.c_int
        L.so_severe.argtypes = [C.c_int, C.c_double, C.c_double, C.c_double, C.c_double]
        L.so_severe.restype = C.c_int
        L.so_percentile.argtypes = [dp, C.c_size_t, C.c_double]
        L.so_percentile.restype = C.c_double
        L.so_adaptive_iqr.argtypes = [dp, C.c_size_t, C.c_double, C.c_int, C.c_double,
                                      C.c_double, C.c_double, C.c_double, C.c_double, dp,
                                      C.POINTER(C.c_int)]
        L.so_adaptive_iqr.restype = C.c_int
        L.so_create.argtypes = [C.POINTER(_Params)]
        L.so_create.restype = C.c_void_p
        L.so_destroy.argtypes = [C.c_void_p]
        L.so_set_directions.argtypes = [C.c_void_p, u16p, C.c_int]
        L.so_set_directions.restype = C.c_int
        L.so_destroy.restype = None
        L.so_update_reference.argtypes = [C.c_void_p, u16p, C.c_int, dp]
        L.so_update_reference.restype = C.c_int
        L.so_verify.argtypes = [C.c_void_p, u16p, C.c_int, dp, C.POINTER(C.c_uint32)]
        L.so_verify.restype = C.c_int
        L.so_sliced_wasserstein.argtypes = [u16p, dp, C.c_size_t, C.c_size_t, u16p, C.c_size_t, dp]
        L.so_sliced_wasserstein.restype = C.c_double
        L.so_bf16_round.argtypes = [C.c_double]
        L.so_bf16_round.restype = C.c_uint16
        L.so_replace_if_flagged.argtypes = [C.c_void_p, u16p, C.c_int, C.c_int]
        L.so_replace_if_flagged.restype = C.c_int
        L.so_step_replicas.argtypes = [C.c_void_p, C.POINTER(u16p), C.c_int, C.c_int, C.c_uint, dp, C.POINTER(C.c_uint32)]
        L.so_skip_tainted.argtypes = [C.c_void_p, C.c_int]
        L.so_skip_tainted.restype = None
        L.so_step_replicas.restype = C.c_int
        L.so_count_violation.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int]
        L.so_count_violation.restype = None
        L.so_worker_counters.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int)]
        L.so_worker_counters.restype = None
        L.so_reset_worker.argtypes = [C.c_void_p]
        L.so_reset_worker.restype = None
        L.so_ema.argtypes = [C.c_void_p, C.c_int]
        L.so_ema.restype = dp
        L.so_set_ema.argtypes = [C.c_void_p, C.c_int, dp]
        L.so_set_ema.restype = None
        L.so_history.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, dp, C.c_size_t]
        L.so_history.restype = C.c_size_t
        L.so_thresholds.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, dp]
        L.so_thresholds.restype = C.c_int
        L.so_last_stats.argtypes = [C.c_void_p, C.c_int, dp]
        L.so_last_stats.restype = None
        L.so_counters.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
        L.so_counters.restype = None
        L.so_steps.argtypes = [C.c_void_p, C.c_int]
        L.so_steps.restype = C.c_long
        _lib = L
    return _lib


def _dptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _bits(x) -> np.ndarray:
    """bf16 bit patterns as a contiguous uint16 array (accepts uint16/int16 arrays)."""
    a = np.ascontiguousarray(x)
    if a.dtype == np.int16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("bf16 input must be given as uint16 bit patterns")
    return a


def _u16ptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_uint16))


def bf16_to_f64(bits) -> np.ndarray:
    """bf16 bit patterns -> float64 values (exact)."""
    b = _bits(bits)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


@dataclass
class Params:
    """Hyper-parameters (index 0 = activations, 1 = gradients); defaults from the paper."""
    B: int = 1
    T: int = 1
    d: int = 8
    beta: tuple = (0.90, 0.80)
    k0: tuple = (1.5, 3.0)
    alpha: tuple = (1e-4, 1e-3)
    n_max: tuple = (10, 10)
    gamma_g: tuple = (1.1, 1.01)
    gamma_s: tuple = (0.9, 0.99)
    lam: tuple = (0.15, 0.05)
    eps: tuple = (1e-3, 5e-5)
    shrink_ratio: float = 0.5
    severe_mult: float = 100.0
    l: int = 100
    c: int = 5
    t_forgiveness: int = 100
    metric_mask: int = 15
    R: int = 1
    ema_bf16: int = 0
    ref_over_batch: int = 0
    ref_over_tokens: int = 0

    def to_c(self) -> _Params:
        p = _Params()
        for name in ("beta", "k0", "alpha", "gamma_g", "gamma_s", "lam", "eps"):
            arr = getattr(p, name)
            arr[0], arr[1] = getattr(self, name)
        p.n_max[0], p.n_max[1] = self.n_max
        p.shrink_ratio, p.severe_mult = self.shrink_ratio, self.severe_mult
        p.l, p.c, p.t_forgiveness = self.l, self.c, self.t_forgiveness
        p.metric_mask = self.metric_mask
        p.B, p.T, p.d = self.B, self.T, self.d
        p.R = self.R
        p.ema_bf16 = self.ema_bf16
        p.ref_over_batch = self.ref_over_batch
        p.ref_over_tokens = self.ref_over_tokens
        return p


def default_params_from_c() -> dict:
    p = _Params()
    lib().so_default_params(C.byref(p))
    out = {}
    for name, _ in _Params._fields_:
        v = getattr(p, name)
        out[name] = tuple(v) if hasattr(v, "__len__") else v
    return out


def distance(x_bits, m) -> tuple[np.ndarray, np.ndarray, bool]:
    """Omega_i(x, m) of one unit: (gamma[3], stat[8], nonfinite)."""
    xb = _bits(x_bits).reshape(-1)
    mm = np.ascontiguousarray(m, dtype=np.float64).reshape(-1)
    assert xb.size == mm.size and xb.size > 0
    g = np.empty(3)
    s = np.empty(NSTAT)
    nf = lib().so_distance(_u16ptr(xb), _dptr(mm), xb.size, _dptr(g), _dptr(s))
    return g, s, bool(nf)


def token_sums(x_bits, m) -> np.ndarray:
    """Per token row: sum_c x, sum_c x^2, sum_c |x - m|, sign mismatches.  x_bits [..., d] against
    m of the same shape; returns [..., 4]."""
    xb = np.ascontiguousarray(_bits(x_bits))
    mm = np.ascontiguousarray(np.broadcast_to(np.asarray(m, dtype=np.float64), xb.shape))
    d = xb.shape[-1]
    rows = xb.reshape(-1, d)
    mrows = mm.reshape(-1, d)
    out = np.empty((rows.shape[0], 4))
    for i in range(rows.shape[0]):
        xr, mr = np.ascontiguousarray(rows[i]), np.ascontiguousarray(mrows[i])
        lib().so_token_sums(_u16ptr(xr), _dptr(mr), d, _dptr(out[i]))
    return out.reshape(xb.shape[:-1] + (4,))


def out_of_bounds(gamma: float, tau_lower: float, tau_upper: float) -> bool:
    return bool(lib().so_out_of_bounds(gamma, tau_lower, tau_upper))


def severe(flagged: bool, gamma: float, q2: float, tau_upper: float, severe_mult: float) -> bool:
    return bool(lib().so_severe(int(flagged), gamma, q2, tau_upper, severe_mult))


def sliced_wasserstein(x_bits, m, u_bits):
    """Sliced Wasserstein distance of one unit: x bits [tokens, d], m [tokens, d], directions
    u bits [L, d].  Returns (mean over directions, per-direction W1)."""
    xb = _bits(x_bits)
    ub = _bits(u_bits)
    tokens, d = xb.shape[-2] if xb.ndim == 2 else int(np.prod(xb.shape[:-1])), xb.shape[-1]
    xb = xb.reshape(tokens, d)
    mm = np.ascontiguousarray(m, dtype=np.float64).reshape(tokens, d)
    Ld = ub.shape[0]
    assert ub.shape == (Ld, d)
    w1 = np.empty(Ld)
    val = lib().so_sliced_wasserstein(_u16ptr(xb), _dptr(mm), tokens, d, _u16ptr(np.ascontiguousarray(ub)), Ld, _dptr(w1))
    return float(val), w1


def bf16_round(v: float) -> int:
    """double -> bf16 bit pattern, round to nearest even in one step."""
    return int(lib().so_bf16_round(float(v)))


def percentile(sorted_vals, p: float) -> float:
    a = np.ascontiguousarray(sorted_vals, dtype=np.float64)
    return float(lib().so_percentile(_dptr(a), a.size, p))


def adaptive_iqr(window, k_prev, alpha, n_max, gamma_g, gamma_s, lam, eps, shrink_ratio=0.5):
    """Alg. 5 on one window.  Returns (thr[6] or None, (grow_iters, shrink_iters))."""
    w = np.ascontiguousarray(window, dtype=np.float64)
    thr = np.zeros(NTHR)
    thr[3] = k_prev
    it = (C.c_int * 2)()
    ok = lib().so_adaptive_iqr(_dptr(w), w.size, alpha, n_max, gamma_g, gamma_s, lam, eps,
                               shrink_ratio, _dptr(thr), it)
    return (thr if ok else None), (it[0], it[1])


class Verifier:
    """State of one stage boundary: EMAs, histories, thresholds, counters."""

    def __init__(self, params: Params):
        self.params = params
        self._h = lib().so_create(C.byref(params.to_c()))
        if not self._h:
            raise ValueError("invalid oracle parameters")
        self.B, self.T, self.d = params.B, params.T, params.d
        self.rows = 1 + params.B
        self.R = params.R
        self.N = params.B * params.T * params.d
        self.nm = 3   # metrics in use: the columns of every score array returned below

    def close(self):
        if self._h:
            lib().so_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_directions(self, u_bits) -> None:
        """Sec. 3.1: switch the sliced Wasserstein metric on with the caller's directions
        (bf16 bit patterns, [L, d]); only before the first step."""
        ub = _bits(u_bits)
        assert ub.ndim == 2 and ub.shape[1] == self.d
        if lib().so_set_directions(self._h, _u16ptr(ub.reshape(-1)), ub.shape[0]) != 0:
            raise RuntimeError("so_set_directions refused (steps already taken?)")
        self.nm = NMETRIC

    def update_reference(self, x_bits, kind: int):
        xb = _bits(x_bits).reshape(-1)
        assert xb.size == self.N
        scores = np.empty((self.rows, NMETRIC))
        bad = lib().so_update_reference(self._h, _u16ptr(xb), kind, _dptr(scores))
        return scores[:, :self.nm].copy(), bool(bad)

    def verify(self, x_bits, kind: int):
        xb = _bits(x_bits).reshape(-1)
        assert xb.size == self.N
        scores = np.empty((self.rows, NMETRIC))
        flags = np.zeros(self.rows, dtype=np.uint32)
        commit = lib().so_verify(self._h, _u16ptr(xb), kind, _dptr(scores),
                                 flags.ctypes.data_as(C.POINTER(C.c_uint32)))
        return scores[:, :self.nm].copy(), flags, bool(commit)

    def replace_if_flagged(self, x_bits, kind: int, fill: int = 0):
        """Alg. 4 on a copy of x: (new bit patterns, replaced?)."""
        xb = _bits(x_bits).reshape(-1).copy()
        assert xb.size == self.N
        did = lib().so_replace_if_flagged(self._h, _u16ptr(xb), kind, fill)
        return xb.reshape(self.B, self.T, self.d), bool(did)

    def step_replicas(self, xs_bits, kind: int, warmup: bool = False, tainted_in: int = 0):
        """One iteration with all R workers' tensors: (scores [R,1+B,M], flags [R,1+B], number of
        submissions that entered the EMA).  tainted_in: bit r = worker r was tainted at another
        stage (its entry of xs_bits may be None)."""
        assert len(xs_bits) == self.R
        keep = [None if x is None else _bits(x).reshape(-1) for x in xs_bits]
        assert all(k is None or k.size == self.N for k in keep)
        assert all(k is not None or (tainted_in >> r) & 1 for r, k in enumerate(keep))
        ptrs = (C.POINTER(C.c_uint16) * self.R)(*[C.POINTER(C.c_uint16)() if k is None else _u16ptr(k)
                                                  for k in keep])
        scores = np.empty((self.R, self.rows, NMETRIC))
        flags = np.zeros((self.R, self.rows), dtype=np.uint32)
        n = lib().so_step_replicas(self._h, ptrs, kind, int(warmup), int(tainted_in), _dptr(scores),
                                   flags.ctypes.data_as(C.POINTER(C.c_uint32)))
        return scores[:, :, :self.nm].copy(), flags, int(n)

    def skip_tainted(self, kind: int) -> None:
        """The worker this verifier follows was tainted at another stage in this step."""
        lib().so_skip_tainted(self._h, kind)

    def count_violation(self, flagged: bool, severe: bool, r: int = 0) -> None:
        """One step of worker r's violation counter (Sec. 3.1) without a submission."""
        lib().so_count_violation(self._h, r, int(bool(flagged)), int(bool(severe)))

    def worker_counters(self, r: int) -> tuple[int, int, int]:
        out = (C.c_int * 3)()
        lib().so_worker_counters(self._h, r, out)
        return out[0], out[1], out[2]

    def reset_worker(self):
        lib().so_reset_worker(self._h)

    def ema(self, kind: int) -> np.ndarray:
        p = lib().so_ema(self._h, kind)
        shape = self.ref_shape()
        return np.ctypeslib.as_array(p, shape=(int(np.prod(shape)),)).copy().reshape(shape)

    def ref_shape(self) -> tuple:
        """[B,T,d], or with the reference reduced over the samples / the tokens: [T,d], [B,d], [d]."""
        over_b, over_t = self.params.ref_over_batch, self.params.ref_over_tokens
        return tuple(([] if over_b else [self.B]) + ([] if over_t else [self.T]) + [self.d])

    def set_ema(self, kind: int, m):
        mm = np.ascontiguousarray(m, dtype=np.float64).reshape(-1)
        assert mm.size == int(np.prod(self.ref_shape()))
        lib().so_set_ema(self._h, kind, _dptr(mm))

    def history(self, kind: int, level: int, metric: int) -> np.ndarray:
        cap = self.params.l * self.R * (self.B if level else 1)
        out = np.empty(cap)
        n = lib().so_history(self._h, kind, level, metric, _dptr(out), cap)
        return out[:n].copy()

    def thresholds(self, kind: int):
        """(thr[2][M][6], valid[2][M]) -- q1 q2 q3 k tau_lower tau_upper; M metrics in use."""
        thr = np.zeros((2, self.nm, NTHR))
        valid = np.zeros((2, self.nm), dtype=bool)
        for L in range(2):
            for i in range(self.nm):
                t = np.zeros(NTHR)
                valid[L, i] = bool(lib().so_thresholds(self._h, kind, L, i, _dptr(t)))
                thr[L, i] = t
        return thr, valid

    def last_stats(self, kind: int) -> np.ndarray:
        s = np.empty((self.rows, NSTAT))
        lib().so_last_stats(self._h, kind, _dptr(s))
        return s

    def counters(self) -> tuple[int, int, int]:
        out = (C.c_int * 3)()
        lib().so_counters(self._h, out)
        return out[0], out[1], out[2]

    def steps(self, kind: int) -> int:
        return int(lib().so_steps(self._h, kind))
