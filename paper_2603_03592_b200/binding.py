"""ctypes binding of ``libsentinel.so`` -- the same names as ``include/sentinel.h``.

Argument marshalling only: every step of the check runs in the library's CUDA kernels.  Torch
is used for device memory and streams; tensors are passed as raw pointers.  There is no CPU
fallback: if the library is missing or cannot be loaded, importing ``lib()`` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import _build

ACT, GRAD = 0, 1
NUM_METRICS, NUM_STATS, NUM_THRESHOLDS = 3, 8, 6
MAX_METRICS = 4        # with the sliced Wasserstein distance (Verifier.sentinel_set_directions)
MAX_B, MAX_WINDOW = 64, 4096

OK = 0
ERR_INVALID_ARG, ERR_SHAPE_MISMATCH, ERR_UNALIGNED, ERR_CUDA = -1, -2, -3, -4
ERR_STATE_SIZE, ERR_TIMEOUT, ERR_UNSUPPORTED = -5, -6, -7

FLAG_L1, FLAG_L2Z, FLAG_SFR, FLAG_SWD = 1 << 0, 1 << 1, 1 << 2, 1 << 3
FLAG_NONFINITE = 1 << 7
FLAG_COMMITTED, FLAG_SEVERE, FLAG_BANNED, FLAG_NO_THRESHOLDS = 1 << 16, 1 << 17, 1 << 18, 1 << 19
FLAG_NATURAL_SHIFT = 1 << 20
FLAG_TAINTED_ELSEWHERE = 1 << 21
MAX_WORKERS = 16

EXPORTS = (
    "sentinel_default_config", "sentinel_verifier_create", "sentinel_verify",
    "sentinel_set_directions", "sentinel_num_metrics", "sentinel_verify_replicas_tainted", "sentinel_skip_tainted",
    "sentinel_update_reference", "sentinel_verify_host", "sentinel_distance",
    "sentinel_verify_replicas", "sentinel_update_reference_replicas", "sentinel_get_worker_counters",
    "sentinel_verify_strided", "sentinel_update_reference_strided",
    "sentinel_distance_noalloc", "sentinel_replace_if_flagged", "sentinel_sliced_wasserstein",
    "sentinel_get_stats", "sentinel_get_thresholds", "sentinel_get_counters",
    "sentinel_set_token_stats_buffer", "sentinel_reset_worker", "sentinel_state_bytes",
    "sentinel_export_state", "sentinel_import_state", "sentinel_last_error", "sentinel_destroy",
    "sentinel_bounds_violations",
)


class sentinel_config(C.Structure):
    _fields_ = [
        ("beta", C.c_double * 2), ("k0", C.c_double * 2), ("alpha", C.c_double * 2),
        ("n_max", C.c_int * 2), ("gamma_grow", C.c_double * 2), ("gamma_shrink", C.c_double * 2),
        ("lambda_min", C.c_double * 2), ("iqr_eps", C.c_double * 2),
        ("shrink_ratio", C.c_double), ("severe_mult", C.c_double),
        ("window_steps", C.c_int), ("ban_violations", C.c_int), ("forgiveness_steps", C.c_int),
        ("metric_mask", C.c_uint), ("B", C.c_int), ("T", C.c_int), ("d", C.c_int),
        ("device", C.c_int), ("n_workers", C.c_int), ("ema_bf16", C.c_int), ("ref_over_batch", C.c_int), ("ref_over_tokens", C.c_int),
    ]


class SentinelError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("sentinel error %d: %s" % (code, message))
        self.code = code


_lib = None
_lib_file = None          # None: the normal build; else the path of the library to load


def lib_path() -> str:
    return _lib_file or _build.LIB


def use_library(path: str | None) -> None:
    """Switch the binding to another build of the library (the checked build, for one) or, with
    None, back to the normal one.  Handles made with one build must be closed before the switch."""
    global _lib, _lib_file
    _lib, _lib_file = None, path


def sentinel_bounds_violations(device: int = 0) -> tuple[int, int]:
    """(skipped accesses, site of the first) of the checked build; raises on the normal one."""
    count, site = C.c_ulonglong(0), C.c_int(0)
    _check(lib().sentinel_bounds_violations(device, C.byref(count), C.byref(site)))
    return int(count.value), int(site.value)


def lib():
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise ImportError(
                "libsentinel.so is missing at %s: build it with "
                "`python -m paper_2603_03592_b200._build` (needs nvcc)" % path)
        L = C.CDLL(path)
        vp, ip = C.c_void_p, C.c_int
        L.sentinel_default_config.argtypes = [C.POINTER(sentinel_config)]
        L.sentinel_verifier_create.argtypes = [C.POINTER(sentinel_config), C.POINTER(vp)]
        L.sentinel_verify.argtypes = [vp, vp, ip, ip, ip, ip, vp, vp, vp]
        L.sentinel_set_directions.argtypes = [vp, vp, ip, vp]
        L.sentinel_num_metrics.argtypes = [vp]
        L.sentinel_update_reference.argtypes = [vp, vp, ip, ip, ip, ip, vp, vp]
        L.sentinel_verify_host.argtypes = [vp, vp, ip, ip, ip, ip, vp, vp, vp]
        L.sentinel_distance.argtypes = [vp, vp, ip, ip, ip, ip, vp, vp, vp]
        L.sentinel_distance_noalloc.argtypes = [vp, vp, ip, ip, ip, ip, vp, vp, vp]
        L.sentinel_sliced_wasserstein.argtypes = [vp, vp, vp, ip, ip, ip, ip, ip, vp, vp]
        L.sentinel_replace_if_flagged.argtypes = [vp, vp, ip, ip, ip, ip, ip, vp, vp]
        L.sentinel_get_stats.argtypes = [vp, ip, vp, vp]
        L.sentinel_get_thresholds.argtypes = [vp, ip, vp, vp, vp]
        L.sentinel_get_counters.argtypes = [vp, vp, vp]
        L.sentinel_set_token_stats_buffer.argtypes = [vp, vp]
        L.sentinel_reset_worker.argtypes = [vp, ip, vp]
        L.sentinel_verify_strided.argtypes = [vp, vp, ip, ip, ip, ip, C.c_longlong, vp, vp, vp]
        L.sentinel_update_reference_strided.argtypes = [vp, vp, ip, ip, ip, ip, C.c_longlong, vp, vp]
        L.sentinel_verify_replicas.argtypes = [vp, vp, ip, ip, ip, ip, vp, vp, vp]
        L.sentinel_update_reference_replicas.argtypes = [vp, vp, ip, ip, ip, ip, vp, vp, vp]
        L.sentinel_get_worker_counters.argtypes = [vp, ip, vp, vp]
        L.sentinel_verify_replicas_tainted.argtypes = [vp, vp, ip, C.c_uint, ip, ip, ip, vp, vp, vp]
        L.sentinel_skip_tainted.argtypes = [vp, ip, vp]
        L.sentinel_state_bytes.argtypes = [vp]
        L.sentinel_state_bytes.restype = C.c_size_t
        L.sentinel_export_state.argtypes = [vp, vp, C.c_size_t, vp]
        L.sentinel_import_state.argtypes = [vp, vp, C.c_size_t, vp]
        L.sentinel_last_error.argtypes = [vp]
        L.sentinel_last_error.restype = C.c_char_p
        L.sentinel_destroy.argtypes = [vp]
        L.sentinel_bounds_violations.argtypes = [ip, vp, vp]
        for name in EXPORTS:
            if name not in ("sentinel_state_bytes", "sentinel_last_error"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _check(code: int, handle=None):
    if code != OK:
        msg = lib().sentinel_last_error(handle)
        raise SentinelError(code, msg.decode() if msg else "")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def sentinel_default_config(**overrides) -> sentinel_config:
    cfg = sentinel_config()
    _check(lib().sentinel_default_config(C.byref(cfg)))
    known = {name for name, _ in sentinel_config._fields_}
    for k, v in overrides.items():
        if k not in known:
            raise TypeError("sentinel_config has no field %r" % k)
        cur = getattr(cfg, k)
        if hasattr(cur, "__len__"):
            cur[0], cur[1] = v
        else:
            setattr(cfg, k, v)
    return cfg


def sentinel_distance(x: torch.Tensor, m: torch.Tensor, scores_out: torch.Tensor,
                      stats_out: torch.Tensor | None = None, stream=None) -> None:
    """Stateless Omega_i(x, m) for every unit; outputs are device tensors."""
    B, T, d = x.shape
    _check(lib().sentinel_distance(_ptr(x), _ptr(m), B, T, d, x.device.index or 0,
                                   _stream_ptr(stream), _ptr(scores_out), _ptr(stats_out)))


def sentinel_sliced_wasserstein(x: torch.Tensor, m: torch.Tensor, u_bf16: torch.Tensor,
                                sw_out: torch.Tensor, stream=None) -> None:
    """Sliced Wasserstein distance of every unit along the caller's directions u (bf16 [L, d])."""
    B, T, d = x.shape
    _check(lib().sentinel_sliced_wasserstein(_ptr(x), _ptr(m), _ptr(u_bf16), u_bf16.shape[0], B, T, d,
                                             x.device.index or 0, _stream_ptr(stream), _ptr(sw_out)))


NOALLOC_SCRATCH_BYTES = 65536


def sentinel_distance_noalloc(x: torch.Tensor, m: torch.Tensor, scores_out: torch.Tensor,
                              stats_out: torch.Tensor | None = None, stream=None) -> None:
    """``sentinel_distance`` for callers that may not allocate device memory during the call
    (frozen pools, fixed budgets, latency-critical loops): its scratch is a fixed array inside
    the library.  Calls on one device share that array, so keep them ordered on one stream;
    make the first call on a device outside any stream capture."""
    B, T, d = x.shape
    _check(lib().sentinel_distance_noalloc(_ptr(x), _ptr(m), B, T, d, x.device.index or 0,
                                           _stream_ptr(stream), _ptr(scores_out), _ptr(stats_out)))


class Verifier:
    """One stage boundary (a ``sentinel_verifier`` handle).  Methods mirror the C entry points."""

    def __init__(self, B: int, T: int, d: int, device: int = 0, **overrides):
        self.cfg = sentinel_default_config(B=B, T=T, d=d, device=device, **overrides)
        self.B, self.T, self.d = B, T, d
        self.R = self.cfg.n_workers
        self.rows = 1 + B
        self.device = torch.device("cuda", device)
        h = C.c_void_p()
        _check(lib().sentinel_verifier_create(C.byref(self.cfg), C.byref(h)))
        self._h = h
        self.M = NUM_METRICS          # columns of every score array

    def sentinel_set_directions(self, u_bf16: torch.Tensor, stream=None) -> None:
        """Sec. 3.1: adds the sliced Wasserstein distance along the caller's directions
        (bf16 [L, d], L in 4/8/16) as a fourth metric; only before the first step."""
        assert u_bf16.dtype == torch.bfloat16 and u_bf16.is_contiguous() and u_bf16.shape[1] == self.d
        _check(lib().sentinel_set_directions(self._h, _ptr(u_bf16), u_bf16.shape[0], _stream_ptr(stream)), self._h)
        self.M = self.sentinel_num_metrics()

    def sentinel_num_metrics(self) -> int:
        return int(lib().sentinel_num_metrics(self._h))

    # -- hot path ---------------------------------------------------------------------------
    def sentinel_verify(self, x: torch.Tensor, kind: int, scores_out: torch.Tensor,
                        flags_out: torch.Tensor, stream=None) -> None:
        B, T, d = x.shape
        _check(lib().sentinel_verify(self._h, _ptr(x), kind, B, T, d, _stream_ptr(stream),
                                     _ptr(scores_out), _ptr(flags_out)), self._h)

    def sentinel_update_reference(self, x: torch.Tensor, kind: int,
                                  scores_out: torch.Tensor | None = None, stream=None) -> None:
        B, T, d = x.shape
        _check(lib().sentinel_update_reference(self._h, _ptr(x), kind, B, T, d,
                                               _stream_ptr(stream), _ptr(scores_out)), self._h)

    def sentinel_verify_host(self, x_host: torch.Tensor, kind: int, scores_host: torch.Tensor,
                             flags_host: torch.Tensor, stream=None) -> None:
        B, T, d = x_host.shape
        _check(lib().sentinel_verify_host(self._h, _ptr(x_host), kind, B, T, d,
                                          _stream_ptr(stream), _ptr(scores_host),
                                          _ptr(flags_host)), self._h)

    def sentinel_verify_strided(self, x_wide: torch.Tensor, kind: int, scores_out: torch.Tensor,
                                flags_out: torch.Tensor, stream=None) -> None:
        """x_wide: [B, T, row_stride] bf16 of which the first d channels of every row are verified."""
        _check(lib().sentinel_verify_strided(self._h, _ptr(x_wide), kind, self.B, self.T, self.d,
                                             x_wide.shape[2], _stream_ptr(stream), _ptr(scores_out),
                                             _ptr(flags_out)), self._h)

    def sentinel_update_reference_strided(self, x_wide: torch.Tensor, kind: int,
                                          scores_out: torch.Tensor | None = None, stream=None) -> None:
        _check(lib().sentinel_update_reference_strided(self._h, _ptr(x_wide), kind, self.B, self.T, self.d,
                                                       x_wide.shape[2], _stream_ptr(stream),
                                                       _ptr(scores_out)), self._h)

    def _worker_pointers(self, xs):
        assert len(xs) == self.R, "one tensor per worker"
        return (C.c_void_p * self.R)(*[None if x is None else x.data_ptr() for x in xs])

    def sentinel_verify_replicas(self, xs, kind: int, scores_out: torch.Tensor,
                                 flags_out: torch.Tensor, stream=None) -> None:
        """One iteration with all workers' tensors (worker loop of Alg. 2/3, mean over the clean)."""
        B, T, d = xs[0].shape
        _check(lib().sentinel_verify_replicas(self._h, self._worker_pointers(xs), kind, B, T, d,
                                              _stream_ptr(stream), _ptr(scores_out), _ptr(flags_out)), self._h)

    def sentinel_update_reference_replicas(self, xs, kind: int, scores_out: torch.Tensor,
                                           flags_out: torch.Tensor | None = None, stream=None) -> None:
        B, T, d = xs[0].shape
        _check(lib().sentinel_update_reference_replicas(self._h, self._worker_pointers(xs), kind, B, T, d,
                                                        _stream_ptr(stream), _ptr(scores_out),
                                                        _ptr(flags_out)), self._h)

    def sentinel_verify_replicas_tainted(self, xs, kind: int, tainted_in: int, scores_out: torch.Tensor,
                                         flags_out: torch.Tensor, stream=None) -> None:
        """As sentinel_verify_replicas; bit r of tainted_in: worker r was tainted at another stage and
        is not collected (xs[r] may be None)."""
        _check(lib().sentinel_verify_replicas_tainted(self._h, self._worker_pointers(xs), kind, tainted_in,
                                                      self.B, self.T, self.d, _stream_ptr(stream),
                                                      _ptr(scores_out), _ptr(flags_out)), self._h)

    def sentinel_skip_tainted(self, kind: int, stream=None) -> None:
        _check(lib().sentinel_skip_tainted(self._h, kind, _stream_ptr(stream)), self._h)

    def step_replicas(self, xs, kind: int, warmup: bool = False, stream=None, tainted_in: int = 0):
        scores = torch.empty(self.R, self.rows, self.M, dtype=torch.float32, device=self.device)
        flags = torch.zeros(self.R, self.rows, dtype=torch.int32, device=self.device)
        if warmup:
            self.sentinel_update_reference_replicas(xs, kind, scores, flags, stream)
        elif tainted_in:
            self.sentinel_verify_replicas_tainted(xs, kind, tainted_in, scores, flags, stream)
        else:
            self.sentinel_verify_replicas(xs, kind, scores, flags, stream)
        return scores, flags

    def sentinel_get_worker_counters(self, worker: int, stream=None) -> tuple:
        out = (C.c_longlong * 3)()
        _check(lib().sentinel_get_worker_counters(self._h, worker, out, _stream_ptr(stream)), self._h)
        return out[0], out[1], out[2]

    def sentinel_replace_if_flagged(self, x_inout: torch.Tensor, kind: int, fill: int = 0,
                                    replaced_out: torch.Tensor | None = None, stream=None) -> None:
        """Alg. 4: overwrite x with the reference (fill=0) or zeros (fill=1) iff the last
        verified step of this kind was flagged; decided on the device."""
        B, T, d = x_inout.shape
        _check(lib().sentinel_replace_if_flagged(self._h, _ptr(x_inout), kind, B, T, d, fill,
                                                 _stream_ptr(stream), _ptr(replaced_out)), self._h)

    # convenience wrappers that allocate the outputs (tests, examples)
    def verify(self, x: torch.Tensor, kind: int, stream=None):
        scores = torch.empty(self.rows, self.M, dtype=torch.float32, device=x.device)
        flags = torch.empty(self.rows, dtype=torch.int32, device=x.device)
        self.sentinel_verify(x, kind, scores, flags, stream)
        return scores, flags

    def update_reference(self, x: torch.Tensor, kind: int, stream=None):
        scores = torch.empty(self.rows, self.M, dtype=torch.float32, device=x.device)
        self.sentinel_update_reference(x, kind, scores, stream)
        return scores

    # -- queries ----------------------------------------------------------------------------
    def sentinel_get_stats(self, kind: int, stream=None) -> torch.Tensor:
        out = torch.empty(self.rows, NUM_STATS, dtype=torch.float32, device=self.device)
        _check(lib().sentinel_get_stats(self._h, kind, _ptr(out), _stream_ptr(stream)), self._h)
        return out

    def sentinel_get_thresholds(self, kind: int, stream=None):
        thr = (C.c_double * (2 * self.M * NUM_THRESHOLDS))()
        valid = (C.c_int * (2 * self.M))()
        _check(lib().sentinel_get_thresholds(self._h, kind, thr, valid, _stream_ptr(stream)), self._h)
        t = torch.tensor(list(thr), dtype=torch.float64).reshape(2, self.M, NUM_THRESHOLDS)
        v = torch.tensor(list(valid), dtype=torch.bool).reshape(2, self.M)
        return t.numpy(), v.numpy()

    def sentinel_get_counters(self, stream=None) -> dict:
        out = (C.c_longlong * 6)()
        _check(lib().sentinel_get_counters(self._h, out, _stream_ptr(stream)), self._h)
        return {"violations": out[0], "clean_streak": out[1], "banned": out[2],
                "steps_act": out[3], "steps_grad": out[4], "error": out[5]}

    def sentinel_set_token_stats_buffer(self, buf: torch.Tensor | None) -> None:
        self._token_buf = buf          # keep the tensor alive while registered
        _check(lib().sentinel_set_token_stats_buffer(self._h, _ptr(buf)), self._h)

    def sentinel_reset_worker(self, worker: int = 0, stream=None) -> None:
        _check(lib().sentinel_reset_worker(self._h, worker, _stream_ptr(stream)), self._h)

    # -- checkpointing ------------------------------------------------------------------------
    def sentinel_state_bytes(self) -> int:
        return int(lib().sentinel_state_bytes(self._h))

    def sentinel_export_state(self, stream=None) -> bytearray:
        n = self.sentinel_state_bytes()
        buf = bytearray(n)
        cbuf = (C.c_char * n).from_buffer(buf)
        _check(lib().sentinel_export_state(self._h, cbuf, n, _stream_ptr(stream)), self._h)
        return buf

    def sentinel_import_state(self, blob, stream=None) -> None:
        data = bytes(blob)
        _check(lib().sentinel_import_state(self._h, data, len(data), _stream_ptr(stream)), self._h)

    # -- lifetime -----------------------------------------------------------------------------
    def sentinel_destroy(self) -> None:
        if getattr(self, "_h", None):
            h, self._h = self._h, None
            _check(lib().sentinel_destroy(h))

    close = sentinel_destroy

    def __del__(self):
        try:
            self.sentinel_destroy()
        except Exception:
            pass
