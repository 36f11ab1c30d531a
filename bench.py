#!/usr/bin/env python
"""Benchmark of the Sentinel verifier check on B200.

One *step* is one microbatch crossing a stage boundary: ``sentinel_verify`` on the activation
tensor h (forward) and on the activation-gradient tensor g (backward), i.e. two launches of
the streaming kernel, each of which reads x (bf16) and the reference m (fp32) once and writes
the EMA candidate once: 10 bytes per element.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

Prints ONE JSON line.  ``value`` is verified GB/s (10 B/element moved, all ranks) with inputs
resident in HBM; ``e2e`` is the same metric through ``sentinel_verify_host`` with pinned host
buffers (H2D of x and D2H of scores/flags inside the timed region).  With N > 1 (torchrun)
every rank runs an independent replica of the workload on its own GPU: the check has no
cross-GPU data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_03592_b200 import replicas, synth  # noqa: E402

ACT, GRAD = 0, 1
BYTES_PER_ELEMENT = 10          # 2 (x, bf16 read) + 4 (m read) + 4 (EMA candidate write)
MAX_DISTINCT = 24               # distinct input tensors per kind kept resident
FOUR_METRIC_BYTES = 12          # a verified tensor with the sliced Wasserstein distance: x twice, the reference read and written
# dram__bytes_read.sum + dram__bytes_write.sum per element of the current stream_kernel, from the
# ncu capture summarised in profiles/all_kernels_cfg3_ncu.md (B=8 x 4096 x 4096; traffic
# grows in proportion to the element count, so a launch of N elements moves this times N).
# Set to None whenever the kernel changes until the capture is retaken.
NCU_DRAM_BYTES_PER_ELEMENT = 9.672


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the benchmark runs; a summary
    is taken over the samples that fall inside a wall-clock window (the timed region)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    BAD = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()          # the exact process started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    @staticmethod
    def _when(stamp: str, fallback: float) -> float:
        try:                               # "2026/01/31 12:00:00.123", the sampler's own clock
            head, _, ms = stamp.partition(".")
            return time.mktime(time.strptime(head, "%Y/%m/%d %H:%M:%S")) + (float("0." + ms) if ms else 0.0)
        except ValueError:
            return fallback

    def summary(self, t0: float | None = None, t1: float | None = None) -> dict:
        """Median SM clock and the throttle reasons seen between wall-clock times t0 and t1 (all
        samples if no window is given or none fell inside it)."""
        rows = []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for seen, line in list(self.lines):
            tok = [t.strip() for t in line.split(",")]
            if len(tok) < 7:
                continue
            try:
                rows.append((self._when(tok[0], seen), float(tok[1]), float(tok[2]),
                             [n for n, v in zip(names, tok[3:7]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in rows if t0 is not None and t0 - 0.02 <= r[0] <= t1 + 0.02]
        used, window = (inside, "timed region") if inside else (rows, "whole run")
        sm = sorted(r[1] for r in used)
        reasons = sorted({n for r in used for n in r[3]})
        return {"sm_mhz": sm[len(sm) // 2] if sm else None,
                "sm_max_mhz": max((r[2] for r in used), default=None),
                "samples": len(sm), "window": window, "reasons": reasons,
                "rejected": any(n in self.BAD for n in reasons)}


def build_stream(w, boundary, device, count, distinct):
    """`count` microbatches per kind after the warm-up, following the workload's recipe."""
    xs = {ACT: [], GRAD: [], "corrupted": {ACT: [], GRAD: []}}
    n = min(count, distinct)
    for kind in (ACT, GRAD):
        for i in range(n):
            x, name = synth.microbatch(w, boundary, kind, w.warmup + i, device)
            xs[kind].append(x)
            xs["corrupted"][kind].append(name is not None)
    return xs


MIN_TIMED_MS = 200.0            # device time the timed region covers at least, whatever --steps is


EXTRAS_MIN_MS = 60.0            # device time each figure after the timed region covers at least (--extras-ms)


def timed_calls(fn, stream, min_ms=None, min_calls=6, max_calls=400):
    """Median and best duration (ms) of fn(i), one CUDA-event pair per call on `stream`, over at
    least min_calls calls and min_ms of device time."""
    durations = []
    i = 0
    min_ms = EXTRAS_MIN_MS if min_ms is None else min_ms
    while True:
        batch = min_calls if not durations else max(2, min(64, int(min_calls * 1.5)))
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(batch + 1)]
        marks[0].record(stream)
        for k in range(batch):
            fn(i)
            i += 1
            marks[k + 1].record(stream)
        torch.cuda.synchronize()
        durations += [marks[k].elapsed_time(marks[k + 1]) for k in range(batch)]
        if (sum(durations) >= min_ms and len(durations) >= min_calls) or len(durations) >= max_calls:
            break
    durations.sort()
    return durations[len(durations) // 2], durations[0], len(durations)


class Measured:
    """What measure_workload leaves behind for the figures taken after the timed region."""


def measure_workload(binding, w, args, rank, world, local_rank, sampler, steps, warmup, min_ms, distinct):
    """The timed region of one workload: `steps` verified microbatches per boundary (h and g each),
    repeated until at least min_ms of device time have passed.  Returns (figures, Measured)."""
    device = torch.device("cuda", local_rank)
    N = w.B * w.T * w.d
    nb = w.boundaries                               # independent stage boundaries, one stream each
    main = torch.cuda.current_stream()
    streams = [main] if nb == 1 else [torch.cuda.Stream(device=device) for _ in range(nb)]
    vs = [binding.Verifier(w.B, w.T, w.d, device=local_rank) for _ in range(nb)]

    # reference warm-up on clean traffic (untimed set-up, as the method prescribes)
    for b, v in enumerate(vs):
        for t in range(w.warmup):
            for kind in (ACT, GRAD):
                v.sentinel_update_reference(synth.clean(w, b, kind, t, device), kind)
    torch.cuda.synchronize()

    distinct = distinct if nb == 1 else min(distinct, 12)   # 8 boundaries: bound the footprint
    xs = [build_stream(w, b, device, warmup + steps, distinct) for b in range(nb)]
    nd = len(xs[0][ACT])
    scores = torch.empty(nb, 2, 1 + w.B, 3, dtype=torch.float32, device=device)
    flags = torch.empty(nb, 2, 1 + w.B, dtype=torch.int32, device=device)
    flag_log = torch.zeros(nd, nb, 2, 1 + w.B, dtype=torch.int32, device=device)   # flags of the last pass over each input
    torch.cuda.synchronize()

    def step(i):
        for b, (v, s) in enumerate(zip(vs, streams)):
            v.sentinel_verify(xs[b][ACT][i % nd], ACT, scores[b, 0], flag_log[i % nd, b, 0], s)
            v.sentinel_verify(xs[b][GRAD][i % nd], GRAD, scores[b, 1], flag_log[i % nd, b, 1], s)

    def fork():                                      # side streams start after `main` gets here
        if nb > 1:
            ev = torch.cuda.Event()
            ev.record(main)
            for s in streams:
                s.wait_event(ev)

    def join():                                      # `main` continues after every side stream
        if nb > 1:
            for s in streams:
                ev = torch.cuda.Event()
                ev.record(s)
                main.wait_event(ev)

    fork()
    for i in range(warmup):
        step(i)
    join()
    torch.cuda.synchronize()

    # how often the list of `steps` steps is gone through: an estimate from a short untimed pass
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main)
    fork()
    for i in range(min(steps, 4)):
        step(warmup + i)
    join()
    e1.record(main)
    torch.cuda.synchronize()
    est_ms = e0.elapsed_time(e1) / min(steps, 4)
    repeats = max(1, int(-(-min_ms // max(est_ms * steps, 1e-3))))
    repeats = int(replicas.max_over_ranks(repeats))      # every rank times the same number of steps
    timed = steps * repeats

    replicas.barrier()
    torch.cuda.synchronize()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(timed + 1)]
    t_wall0 = time.time()
    marks[0].record(main)
    fork()
    for i in range(timed):
        step(warmup + (i % steps))
        if nb == 1:
            marks[i + 1].record(main)
    join()
    if nb > 1:
        marks[-1].record(main)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    replicas.barrier()
    torch.cuda.synchronize()
    local_ms = marks[0].elapsed_time(marks[-1])
    if nb == 1:
        step_ms = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(timed))
    else:
        step_ms = [local_ms / timed]
    elapsed_ms = replicas.max_over_ranks(local_ms)
    launches = 2 * timed * nb
    time.sleep(0.05)                                 # let the sampler's last lines arrive
    clocks = sampler.summary(t_wall0, t_wall1)

    # what the detector said on the last pass over the inputs (reported, not a target: some of the
    # recipe's corruptions are statistically invisible to these metrics, and a flagged tensor that
    # comes round again is flagged again)
    raised = ((flag_log & 0xFFFF) != 0).any(dim=-1).cpu()                       # [nd, nb, 2]
    n_corrupted = n_flagged = n_both = 0
    seen = min(nd, steps)
    for i in range(seen):
        for b in range(nb):
            for kind in (ACT, GRAD):
                c = xs[b]["corrupted"][kind][(warmup + i) % nd]
                f = bool(raised[(warmup + i) % nd, b, kind])
                n_corrupted += c
                n_flagged += f
                n_both += c and f
    detection = {"tensors": seen * nb * 2, "corrupted": n_corrupted, "flagged": n_flagged,
                 "corrupted_and_flagged": n_both, "distinct_tensors_per_kind": nd,
                 "note": "verdicts of the last pass over the distinct tensors; the stream cycles through them, and "
                         "one that comes round again soon correlates with the reference that absorbed it and is "
                         "flagged as a replay"}

    bytes_step = 2 * N * BYTES_PER_ELEMENT * nb             # two tensors per boundary per step
    cycle_bytes = nb * nd * 2 * N * BYTES_PER_ELEMENT       # one pass over the cycled inputs, against the 126 MB L2
    if cycle_bytes > 4 * 126e6:
        l2_note = "inputs larger than L2: %d MiB read+written per launch, %d distinct tensors per kind" % (
            N * BYTES_PER_ELEMENT >> 20, nd)
    else:
        l2_note = ("inputs and state of a whole cycle (%d MiB) stay near the 126 MB L2: a launch-latency figure, "
                   "not a bandwidth figure" % (cycle_bytes >> 20))
    gbs = world * timed * bytes_step / (elapsed_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak_gbs()
    kernel_ms = local_ms / launches                         # the timed region holds these launches only
    achieved = N * BYTES_PER_ELEMENT / (kernel_ms * 1e-3) / 1e9
    fig = {
        "value": round(gbs, 1), "ms_per_step": round(elapsed_ms / timed, 4),
        "ms_per_step_median": round(step_ms[len(step_ms) // 2], 4), "ms_per_step_best": round(step_ms[0], 4),
        "timed_steps": timed, "repeats": repeats, "timed_ms": round(elapsed_ms, 2),
        "microbatches_per_s": round(world * timed * nb / (elapsed_ms * 1e-3), 1),
        "tensor_gbs": round(world * timed * nb * 2 * N * 2 / (elapsed_ms * 1e-3) / 1e9, 1),
        "frac_of_8000_nominal": round(gbs / world / 8000.0, 4),
        "gpu_launches": launches, "detection": detection, "clocks": clocks, "l2": l2_note,
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "peak_source": "%s copy bandwidth" % peak_kind,
                     "kernel": "stream_kernel", "avg_launch_ms": round(kernel_ms, 4),
                     "note": ("launches of different boundaries overlap: time per launch is the "
                              "timed region divided by the launches" if nb > 1 else
                              "timed region / launches; the region holds these launches only"),
                     "traffic": (args.traffic if args.traffic is not None else
                                 (round(NCU_DRAM_BYTES_PER_ELEMENT * N) if NCU_DRAM_BYTES_PER_ELEMENT else None)),
                     "traffic_source": "ncu on B=8x4096x4096, scaled by element count"},
    }
    m = Measured()
    m.vs, m.xs, m.nd, m.N, m.nb, m.scores, m.flags, m.main, m.device = vs, xs, nd, N, nb, scores, flags, main, device
    m.bytes_step = bytes_step
    return fig, m


def workload_text(w):
    nb = w.boundaries
    return "%s: B=%d x T=%d x d=%d bf16, activations %s, gradients N(0,%g), %g%% corrupted%s" % (
        w.name, w.B, w.T, w.d, w.act, w.grad_std, 100 * w.corrupt_rate,
        ", %d boundaries on %d CUDA streams" % (nb, nb) if nb > 1 else "")


def run_ours(args, rank, world, local_rank):
    from paper_2603_03592_b200 import binding
    binding.lib()                                   # no library, no benchmark: there is no fallback
    torch.cuda.set_device(local_rank)
    w = synth.WORKLOADS[args.workload]
    with ClockSampler(local_rank) as sampler:
        fig, m = measure_workload(binding, w, args, rank, world, local_rank, sampler, args.steps, args.warmup,
                                  args.min_ms, args.distinct)
        if fig["clocks"]["rejected"]:               # a thermal or hardware slowdown: measured again, once
            for v in m.vs:
                v.sentinel_destroy()
            del m
            torch.cuda.empty_cache()
            first = fig["clocks"]
            fig, m = measure_workload(binding, w, args, rank, world, local_rank, sampler, args.steps, args.warmup,
                                      args.min_ms, args.distinct)
            fig["clocks"]["first_attempt"] = first
        out = run_after_timed_region(binding, w, args, rank, world, local_rank, fig, m, sampler)
    return out


def run_after_timed_region(binding, w, args, rank, world, local_rank, fig, m, sampler):
    vs, xs, nd, N, nb, scores, flags, main, device = m.vs, m.xs, m.nd, m.N, m.nb, m.scores, m.flags, m.main, m.device
    violations = sum(int(v.sentinel_get_counters()["violations"]) for v in vs)

    # The figures below are taken outside the timed region, each over at least 60 ms of device
    # time: the median of per-call CUDA-event durations on the launching stream.
    extras = nb == 1 and args.extras and world == 1     # the extra figures are single-GPU figures
    extra_keys = {}
    pick1 = lambda i: xs[0][ACT][i % nd]

    if extras:   # gradient replacement (Alg. 4) after a flagged step
        v0 = vs[0]
        loud = (xs[0][GRAD][0].float() * 64.0).to(torch.bfloat16)
        v0.sentinel_verify(loud, GRAD, scores[0, 1], flags[0, 1], main)       # flagged: no commit
        outs = [torch.empty_like(loud) for _ in range(4)]
        for o in outs:
            v0.sentinel_replace_if_flagged(o, GRAD, 0, None, main)
        rms, rbest, rn = timed_calls(lambda i: v0.sentinel_replace_if_flagged(outs[i % 4], GRAD, 0, None, main), main)
        extra_keys["gradient_replacement"] = {
            "kernel": "replace_kernel", "bytes_per_element": 6, "ms_per_launch": round(rms, 4),
            "ms_best": round(rbest, 4), "calls": rn, "achieved_gbs": round(6 * N / (rms * 1e-3) / 1e9, 1),
            "flagged": bool(int(flags[0, 1, 0]) & 0xFFFF)}
        del outs, loud

    if extras and 8 * w.d * 2 <= 200 * 1024 and w.T <= 16384:   # sliced Wasserstein distance along 8 directions
        g = torch.Generator(device=device).manual_seed(11)
        u = torch.randn(8, w.d, generator=g, device=device)
        u = (u / u.norm(dim=1, keepdim=True)).to(torch.bfloat16).contiguous()
        ref = xs[0][ACT][1 % nd].float().mul_(0.1).contiguous()
        sw = torch.empty(1 + w.B, dtype=torch.float32, device=device)
        for _ in range(2):
            binding.sentinel_sliced_wasserstein(xs[0][ACT][0], ref, u, sw, main)
        sms, sbest, sn = timed_calls(lambda i: binding.sentinel_sliced_wasserstein(pick1(i), ref, u, sw, main), main)
        swd = {"directions": 8, "bytes_per_element": 6, "ms_per_call": round(sms, 4), "ms_best": round(sbest, 4),
               "calls": sn, "achieved_gbs": round(6 * N / (sms * 1e-3) / 1e9, 1),
               "kernels": "swd_project_ref_mma_kernel + swd_sort_samples_kernel + swd_merge_kernel (all rounds but the last) + swd_w1_kernel", "value_row0": float(sw[0])}
        del ref
        # the same distance as the verifier's fourth metric: one verified tensor per call
        v4 = binding.Verifier(w.B, w.T, w.d, device=local_rank)
        v4.sentinel_set_directions(u, main)
        s4 = torch.empty(1 + w.B, 4, dtype=torch.float32, device=device)
        f4 = torch.zeros(1 + w.B, dtype=torch.int32, device=device)
        for i in range(4):
            v4.sentinel_update_reference(pick1(i), ACT, s4, main)
        v4.sentinel_verify(pick1(4), ACT, s4, f4, main)
        vms, vbest, vn = timed_calls(lambda i: v4.sentinel_verify(pick1(5 + i), ACT, s4, f4, main), main)
        swd["verify_with_four_metrics"] = {"ms_per_tensor": round(vms, 4), "ms_best": round(vbest, 4), "calls": vn,
                                           "bytes_per_element": FOUR_METRIC_BYTES,
                                           "achieved_gbs": round(FOUR_METRIC_BYTES * N / (vms * 1e-3) / 1e9, 1)}
        v4.close()
        # ... and with the reference stored as bf16: x twice, the reference twice (projected afresh) and written once
        v4b = binding.Verifier(w.B, w.T, w.d, device=local_rank, ema_bf16=1)
        v4b.sentinel_set_directions(u, main)
        for i in range(4):
            v4b.sentinel_update_reference(pick1(i), ACT, s4, main)
        v4b.sentinel_verify(pick1(4), ACT, s4, f4, main)
        wms, wbest, wn = timed_calls(lambda i: v4b.sentinel_verify(pick1(5 + i), ACT, s4, f4, main), main)
        swd["verify_with_four_metrics_bf16_reference"] = {"ms_per_tensor": round(wms, 4), "ms_best": round(wbest, 4),
                                                          "calls": wn, "bytes_per_element": 10,
                                                          "achieved_gbs": round(10 * N / (wms * 1e-3) / 1e9, 1)}
        v4b.close()
        extra_keys["sliced_wasserstein"] = swd

    if extras:   # one iteration with R workers of the stage (2R B/element of tensors + the reference read and written)
        R = 4 if 100 * 4 * (w.B + 1) <= 4096 else 2
        vr = binding.Verifier(w.B, w.T, w.d, device=local_rank, n_workers=R)
        rs = torch.empty(R, 1 + w.B, 3, dtype=torch.float32, device=device)
        rf = torch.zeros(R, 1 + w.B, dtype=torch.int32, device=device)
        pick = lambda i: [xs[0][ACT][(i * R + r) % nd] for r in range(R)]
        for i in range(4):
            vr.sentinel_update_reference_replicas(pick(i), ACT, rs, rf, main)
        vr.sentinel_verify_replicas(pick(4), ACT, rs, rf, main)
        qms, qbest, qn = timed_calls(lambda i: vr.sentinel_verify_replicas(pick(5 + i), ACT, rs, rf, main), main)
        per_el = 2 * R + 8
        extra_keys["multi_worker_iteration"] = {
            "workers": R, "bytes_per_element": per_el, "ms_per_iteration": round(qms, 4), "ms_best": round(qbest, 4),
            "calls": qn, "achieved_gbs": round(per_el * N / (qms * 1e-3) / 1e9, 1),
            "submissions_per_s": round(R / (qms * 1e-3), 1),
            "flagged_workers_last_iteration": int(((rf[:, 0] & 0xFFFF) != 0).sum()),
            "error_word": int(vr.sentinel_get_counters()["error"]),
            "kernels": "replica_kernel (all workers, speculative mean) + ema_mean_kernel (report bits)"}
        vr.sentinel_destroy()
        # the same iteration with the reference stored as bf16 (2R + 4 B/element)
        vb = binding.Verifier(w.B, w.T, w.d, device=local_rank, n_workers=R, ema_bf16=1)
        for i in range(4):
            vb.sentinel_update_reference_replicas(pick(i), ACT, rs, rf, main)
        vb.sentinel_verify_replicas(pick(4), ACT, rs, rf, main)
        bms, bbest, bn = timed_calls(lambda i: vb.sentinel_verify_replicas(pick(5 + i), ACT, rs, rf, main), main)
        extra_keys["multi_worker_iteration"]["bf16_reference"] = {
            "bytes_per_element": 2 * R + 4, "ms_per_iteration": round(bms, 4), "ms_best": round(bbest, 4), "calls": bn,
            "achieved_gbs": round((2 * R + 4) * N / (bms * 1e-3) / 1e9, 1)}
        vb.sentinel_destroy()

    def single_variant(name, per_el, kernel, **kw):   # a verifier option, one verified tensor per call
        v = binding.Verifier(w.B, w.T, w.d, device=local_rank, **kw)
        s_, f_ = (torch.empty(1 + w.B, 3, dtype=torch.float32, device=device),
                  torch.zeros(1 + w.B, dtype=torch.int32, device=device))
        for i in range(6):
            v.sentinel_update_reference(pick1(i), ACT, s_, main)
        v.sentinel_verify(pick1(6), ACT, s_, f_, main)
        ms, best, n = timed_calls(lambda i: v.sentinel_verify(pick1(7 + i), ACT, s_, f_, main), main)
        err = int(v.sentinel_get_counters()["error"])
        v.sentinel_destroy()
        return {"bytes_per_element": per_el, "ms_per_launch": round(ms, 4), "ms_best": round(best, 4), "calls": n,
                "achieved_gbs": round(per_el * N / (ms * 1e-3) / 1e9, 1), "tensors_per_s": round(1e3 / ms, 1),
                "error_word": err, "kernel": kernel}

    if extras:
        extra_keys["bf16_reference"] = single_variant("bf16", 6, "stream_kernel_t<false, true>", ema_bf16=1)
        if w.B <= 16:
            extra_keys["shared_reference"] = single_variant("shared", 2 + 8.0 / w.B, "shared_ref_kernel", ref_over_batch=1)
        ch = single_variant("channel", 2, "channel_ref_kernel + channel_mean_kernel", ref_over_batch=1, ref_over_tokens=1)
        ch["ms_per_step"] = ch.pop("ms_per_launch")
        ch["ms_per_step_vector_per_sample"] = single_variant("channel_b", 2, "", ref_over_tokens=1)["ms_per_launch"]
        extra_keys["channel_reference"] = ch

    if extras:   # the strided (compressed-signal) layout, rows d+1 apart
        wide = [torch.nn.functional.pad(xs[0][ACT][i % nd], (0, 1)).contiguous() for i in range(3)]
        for i in range(2):
            vs[0].sentinel_update_reference_strided(wide[i], ACT, scores[0, 0], main)
        cms, cbest, cn = timed_calls(lambda i: vs[0].sentinel_update_reference_strided(wide[i % 3], ACT, scores[0, 0], main), main)
        extra_keys["compressed_layout"] = {
            "row_stride": w.d + 1, "bytes_per_element": 10, "ms_per_launch": round(cms, 4), "ms_best": round(cbest, 4),
            "calls": cn, "achieved_gbs": round(10 * N / (cms * 1e-3) / 1e9, 1),
            "kernel": "stream_kernel_t<false, false, true> (funnel-shifted rows)"}
        del wide

    # end to end through the host-buffer entry point
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    hx = [{k: [xs[b][k][i % nd].cpu().pin_memory() for i in range(min(e2e_steps, 2 if nb > 1 else 4))]
           for k in (ACT, GRAD)} for b in range(nb)]
    hs = torch.empty(2, 1 + w.B, 3, dtype=torch.float32).pin_memory()
    hf = torch.empty(2, 1 + w.B, dtype=torch.int32).pin_memory()
    for b, v in enumerate(vs):                       # allocates the staging buffers
        v.sentinel_verify_host(hx[b][ACT][0], ACT, hs[0], hf[0], main)
    torch.cuda.synchronize()
    replicas.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main)
    for i in range(e2e_steps):
        for b, v in enumerate(vs):
            v.sentinel_verify_host(hx[b][ACT][i % len(hx[b][ACT])], ACT, hs[0], hf[0], main)
            v.sentinel_verify_host(hx[b][GRAD][i % len(hx[b][GRAD])], GRAD, hs[1], hf[1], main)
    e1.record(main)
    torch.cuda.synchronize()
    e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1))
    error_word = max(int(v.sentinel_get_counters()["error"]) for v in vs)
    for v in vs:
        v.sentinel_destroy()
    del hx
    h2d_step = 2 * N * 2 * nb
    e2e_gbs = world * e2e_steps * m.bytes_step / (e2e_ms * 1e-3) / 1e9

    out = {
        "metric": "verified GB/s (x bf16 read + reference fp32 read + EMA fp32 write = 10 B/element)",
        "value": fig["value"], "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": fig["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "impl": "sentinel_b200",
        "config": {"workload": workload_text(w),
                   "step": "sentinel_verify(h, ACT) + sentinel_verify(g, GRAD)" + (" on each boundary" if nb > 1 else ""),
                   "timed": "the %d steps gone through %d times (%d steps, %.0f ms of device time): at least %.0f ms "
                            "whatever --steps is" % (args.steps, fig["repeats"], fig["timed_steps"], fig["timed_ms"], args.min_ms),
                   "l2": fig["l2"], "replicas": world},
        "timed_steps": fig["timed_steps"], "microbatches_per_s": fig["microbatches_per_s"],
        "tensor_gbs": fig["tensor_gbs"], "ms_per_step_median": fig["ms_per_step_median"],
        "ms_per_step_best": fig["ms_per_step_best"], "frac_of_8000_nominal": fig["frac_of_8000_nominal"],
        "gpu_launches": fig["gpu_launches"], "violations_seen": violations, "error_word": error_word,
        "detection": fig["detection"], "clocks": fig["clocks"],
        "e2e": {"value": round(e2e_gbs, 2), "unit": "GB/s", "steps": e2e_steps,
                "h2d_bytes_per_step": h2d_step, "d2h_bytes_per_step": 2 * (1 + w.B) * (3 * 4 + 4) * nb,
                "bound": "pcie", "h2d_gbs": round(world * e2e_steps * h2d_step / (e2e_ms * 1e-3) / 1e9, 2),
                "note": "one staging buffer: copy in, launch, copy out, in stream order; the host-to-device copy is "
                        "what the time is spent on",
                "api": "sentinel_verify_host"},
        "roofline": fig["roofline"],
    }
    out.update(extra_keys)

    # the other stream configurations, after this one's buffers are gone: same measurement, shorter
    if extras and args.workload == "cfg4" and args.also:
        del xs, vs, m.xs, m.vs, scores, flags
        torch.cuda.empty_cache()
        for name in args.also.split(","):
            wo = synth.WORKLOADS[name]
            f2, m2 = measure_workload(binding, wo, args, rank, world, local_rank, sampler, min(args.steps, 24),
                                      args.warmup, args.min_ms / 2, 12)
            for v in m2.vs:
                v.sentinel_destroy()
            del m2
            torch.cuda.empty_cache()
            out[name] = {"workload": workload_text(wo), "value": f2["value"], "unit": "GB/s",
                         "ms_per_launch": f2["roofline"]["avg_launch_ms"], "frac": f2["roofline"]["frac"],
                         "frac_of_8000_nominal": f2["frac_of_8000_nominal"],
                         "microbatches_per_s": f2["microbatches_per_s"], "ms_per_step_median": f2["ms_per_step_median"],
                         "timed_steps": f2["timed_steps"], "gpu_launches": f2["gpu_launches"], "clocks": f2["clocks"]}
    if rank == 0 and args.cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(w, args.cpu_seconds)
        out["cpu_baseline"]["all_cores"] = cpu_baseline_all_cores(w, args.cpu_seconds)
    return out


def oracle_sample_shape(w, rows):
    """A bounded slice of the workload for the CPU oracle: one sample, `rows` token rows."""
    return synth.scaled(w, w.name + "_cpu_sample", 1, min(rows, w.T), w.d)


def cpu_baseline(w, budget_s):
    """The float64 oracle, as it stands, timed on this host on a bounded sample."""
    import oracle
    ws = oracle_sample_shape(w, 8192)
    n = ws.B * ws.T * ws.d
    v = oracle.Verifier(oracle.Params(B=ws.B, T=ws.T, d=ws.d))
    for kind in (ACT, GRAD):
        v.update_reference(synth.bits(synth.clean(ws, 0, kind, 0)), kind)
    done, t_total = 0, 0.0
    while t_total < budget_s and done < 8:
        xa = synth.bits(synth.clean(ws, 0, ACT, 1 + done))
        xg = synth.bits(synth.clean(ws, 0, GRAD, 1 + done))
        t0 = time.perf_counter()
        v.verify(xa, ACT)
        v.verify(xg, GRAD)
        t_total += time.perf_counter() - t0
        done += 1
    v.close()
    return {"value": round(done * 2 * n * BYTES_PER_ELEMENT / t_total / 1e9, 4), "unit": "GB/s",
            "cores": 1, "kind": "oracle",
            "host_cores_available": len(os.sched_getaffinity(0)),
            "sample": "%d steps (h and g) of one sample [1,%d,%d] of the workload, float64, single thread"
                      % (done, ws.T, ws.d),
            "ms_per_step": round(1e3 * t_total / done, 1)}


def _oracle_process(name, rows, index, budget_s, gate, results):
    """One of the processes of cpu_baseline_all_cores: its own slice of the workload, its own oracle
    verifier (unchanged, single-threaded), timed between a common start and its own end."""
    torch.set_num_threads(1)
    import oracle
    ws = oracle_sample_shape(synth.WORKLOADS[name], rows)
    v = oracle.Verifier(oracle.Params(B=ws.B, T=ws.T, d=ws.d))
    for kind in (ACT, GRAD):
        v.update_reference(synth.bits(synth.clean(ws, index, kind, 0)), kind)
    xs = [(synth.bits(synth.clean(ws, index, ACT, 1 + i)), synth.bits(synth.clean(ws, index, GRAD, 1 + i)))
          for i in range(2)]
    gate.wait()                                      # every process starts its steps together
    t0 = time.perf_counter()
    done = 0
    while time.perf_counter() - t0 < budget_s:
        v.verify(xs[done % 2][0], ACT)
        v.verify(xs[done % 2][1], GRAD)
        done += 1
    results.put((done, time.perf_counter() - t0, ws.B * ws.T * ws.d))
    v.close()


def cpu_baseline_all_cores(w, budget_s):
    """The same oracle on every core this process may use: one process per core (started with
    `spawn`: a fork after the first CUDA call would hang), each verifying its own slice."""
    import multiprocessing as mp
    cores = len(os.sched_getaffinity(0))
    rows = 1024
    ctx = mp.get_context("spawn")
    gate, results = ctx.Barrier(cores), ctx.Queue()
    procs = [ctx.Process(target=_oracle_process, args=(w.name, rows, i, min(budget_s, 10.0), gate, results))
             for i in range(cores)]
    for p in procs:
        p.start()
    got = []
    try:
        for _ in procs:
            got.append(results.get(timeout=180 + budget_s))
    except Exception as e:                            # a process died: report what there is
        for p in procs:
            p.terminate()
        return {"unavailable": "all-cores run failed: %r" % (e,), "cores": cores}
    for p in procs:
        p.join()
    steps = sum(g[0] for g in got)
    wall = max(g[1] for g in got)
    n = got[0][2]
    return {"value": round(steps * 2 * n * BYTES_PER_ELEMENT / wall / 1e9, 4), "unit": "GB/s", "cores": cores,
            "kind": "oracle",
            "sample": "%d processes, one per core, each %d..%d steps (h and g) of its own slice [1,%d,%d] of the "
                      "workload, float64, for %.0f s" % (cores, min(g[0] for g in got), max(g[0] for g in got),
                                                         min(rows, w.T), w.d, wall)}


def run_reference(args, rank, world):
    """--impl reference: the CPU oracle on the same workload's shape, each step a bounded sample."""
    if rank != 0:
        return None
    import oracle
    w = synth.WORKLOADS[args.workload]
    ws = oracle_sample_shape(w, 1024)
    n = ws.B * ws.T * ws.d
    v = oracle.Verifier(oracle.Params(B=ws.B, T=ws.T, d=ws.d))
    for t in range(2):
        for kind in (ACT, GRAD):
            v.update_reference(synth.bits(synth.clean(ws, 0, kind, t)), kind)
    xs = [(synth.bits(synth.clean(ws, 0, ACT, 2 + i)), synth.bits(synth.clean(ws, 0, GRAD, 2 + i)))
          for i in range(min(args.warmup + args.steps, 8))]
    for i in range(args.warmup):
        v.verify(xs[i % len(xs)][0], ACT)
        v.verify(xs[i % len(xs)][1], GRAD)
    t0 = time.perf_counter()
    for i in range(args.steps):
        xa, xg = xs[(args.warmup + i) % len(xs)]
        v.verify(xa, ACT)
        v.verify(xg, GRAD)
    dt = time.perf_counter() - t0
    v.close()
    gbs = args.steps * 2 * n * BYTES_PER_ELEMENT / dt / 1e9
    sample = "each step: h and g of one sample slice [1,%d,%d] of %s, float64, single thread" % (ws.T, ws.d, w.name)
    return {
        "metric": "verified GB/s (x bf16 read + reference fp32 read + EMA fp32 write = 10 B/element)",
        "value": round(gbs, 4), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(1e3 * dt / args.steps, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "impl": "reference",
        "config": {"workload": "%s: B=%d x T=%d x d=%d bf16" % (w.name, w.B, w.T, w.d), "sample": sample},
        "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    global EXTRAS_MIN_MS
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--distinct", type=int, default=MAX_DISTINCT,
                    help="distinct input tensors per kind kept resident (they rotate beyond that)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--no-extras", dest="extras", action="store_false",
                    help="skip the extra figures measured after the timed region")
    ap.add_argument("--min-ms", type=float, default=MIN_TIMED_MS,
                    help="device time the timed region covers at least (the steps are gone through again)")
    ap.add_argument("--extras-ms", type=float, default=EXTRAS_MIN_MS,
                    help="device time each figure taken after the timed region covers at least")
    ap.add_argument("--also", default="cfg3,cfg5",
                    help="workloads measured after the default one (cfg4) in the same run; '' for none")
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu DRAM bytes per launch of the current kernel, if known")
    args = ap.parse_args()
    EXTRAS_MIN_MS = args.extras_ms
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":        # rank 0 alone works; no process group is needed
        rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
        out = run_reference(args, rank, world)
    else:
        rank, world, local_rank = replicas.init_from_env(backend="nccl")
        out = run_ours(args, rank, world, local_rank)
        replicas.shutdown()
    if rank == 0 and out is not None:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
