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
# dram__bytes_read.sum + dram__bytes_write.sum per element of the current stream_kernel, from the
# ncu capture summarised in profiles/stream_kernel_cfg3_ncu_full.md (B=8 x 4096 x 4096; traffic
# grows in proportion to the element count, so a launch of N elements moves this times N).
# Set to None whenever the kernel changes until the capture is retaken.
NCU_DRAM_BYTES_PER_ELEMENT = 9.679


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

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
            self.lines.append(line.strip())

    def __exit__(self, *exc):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()          # the exact process started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self) -> dict:
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            tok = [t.strip() for t in line.split(",")]
            if len(tok) < 6:
                continue
            try:
                sm.append(float(tok[0]))
                smax.append(float(tok[1]))
            except ValueError:
                continue
            for name, val in zip(names, tok[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


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


def run_ours(args, rank, world, local_rank):
    from paper_2603_03592_b200 import binding
    binding.lib()                                   # no library, no benchmark: there is no fallback
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    w = synth.WORKLOADS[args.workload]
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

    total = args.warmup + args.steps
    distinct = args.distinct if nb == 1 else min(args.distinct, 12)   # 8 boundaries: bound the footprint
    xs = [build_stream(w, b, device, total, distinct) for b in range(nb)]
    nd = len(xs[0][ACT])
    scores = torch.empty(nb, 2, 1 + w.B, 3, dtype=torch.float32, device=device)
    flags = torch.empty(nb, 2, 1 + w.B, dtype=torch.int32, device=device)
    flag_log = torch.zeros(total, nb, 2, 1 + w.B, dtype=torch.int32, device=device)   # every step's flags
    torch.cuda.synchronize()

    def step(i):
        for b, (v, s) in enumerate(zip(vs, streams)):
            v.sentinel_verify(xs[b][ACT][i % nd], ACT, scores[b, 0], flag_log[i, b, 0], s)
            v.sentinel_verify(xs[b][GRAD][i % nd], GRAD, scores[b, 1], flag_log[i, b, 1], s)

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
    for i in range(args.warmup):
        step(i)
    join()
    torch.cuda.synchronize()
    replicas.barrier()
    torch.cuda.synchronize()

    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    with ClockSampler(local_rank) as clocks:
        marks[0].record(main)
        fork()
        for i in range(args.steps):
            step(args.warmup + i)
            if nb == 1:
                marks[i + 1].record(main)
        join()
        if nb > 1:
            marks[-1].record(main)
        torch.cuda.synchronize()
    replicas.barrier()
    torch.cuda.synchronize()
    local_ms = elapsed_ms = marks[0].elapsed_time(marks[-1])
    if nb == 1:
        step_ms = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps))
    else:
        step_ms = [local_ms / args.steps]
    elapsed_ms = replicas.max_over_ranks(elapsed_ms)
    launches = 2 * args.steps * nb
    violations = sum(int(v.sentinel_get_counters()["violations"]) for v in vs)
    # what the detector said on the timed steps (reported, not a target: some of the recipe's
    # corruptions are statistically invisible to these metrics, and a flagged tensor that comes
    # round again is flagged again)
    raised = ((flag_log[args.warmup:] & 0xFFFF) != 0).any(dim=-1).cpu()              # [steps, nb, 2]
    n_corrupted = n_flagged = n_both = 0
    for i in range(args.steps):
        for b in range(nb):
            for kind in (ACT, GRAD):
                c = xs[b]["corrupted"][kind][(args.warmup + i) % nd]
                f = bool(raised[i, b, kind])
                n_corrupted += c
                n_flagged += f
                n_both += c and f
    detection = {"tensors": args.steps * nb * 2, "corrupted": n_corrupted, "flagged": n_flagged,
                 "corrupted_and_flagged": n_both, "distinct_tensors_per_kind": nd,
                 "note": "the stream cycles through the distinct tensors; one that comes round again soon "
                         "correlates with the reference that absorbed it and is flagged as a replay"}

    # extra figure, outside the timed region: gradient replacement (Alg. 4) after a flagged step
    extras = nb == 1 and args.extras and world == 1     # the extra figures are single-GPU figures
    replace = None
    if extras:
        v0 = vs[0]
        loud = (xs[0][GRAD][0].float() * 64.0).to(torch.bfloat16)
        v0.sentinel_verify(loud, GRAD, scores[0, 1], flags[0, 1], main)       # flagged: no commit
        outs = [torch.empty_like(loud) for _ in range(4)]
        for o in outs:
            v0.sentinel_replace_if_flagged(o, GRAD, 0, None, main)
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        r0.record(main)
        for i in range(12):
            v0.sentinel_replace_if_flagged(outs[i % 4], GRAD, 0, None, main)
        r1.record(main)
        torch.cuda.synchronize()
        rms = r0.elapsed_time(r1) / 12
        replace = {"kernel": "replace_kernel", "bytes_per_element": 6, "ms_per_launch": round(rms, 4),
                   "achieved_gbs": round(6 * N / (rms * 1e-3) / 1e9, 1),
                   "flagged": bool(int(flags[0, 1, 0]) & 0xFFFF)}

    # extra figure, outside the timed region: sliced Wasserstein distance along 8 directions
    swd = None
    if extras and 8 * w.d * 2 <= 200 * 1024 and w.T <= 16384:
        g = torch.Generator(device=device).manual_seed(11)
        u = torch.randn(8, w.d, generator=g, device=device)
        u = (u / u.norm(dim=1, keepdim=True)).to(torch.bfloat16).contiguous()
        ref = xs[0][ACT][1 % nd].float().mul_(0.1).contiguous()
        sw = torch.empty(1 + w.B, dtype=torch.float32, device=device)
        for _ in range(2):
            binding.sentinel_sliced_wasserstein(xs[0][ACT][0], ref, u, sw, main)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        s0.record(main)
        for i in range(8):
            binding.sentinel_sliced_wasserstein(xs[0][ACT][i % nd], ref, u, sw, main)
        s1.record(main)
        torch.cuda.synchronize()
        sms = s0.elapsed_time(s1) / 8
        swd = {"directions": 8, "bytes_per_element": 6, "ms_per_call": round(sms, 4),
               "achieved_gbs": round(6 * N / (sms * 1e-3) / 1e9, 1),
               "kernels": "swd_project_kernel + sort, merge, finish", "value_row0": float(sw[0])}
        del ref
        # the same distance as the verifier's fourth metric: one verified tensor per call, the
        # projection / sort chain (x only: the reference's projections are carried along) followed by
        # the streaming launch: 2 + 6 B/element read, 4 written
        v4 = binding.Verifier(w.B, w.T, w.d, device=local_rank)
        v4.sentinel_set_directions(u, main)
        s4 = torch.empty(1 + w.B, 4, dtype=torch.float32, device=device)
        f4 = torch.zeros(1 + w.B, dtype=torch.int32, device=device)
        for i in range(4):
            v4.sentinel_update_reference(xs[0][ACT][i % nd], ACT, s4, main)
        v4.sentinel_verify(xs[0][ACT][4 % nd], ACT, s4, f4, main)
        torch.cuda.synchronize()
        s0.record(main)
        for i in range(8):
            v4.sentinel_verify(xs[0][ACT][(5 + i) % nd], ACT, s4, f4, main)
        s1.record(main)
        torch.cuda.synchronize()
        vms = s0.elapsed_time(s1) / 8
        swd["verify_with_four_metrics"] = {"ms_per_tensor": round(vms, 4), "bytes_per_element": 12,
                                           "achieved_gbs": round(12 * N / (vms * 1e-3) / 1e9, 1)}
        v4.close()

    # extra figure, outside the timed region: one iteration with R workers of the stage
    # (one launch: 2R B/element of tensors + 4 B read and 4 B written of the reference)
    replicas_fig = None
    if extras:
        R = 4 if 100 * 4 * (w.B + 1) <= 4096 else 2
        vr = binding.Verifier(w.B, w.T, w.d, device=local_rank, n_workers=R)
        rs = torch.empty(R, 1 + w.B, 3, dtype=torch.float32, device=device)
        rf = torch.zeros(R, 1 + w.B, dtype=torch.int32, device=device)
        pick = lambda i: [xs[0][ACT][(i * R + r) % nd] for r in range(R)]
        for i in range(4):
            vr.sentinel_update_reference_replicas(pick(i), ACT, rs, rf, main)
        vr.sentinel_verify_replicas(pick(4), ACT, rs, rf, main)
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        q0.record(main)
        for i in range(6):
            vr.sentinel_verify_replicas(pick(5 + i), ACT, rs, rf, main)
        q1.record(main)
        torch.cuda.synchronize()
        qms = q0.elapsed_time(q1) / 6
        per_el = 2 * R + 8                      # every tensor once, the reference read and written once
        flagged_workers = int(((rf[:, 0] & 0xFFFF) != 0).sum())
        replicas_fig = {"workers": R, "bytes_per_element": per_el, "ms_per_iteration": round(qms, 4),
                        "achieved_gbs": round(per_el * N / (qms * 1e-3) / 1e9, 1),
                        "submissions_per_s": round(R / (qms * 1e-3), 1),
                        "flagged_workers_last_iteration": flagged_workers,
                        "kernels": "replica_kernel (all workers, speculative mean) + ema_mean_kernel (report bits)"}
        vr.sentinel_destroy()

    # extra figure, outside the timed region: the reference kept as bf16 (6 B/element per tensor)
    half = None
    if extras:
        vh = binding.Verifier(w.B, w.T, w.d, device=local_rank, ema_bf16=1)
        hs_, hf_ = torch.empty(1 + w.B, 3, dtype=torch.float32, device=device), torch.zeros(1 + w.B, dtype=torch.int32, device=device)
        for i in range(6):
            vh.sentinel_update_reference(xs[0][ACT][i % nd], ACT, hs_, main)
        vh.sentinel_verify(xs[0][ACT][6 % nd], ACT, hs_, hf_, main)
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        h0.record(main)
        for i in range(20):
            vh.sentinel_verify(xs[0][ACT][(7 + i) % nd], ACT, hs_, hf_, main)
        h1.record(main)
        torch.cuda.synchronize()
        hms = h0.elapsed_time(h1) / 20
        half = {"bytes_per_element": 6, "ms_per_launch": round(hms, 4),
                "achieved_gbs": round(6 * N / (hms * 1e-3) / 1e9, 1),
                "tensors_per_s": round(1e3 / hms, 1), "kernel": "stream_kernel_t<false, true>"}
        vh.sentinel_destroy()

    # extra figure, outside the timed region: one [T,d] reference for all samples (2 + 8/B B/element)
    shared = None
    if extras and w.B <= 16:
        vsr = binding.Verifier(w.B, w.T, w.d, device=local_rank, ref_over_batch=1)
        ss_, sf_ = torch.empty(1 + w.B, 3, dtype=torch.float32, device=device), torch.zeros(1 + w.B, dtype=torch.int32, device=device)
        for i in range(6):
            vsr.sentinel_update_reference(xs[0][ACT][i % nd], ACT, ss_, main)
        vsr.sentinel_verify(xs[0][ACT][6 % nd], ACT, ss_, sf_, main)
        z0, z1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        z0.record(main)
        for i in range(20):
            vsr.sentinel_verify(xs[0][ACT][(7 + i) % nd], ACT, ss_, sf_, main)
        z1.record(main)
        torch.cuda.synchronize()
        zms = z0.elapsed_time(z1) / 20
        per_el = 2 + 8.0 / w.B
        shared = {"bytes_per_element": per_el, "ms_per_launch": round(zms, 4),
                  "achieved_gbs": round(per_el * N / (zms * 1e-3) / 1e9, 1),
                  "tensors_per_s": round(1e3 / zms, 1), "kernel": "shared_ref_kernel"}
        vsr.sentinel_destroy()

    # extra figure, outside the timed region: one [d] reference for all tokens (x alone streams, 2 B/element)
    channel = None
    if extras:
        vcr = binding.Verifier(w.B, w.T, w.d, device=local_rank, ref_over_batch=1, ref_over_tokens=1)
        cs_, cf_ = torch.empty(1 + w.B, 3, dtype=torch.float32, device=device), torch.zeros(1 + w.B, dtype=torch.int32, device=device)
        for i in range(6):
            vcr.sentinel_update_reference(xs[0][ACT][i % nd], ACT, cs_, main)
        vcr.sentinel_verify(xs[0][ACT][6 % nd], ACT, cs_, cf_, main)
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        q0.record(main)
        for i in range(20):
            vcr.sentinel_verify(xs[0][ACT][(7 + i) % nd], ACT, cs_, cf_, main)
        q1.record(main)
        torch.cuda.synchronize()
        qms = q0.elapsed_time(q1) / 20
        channel = {"bytes_per_element": 2, "ms_per_step": round(qms, 4),
                   "achieved_gbs": round(2 * N / (qms * 1e-3) / 1e9, 1),
                   "tensors_per_s": round(1e3 / qms, 1), "kernels": "channel_ref_kernel + channel_mean_kernel"}
        vcr.sentinel_destroy()
        # the same with a vector per sample ([B,d])
        vps = binding.Verifier(w.B, w.T, w.d, device=local_rank, ref_over_tokens=1)
        for i in range(6):
            vps.sentinel_update_reference(xs[0][ACT][i % nd], ACT, cs_, main)
        vps.sentinel_verify(xs[0][ACT][6 % nd], ACT, cs_, cf_, main)
        torch.cuda.synchronize()
        q0.record(main)
        for i in range(20):
            vps.sentinel_verify(xs[0][ACT][(7 + i) % nd], ACT, cs_, cf_, main)
        q1.record(main)
        torch.cuda.synchronize()
        channel["ms_per_step_vector_per_sample"] = round(q0.elapsed_time(q1) / 20, 4)
        vps.sentinel_destroy()

    # extra figure, outside the timed region: the strided (compressed-signal) layout, rows d+1 apart
    strided = None
    if extras:
        wide = [torch.nn.functional.pad(xs[0][ACT][i % nd], (0, 1)).contiguous() for i in range(3)]
        for i in range(2):
            vs[0].sentinel_update_reference_strided(wide[i], ACT, scores[0, 0], main)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        c0.record(main)
        for i in range(9):
            vs[0].sentinel_update_reference_strided(wide[i % 3], ACT, scores[0, 0], main)
        c1.record(main)
        torch.cuda.synchronize()
        cms = c0.elapsed_time(c1) / 9
        strided = {"row_stride": w.d + 1, "bytes_per_element": 10, "ms_per_launch": round(cms, 4),
                   "achieved_gbs": round(10 * N / (cms * 1e-3) / 1e9, 1), "kernel": "stream_kernel_t<false, false, true> (funnel-shifted rows)"}
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
    for v in vs:
        v.sentinel_destroy()

    bytes_step = 2 * N * BYTES_PER_ELEMENT * nb             # two tensors per boundary per step
    # what one pass over the cycled inputs touches, against the 126 MB L2
    cycle_bytes = nb * nd * 2 * N * BYTES_PER_ELEMENT
    if cycle_bytes > 4 * 126e6:
        l2_note = "inputs larger than L2: %d MiB read+written per launch, %d distinct tensors per kind" % (
            N * BYTES_PER_ELEMENT >> 20, nd)
    else:
        l2_note = ("inputs and state of a whole cycle (%d MiB) stay near the 126 MB L2: a launch-latency figure, "
                   "not a bandwidth figure" % (cycle_bytes >> 20))
    gbs = world * args.steps * bytes_step / (elapsed_ms * 1e-3) / 1e9
    e2e_gbs = world * e2e_steps * bytes_step / (e2e_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak_gbs()
    kernel_ms = local_ms / launches              # the timed region holds these launches only
    achieved = N * BYTES_PER_ELEMENT / (kernel_ms * 1e-3) / 1e9
    out = {
        "metric": "verified GB/s (x bf16 read + reference fp32 read + EMA fp32 write = 10 B/element)",
        "value": round(gbs, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(elapsed_ms / args.steps, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "impl": "sentinel_b200",
        "config": {"workload": "%s: B=%d x T=%d x d=%d bf16, activations %s, gradients N(0,%g), "
                               "%g%% corrupted%s" % (w.name, w.B, w.T, w.d, w.act, w.grad_std, 100 * w.corrupt_rate,
                                                     ", %d boundaries on %d CUDA streams" % (nb, nb) if nb > 1 else ""),
                   "step": "sentinel_verify(h, ACT) + sentinel_verify(g, GRAD)" + (" on each boundary" if nb > 1 else ""),
                   "l2": l2_note,
                   "replicas": world},
        "microbatches_per_s": round(world * args.steps * nb / (elapsed_ms * 1e-3), 1),
        "tensor_gbs": round(world * args.steps * nb * 2 * N * 2 / (elapsed_ms * 1e-3) / 1e9, 1),
        "ms_per_step_median": round(step_ms[len(step_ms) // 2], 4),
        "ms_per_step_best": round(step_ms[0], 4),
        "frac_of_8000_nominal": round(gbs / world / 8000.0, 4),
        "gpu_launches": launches,
        "violations_seen": violations, "detection": detection,
        "clocks": clocks.summary(),
        "e2e": {"value": round(e2e_gbs, 2), "unit": "GB/s", "steps": e2e_steps,
                "h2d_bytes_per_step": 2 * N * 2 * nb,
                "d2h_bytes_per_step": 2 * (1 + w.B) * (3 * 4 + 4) * nb,
                "api": "sentinel_verify_host"},
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "peak_source": "%s copy bandwidth" % peak_kind,
                     "kernel": "stream_kernel",
                     "avg_launch_ms": round(kernel_ms, 4),
                     "note": ("launches of different boundaries overlap: time per launch is the "
                              "timed region divided by the launches" if nb > 1 else
                              "timed region / launches; the region holds these launches only"),
                     "traffic": (args.traffic if args.traffic is not None else
                                 (round(NCU_DRAM_BYTES_PER_ELEMENT * N) if NCU_DRAM_BYTES_PER_ELEMENT else None)),
                     "traffic_source": "ncu on B=8x4096x4096, scaled by element count"},
    }
    if replace is not None:
        out["gradient_replacement"] = replace
    if swd is not None:
        out["sliced_wasserstein"] = swd
    if replicas_fig is not None:
        out["multi_worker_iteration"] = replicas_fig
    if strided is not None:
        out["compressed_layout"] = strided
    if half is not None:
        out["bf16_reference"] = half
    if shared is not None:
        out["shared_reference"] = shared
    if channel is not None:
        out["channel_reference"] = channel
    if rank == 0 and args.cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(w, args.cpu_seconds)
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
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu DRAM bytes per launch of the current kernel, if known")
    args = ap.parse_args()
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
