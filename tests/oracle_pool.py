"""The float64 oracle in worker processes, one per (boundary, kind) stream.

The full-size parity tests verify tensors of up to 512 MiB over dozens of steps; the oracle
needs seconds per tensor, so the streams of a test run side by side on the host's cores while the
GPU path waits for them step by step.  A worker owns one unchanged oracle verifier and advances
one kind of it; the tensor of a step reaches it through a memory-mapped file (bf16 bit patterns
written by the test), small results come back through a queue, and on request the worker writes
its verifier's checkpoint blob into a second file.

Processes are started with ``spawn``: a fork after the first CUDA call of the parent would hang.
"""
from __future__ import annotations

import multiprocessing as mp
import os
import shutil
import tempfile

import numpy as np

ACT, GRAD = 0, 1


def _worker(root, shape, kw, kind, x_path, blob_path, cmd_q, res_q):
    import sys
    for p in (root, os.path.join(root, "tests")):
        if p not in sys.path:
            sys.path.insert(0, p)
    import oracle
    from helpers import oracle_to_blob
    B, T, d = shape
    params = oracle.Params(B=B, T=T, d=d, **kw)
    ov = oracle.Verifier(params)
    x = np.memmap(x_path, dtype=np.uint16, mode="r", shape=shape)
    try:
        while True:
            msg = cmd_q.get()
            if msg[0] == "stop":
                break
            if msg[0] == "step":
                _, t, warm = msg
                thr_before, valid_before = ov.thresholds(kind)
                if warm:
                    scores, _ = ov.update_reference(x, kind)
                    flags, commit = None, True
                else:
                    scores, flags, commit = ov.verify(x, kind)
                thr, valid = ov.thresholds(kind)
                res_q.put(("step", t, np.array(scores), None if flags is None else np.array(flags), bool(commit),
                           np.array(thr_before), np.array(valid_before), np.array(thr), np.array(valid),
                           np.array(ov.last_stats(kind)), int(ov.steps(kind)),
                           [int(ov.history(kind, L, 0).size) for L in (0, 1)]))
            elif msg[0] == "blob":          # the verifier's checkpoint, for a re-alignment of the library
                with open(blob_path, "wb") as fh:
                    fh.write(oracle_to_blob(ov, params))
                res_q.put(("blob", blob_path))
    finally:
        del x
        ov.close()


def scratch_dir(need_bytes: int) -> str:
    """A directory for the tensors in flight: memory-backed if it has the room, else the temp dir."""
    for base in ("/dev/shm", tempfile.gettempdir()):
        try:
            if os.path.isdir(base) and shutil.disk_usage(base).free > need_bytes + (1 << 30):
                return tempfile.mkdtemp(prefix="sentinel_oracle_", dir=base)
        except OSError:
            continue
    return tempfile.mkdtemp(prefix="sentinel_oracle_")


class OracleStream:
    """One oracle worker: a (boundary, kind) stream of a workload."""

    def __init__(self, ctx, root, folder, tag, shape, kw, kind):
        self.kind = kind
        self.x_path = os.path.join(folder, "%s_x.bin" % tag)
        self.blob_path = os.path.join(folder, "%s_state.bin" % tag)
        self.x = np.memmap(self.x_path, dtype=np.uint16, mode="w+", shape=shape)
        self.cmd, self.res = ctx.Queue(), ctx.Queue()
        self.proc = ctx.Process(target=_worker, args=(root, shape, kw, kind, self.x_path, self.blob_path,
                                                      self.cmd, self.res), daemon=True)
        self.proc.start()

    def step(self, bits, t, warm):
        """Hands the worker the tensor of step t: uint16 bit patterns of the stream's shape, or a
        bf16 torch tensor (copied from the device straight into the mapped file)."""
        if hasattr(bits, "data_ptr"):
            import torch
            torch.from_numpy(self.x.view(np.int16)).copy_(bits.detach().contiguous().view(torch.int16))
        else:
            np.copyto(self.x, bits)
        self.cmd.put(("step", t, warm))

    def ready(self):
        if not self.res.empty():
            return True
        if not self.proc.is_alive():
            raise RuntimeError("the oracle process of kind %d ended (exit code %r)" % (self.kind, self.proc.exitcode))
        return False

    def result(self, timeout=900):
        """The worker's next answer; fails (rather than waits) if the process is gone."""
        import queue
        waited = 0.0
        while True:
            try:
                return self.res.get(timeout=1.0)
            except queue.Empty:
                waited += 1.0
                if not self.proc.is_alive():
                    raise RuntimeError("the oracle process of kind %d ended (exit code %r)" % (self.kind, self.proc.exitcode))
                if waited >= timeout:
                    raise TimeoutError("the oracle process of kind %d did not answer in %d s" % (self.kind, timeout))

    def blob(self, timeout=900) -> bytes:
        self.cmd.put(("blob",))
        tag, path = self.result(timeout)
        assert tag == "blob"
        with open(path, "rb") as fh:
            data = fh.read()
        os.remove(path)
        return data

    def close(self):
        try:
            self.cmd.put(("stop",))
            self.proc.join(timeout=30)
            if self.proc.is_alive():
                self.proc.terminate()
        finally:
            del self.x
            for path in (self.x_path, self.blob_path):
                if os.path.exists(path):
                    os.remove(path)


def context():
    return mp.get_context("spawn")
