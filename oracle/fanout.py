"""The single-threaded oracle fanned out over the host's cores by row ranges.

TEST INFRASTRUCTURE ONLY (as the rest of this package).  Nothing of the method's arithmetic lives
here: every worker process calls ``oracle.draft_batch`` / ``oracle.verify_batch`` on a contiguous
range of sequences and the pieces are concatenated, so the results are those of the sequential call
bit for bit.  The logits travel through POSIX shared memory (they are the only large arrays); the
workers are started with ``spawn`` so that a pool may be made after CUDA has been initialised.
"""
from __future__ import annotations

import multiprocessing as mp
import os
from multiprocessing import shared_memory

import numpy as np


def cores() -> int:
    """Host cores this process may run on."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _attach(name, shape):
    shm = shared_memory.SharedMemory(name=name)
    return shm, np.ndarray(shape, np.float32, buffer=shm.buf)


def _work(job):
    from . import oracle as orc   # in the worker: the plain sequential oracle

    kind, method, names, shape, b0, b1, temps, tokens, uniforms, node_kind = job
    if shape is None:            # no shared memory on this host: the rows came with the job
        shms, arrs = [], list(names)
    else:
        shms, arrs = zip(*[_attach(nm, shape) for nm in names])
        arrs = [a[b0:b1] for a in arrs]
    try:
        if kind == "draft":
            out = orc.draft_batch(method, arrs[0], temps, uniforms)
        else:
            out = orc.verify_batch(method, arrs[0], arrs[1], temps, tokens, uniforms, node_kind)
    finally:
        del arrs
        for s in shms:
            s.close()
    return out


class Pool:
    """``Pool(n)`` starts n worker processes (default: one per available core)."""

    def __init__(self, n: int | None = None):
        self.n = max(1, n or cores())
        self._pool = mp.get_context("spawn").Pool(self.n)

    def close(self):
        self._pool.close()
        self._pool.join()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def _share(self, arrays):
        shms = []
        try:
            for a in arrays:
                a = np.ascontiguousarray(a, np.float32)
                shm = shared_memory.SharedMemory(create=True, size=max(a.nbytes, 1))
                shms.append(shm)
                np.ndarray(a.shape, np.float32, buffer=shm.buf)[...] = a
        except (OSError, ValueError) as exc:
            for s in shms:
                s.close()
                s.unlink()
            raise OSError(str(exc))
        return shms

    def _ranges(self, B):
        per = max(1, -(-B // (self.n * 4)))   # a few chunks per worker evens out uneven rows
        return [(b0, min(B, b0 + per)) for b0 in range(0, B, per)]

    def _run(self, kind, method, logits, temps, tokens, uniforms, node_kind):
        B = logits[0].shape[0]
        t = np.asarray(temps, np.float32)
        t = np.full(B, float(t), np.float32) if t.ndim == 0 else t
        try:
            shms = self._share(logits)
        except OSError:          # /dev/shm missing or too small: hand the rows over with the jobs instead
            shms = None
        if shms is None:
            jobs = [(kind, method, [np.ascontiguousarray(a[b0:b1], np.float32) for a in logits], None, b0, b1,
                     t[b0:b1], None if tokens is None else tokens[b0:b1], uniforms[b0:b1], node_kind)
                    for b0, b1 in self._ranges(B)]
            return self._pool.map(_work, jobs)
        try:
            jobs = [(kind, method, [s.name for s in shms], logits[0].shape, b0, b1, t[b0:b1],
                     None if tokens is None else tokens[b0:b1], uniforms[b0:b1], node_kind)
                    for b0, b1 in self._ranges(B)]
            return self._pool.map(_work, jobs)
        finally:
            for s in shms:
                s.close()
                s.unlink()

    def draft_batch(self, method, draft_logits, temperature, uniforms):
        """As ``oracle.draft_batch``, in parallel over ranges of sequences."""
        parts = self._run("draft", method, [draft_logits], temperature, None, uniforms, None)
        return {k: np.concatenate([p[k] for p in parts]) for k in parts[0]}

    def verify_batch(self, method, target_logits, draft_logits, temperature, draft_tokens, uniforms,
                     node_kind=None):
        """As ``oracle.verify_batch``, in parallel over ranges of sequences."""
        parts = self._run("verify", method, [target_logits, draft_logits], temperature, draft_tokens, uniforms,
                          node_kind)
        return np.concatenate(parts)
