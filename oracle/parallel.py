"""Runs oracle work on every host core (test infrastructure only, like the rest of oracle/).

The oracle is one position at a time and single-threaded; positions and groups are
independent, so a full-size parity check or a timed baseline simply hands whole groups to
worker processes.  Each worker is a fresh interpreter (spawn: the parent may hold a CUDA
context, which must not be forked) with numpy limited to one thread.  Inputs are sent to a
worker first and the work is started afterwards, so a timed run does not count the transfer.

Adds no arithmetic: a task is a call of a function of oracle/ (or of the test harness) on
the arrays it was given.
"""
from __future__ import annotations

import importlib
import multiprocessing as mp
import os
import sys
import time
import traceback


def _worker(conn, sys_path):
    for var in ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS", "NUMEXPR_NUM_THREADS"):
        os.environ[var] = "1"
    os.environ["CUDA_VISIBLE_DEVICES"] = ""
    for p in reversed(sys_path):
        if p not in sys.path:
            sys.path.insert(0, p)
    stash = {}
    while True:
        try:
            msg = conn.recv()
        except EOFError:
            return
        op = msg[0]
        try:
            if op == "put":
                stash[msg[1]] = msg[2]
                conn.send(("ok", None))
            elif op == "call":
                _, module, name, keys, common, drop = msg
                fn = getattr(importlib.import_module(module), name)
                out = []
                for key in keys:
                    t0 = time.perf_counter()
                    res = fn(**(stash.pop(key) if drop else stash[key]), **common)
                    out.append((key, time.perf_counter() - t0, res))
                conn.send(("ok", out))
            elif op == "stop":
                conn.send(("ok", None))
                return
        except BaseException:
            conn.send(("error", traceback.format_exc()))


class OracleWorkers:
    """n worker processes.  put() sends a payload (a dict of keyword arguments) to the worker
    that owns its key; call() then runs a function on stored payloads, every worker going
    through its own keys in order, and returns the results with the wall time of that
    compute phase alone and each task's own time.  run() does both for a list of payloads,
    at most one payload per worker in memory at a time."""

    def __init__(self, n: int | None = None, extra_sys_path=()):
        self.n = max(1, n or os.cpu_count() or 1)
        ctx = mp.get_context("spawn")
        paths = list(extra_sys_path) + [os.path.dirname(os.path.dirname(os.path.abspath(__file__)))]
        self.procs, self.conns = [], []
        for _ in range(self.n):
            a, b = ctx.Pipe()
            p = ctx.Process(target=_worker, args=(b, paths), daemon=True)
            p.start()
            b.close()
            self.procs.append(p)
            self.conns.append(a)

    def _answer(self, w):
        status, val = self.conns[w].recv()
        if status != "ok":
            raise AssertionError(f"oracle worker {w} failed:\n{val}")
        return val

    def put(self, key: int, payload: dict):
        self.conns[key % self.n].send(("put", key, payload))
        self._answer(key % self.n)

    def call(self, module: str, function: str, keys, common: dict | None = None, drop: bool = True):
        """Returns (results by key, wall seconds, per-task seconds by key)."""
        per_worker = {}
        for key in keys:
            per_worker.setdefault(key % self.n, []).append(key)
        t0 = time.perf_counter()
        for w, ks in per_worker.items():
            self.conns[w].send(("call", module, function, ks, common or {}, drop))
        results, seconds, failure = {}, {}, None
        for w in per_worker:
            try:
                for key, dt, res in self._answer(w):
                    results[key], seconds[key] = res, dt
            except AssertionError as e:          # drain the other workers before raising
                failure = failure or e
        if failure is not None:
            raise failure
        return results, time.perf_counter() - t0, seconds

    def run(self, module: str, function: str, payloads: list, common: dict | None = None):
        """(results in payload order, wall seconds of the compute phases)."""
        results = [None] * len(payloads)
        wall = 0.0
        for w0 in range(0, len(payloads), self.n):
            wave = list(range(w0, min(w0 + self.n, len(payloads))))
            for i in wave:
                self.put(i, payloads[i])
            res, dt, _ = self.call(module, function, wave, common)
            wall += dt
            for i in wave:
                results[i] = res[i]
        return results, wall

    def close(self):
        for c in self.conns:
            try:
                c.send(("stop",))
                c.recv()
            except Exception:
                pass
            c.close()
        for p in self.procs:
            p.join(timeout=5)
            if p.is_alive():
                p.kill()
        self.procs, self.conns = [], []

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


def encode_logits(t):
    """A torch tensor of logits -> (numpy array of its raw storage, dtype tag): 16-bit types
    travel as int16 so that a group of full-vocabulary rows stays small on the pipe."""
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.float32:
        return t.numpy(), "f32"
    tag = {torch.bfloat16: "bf16", torch.float16: "f16"}[t.dtype]
    return t.view(torch.int16).numpy(), tag


def decode_logits(raw, tag):
    """Inverse of encode_logits: the stored values, exactly, as float32."""
    import numpy as np
    if tag == "f32":
        return raw
    if tag == "f16":
        return raw.view(np.float16).astype(np.float32)
    return (raw.view(np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
