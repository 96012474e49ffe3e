"""Benchmark of the GTO draft-tree pass (build tree -> Draft Tree Reward -> group surrogate
gradient) on synthetic logits at the LLaMA-3.1-8B shape.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload ID]

One step = one pass of the whole hot path over the batch of B positions resident in HBM.
With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs the same
number of its own positions (weak scaling); positions are independent, so no collective is
on the data path - only the timing barrier and the max-over-ranks reduction.

Started directly with --gpus N > 1 (no WORLD_SIZE in the environment) it starts the N ranks
itself under torch.distributed.run.

Timed regions of the GPU arm, in order: (1) the headline: K steps, nothing but the three
calls; (2) the same K steps with every kernel launch bracketed by CUDA events, for the
per-kernel split and the roofline; (3) a sustained region of at least a second of
back-to-back steps, with the SM clock sampled, to show where the pass settles under the
board power limit; (4) the end-to-end leg with the logits in pinned host memory.  At N = 1
the oracle then runs on every host core over groups drawn from the same batch: its
throughput is the CPU baseline, and its results are compared with the library's for those
groups (the `parity` counts).

Prints ONE JSON line on rank 0.  `--impl reference` times the fp64 CPU oracle instead (on a
bounded sample per step), on rank 0 only.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "tree-positions/s (build+reward+grad)"
UNIT = "positions/s"
HBM_FALLBACK_GBS = 6650.0
REFERENCE_BUDGET_S = 150.0  # the oracle arm stops taking new steps after this much wall time
E2E_POSITIONS = 64          # positions per end-to-end step (host buffers of ~2.6 GB at workload 2)
SUSTAINED_SECONDS = 1.2     # length of the back-to-back region
COOLDOWN_SECONDS = 1.0      # idle time before the per-kernel region

# DRAM traffic per processed row of the dominant kernels, from one ncu capture each
# (dram__bytes_read.sum + dram__bytes_write.sum over the launch / rows in the launch).  An
# entry is used only while the kernel source it was taken from is unchanged.
NCU_TRAFFIC = {
    # kernel: (source file, sha256 of that file at capture time, bytes per row, V of the capture)
    # from the ncu capture summarised under profiles/ (row pass, workload 2 shapes at B = 64)
    "draft_rows": ("paper_2509_22134_b200/csrc/row_reduce.cu",
                   "7699dc77e539aabff69340f559f8f2480559800639a44f0c23bb4d98cb358797", (509028864 + 3841536) / 7808, 32000),
    "target_rows": ("paper_2509_22134_b200/csrc/row_reduce.cu",
                    "7699dc77e539aabff69340f559f8f2480559800639a44f0c23bb4d98cb358797", (429928448 + 3473408) / 1673, 128256),
}


def _sha256(path: str) -> str:
    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU through NVML while running."""
    _REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
                0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
                0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.01):
        self.period = period_s
        self.samples, self.stamps, self.reasons, self.max_mhz = [], [], set(), None
        self.mem_samples, self.power_samples = [], []
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.stamps.append(time.perf_counter())
                mask = int(get_reasons(self._h))
                for bit, name in self._REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.mem_samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_MEM)))
                self.power_samples.append(int(nv.nvmlDeviceGetPowerUsage(self._h)) / 1000.0)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples),
                "mem_mhz": statistics.median(self.mem_samples) if self.mem_samples else None,
                "power_w": statistics.median(self.power_samples) if self.power_samples else None}


# ------------------------------------------------------------------------ oracle legs
# Everything between here and workload_config is the CPU-baseline / reference leg: the only
# part of this file that runs the oracle.  The functions named *_task run in worker processes.
def _old_logp_fn(w, with_positions):
    from paper_2509_22134_b200 import synth

    def at(path_logp, path_row, path_token, path_len, first_of):
        out = np.zeros_like(path_logp)
        for i in range(path_logp.shape[0]):
            out[i] = synth.old_logp_from_path(w, path_logp[i:i + 1], path_row[i:i + 1],
                                              path_token[i:i + 1], path_len[i:i + 1], b0=first_of(i))[0]
        return out
    if with_positions:
        return lambda pl, pr, pt, ln, positions: at(pl, pr, pt, ln, lambda i: positions[i])
    return lambda b0: (lambda pl, pr, pt, ln: at(pl, pr, pt, ln, lambda i: b0 + i))


def oracle_group_task(w, draft, draft_tag, target, target_tag, d2t, b0, gpu=None):
    """The oracle's whole pass on one group of m positions (first absolute position b0)."""
    from oracle import gto_oracle as orc
    from oracle import parallel as opar
    out = orc.group_pass(opar.decode_logits(draft, draft_tag), opar.decode_logits(target, target_tag),
                         w.D, w.k, w.g, w.m, _old_logp_fn(w, False)(b0), d2t, w.eta,
                         delta=w.std_delta, eps=w.clip_eps, grad_scale=w.grad_scale)
    return float(out["sur"]["loss"][0])


def oracle_check_task(w, draft, draft_tag, target, target_tag, d2t, b0, gpu):
    """The library's outputs for one group against the oracle (tolerances of oracle/check.py)."""
    from oracle import check as ocheck
    from oracle import parallel as opar

    class Cfg:
        pass
    cfg = Cfg()
    for name in ("B", "G", "D", "k", "g", "m", "eta", "clip_eps", "std_delta", "grad_scale"):
        setattr(cfg, name, getattr(w, name))
    try:
        return ocheck.check_positions(cfg, opar.decode_logits(draft, draft_tag),
                                      opar.decode_logits(target, target_tag), d2t, gpu,
                                      _old_logp_fn(w, True), list(range(b0, b0 + w.m)))
    except AssertionError as e:
        return {"positions": w.m, "failed": 1, "failure": str(e)[:300]}


def _group_payload(w, data, gidx, first_position, p=None):
    """Logits (and, with p, the library's outputs) of group gidx of the batch in `data`."""
    from oracle import parallel as opar
    sl = slice(gidx * w.m, (gidx + 1) * w.m)
    draft, dtag = opar.encode_logits(data["draft"][:, sl])
    target, ttag = opar.encode_logits(data["target"][:, sl])
    d2t = None if data["d2t"] is None else data["d2t"].cpu().numpy().astype(np.int64)
    gpu = None
    if p is not None:
        gpu = {}
        for name, t in p.tree.items():
            gpu[name] = t[:, sl].cpu().numpy()
        for name, t in p.reward.items():
            gpu[name] = (t[sl] if name.startswith("path_") else t[:, sl]).cpu().numpy()
        for name, t in p.stats.items():
            gpu[name] = (t[gidx:gidx + 1] if name == "loss" else t[sl]).cpu().numpy()
        gpu["grad"] = p.grad[sl].float().cpu().numpy().astype(np.float64)
        # rows that carry no gradient are the caller's with GTO_FLAG_GRAD_LIVE_ROWS: the method's value there is 0
        j = np.arange(w.D)[None, :]
        dead = ~((j < gpu["path_len"][:, None]) & (gpu["coeff"][:, None] != 0))
        gpu["grad"][dead] = 0.0
    return dict(w=w, draft=draft, draft_tag=dtag, target=target, target_tag=ttag, d2t=d2t,
                b0=first_position + gidx * w.m, gpu=gpu)


def _host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def cpu_baseline_and_parity(w, data, p, first_position, budget_s=25.0):
    """The oracle on every host core over whole groups drawn (seeded) from the benchmarked
    batch: one group per core, a second wave if the first took under half the budget.
    Returns (cpu_baseline, parity): the throughput of the oracle's pass, and the comparison
    of the library's outputs for the same groups."""
    from oracle.parallel import OracleWorkers
    cores = _host_cores()
    n_groups = w.B // w.m
    rng = np.random.default_rng(w.seed % (1 << 32))
    order = [0] + [int(x) for x in rng.permutation(np.arange(1, n_groups))]
    torch.set_num_threads(1)
    done, wall, cpu_s, reps = [], 0.0, 0.0, []
    with OracleWorkers(min(cores, n_groups)) as pool:
        for wave in range(2):
            groups = order[len(done):len(done) + pool.n]
            if not groups:
                break
            for i, gidx in enumerate(groups):
                pool.put(i, _group_payload(w, data, gidx, first_position, p))
            keys = list(range(len(groups)))
            _, dt, per = pool.call("bench", "oracle_group_task", keys, drop=False)
            wall += dt
            cpu_s += sum(per.values())
            res, _, _ = pool.call("bench", "oracle_check_task", keys)
            reps += [res[i] for i in keys]
            done += groups
            if wall > budget_s / 2:
                break
    n_pos = len(done) * w.m
    base = {"value": n_pos / wall, "unit": UNIT, "cores": min(cores, n_groups), "kind": "oracle",
            "per_core": n_pos / cpu_s,
            "sample": f"{n_pos} positions = {len(done)} whole groups of m={w.m} drawn over the batch "
                      f"(group 0 and a seeded permutation), one group per worker process, "
                      f"{wall:.1f} s wall, fp64 numpy, one thread per process, {cores} host cores"}
    parity = {"groups_checked": len(done), "positions_checked": n_pos, "groups": sorted(done),
              "failed_groups": sum(r.get("failed", 0) for r in reps),
              "near_tie_trees": sum(r.get("near_tie_trees", 0) for r in reps),
              "clip_edge": sum(r.get("clip_edge", 0) for r in reps),
              "ill_conditioned_groups": sum(r.get("ill_conditioned_groups", 0) for r in reps)}
    for key in ("max_lse_err", "max_score_err", "max_reward_rel", "max_adv_err", "max_grad_err"):
        parity[key] = max((r.get(key, 0.0) for r in reps), default=0.0)
    fails = [r["failure"] for r in reps if r.get("failed")]
    if fails:
        parity["first_failure"] = fails[0]
    return base, parity


def run_reference(args, w, rank, world):
    """The oracle as the reference arm, rank 0 only: every step runs one whole group of m
    positions of the workload on each host core (the same groups every step)."""
    if rank != 0:
        return
    from oracle.parallel import OracleWorkers
    from paper_2509_22134_b200 import synth
    device = "cuda:0" if torch.cuda.is_available() else "cpu"
    cores = _host_cores()
    n_workers = max(1, min(cores, w.B // w.m))
    data = synth.generate(w.with_B(n_workers * w.m), device)
    torch.set_num_threads(1)
    wall0 = time.perf_counter()
    with OracleWorkers(n_workers) as pool:
        for i in range(n_workers):
            pool.put(i, _group_payload(w, data, i, 0))
        keys = list(range(n_workers))
        del data
        times = []
        for i in range(args.warmup + args.steps):
            _, dt, _ = pool.call("bench", "oracle_group_task", keys, drop=False)
            if i >= args.warmup:
                times.append(dt)
            if times and time.perf_counter() - wall0 > REFERENCE_BUDGET_S:   # keep the run to a few minutes
                break
    done, dt = len(times), sum(times)
    value = done * n_workers * w.m / dt
    sample = (f"each step = {n_workers} whole groups of m={w.m} positions of the workload (groups "
              f"0..{n_workers - 1}, the same every step), one group per worker process, fp64 numpy, one "
              f"thread per process, {cores} host cores")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": done, "steps_requested": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * dt / max(done, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": n_workers, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(w, n_gpus):
    return {"workload": w.name, "positions_per_gpu": w.B, "global_positions": w.B * n_gpus,
            "V_draft": w.V_draft, "V_target": w.V_target, "D": w.D, "top_k": w.k, "g": w.g, "G": w.G,
            "m": w.m, "logits": w.dtype, "grad": "rows that carry a gradient only (GTO_FLAG_GRAD_LIVE_ROWS)",
            "parallelism": f"replicas x{n_gpus} (positions sharded, no collective)",
            "l2": "inputs (tens of GB) far exceed the 126 MB L2; no flush needed"}


# ---------------------------------------------------------------------------- GPU arm
def shard_first_position(rank: int, positions_per_rank: int) -> int:
    """Absolute index of a rank's first position: ranks own consecutive blocks of whole
    groups, so no group straddles two GPUs and no collective is needed on the data path."""
    return rank * positions_per_rank


def max_over_ranks(values, world: int, device):
    """Element-wise maximum of per-rank device timings (every rank gets the result)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(x) for x in t]


def algorithmic_bytes(w, p):
    """Bytes the method must move per step, from the data-dependent counts of this batch."""
    e = w.elem_bytes
    needed = int((~torch.isnan(p.reward["row_lse_t"])).sum().item())
    path_rows = int(p.reward["path_len"].sum().item())
    coeff_nz = p.stats["coeff"] != 0
    live_rows = int((p.reward["path_len"] * coeff_nz).sum().item())
    return {
        "draft_rows": w.G * w.B * w.R * w.V_draft * e,
        "target_rows": needed * w.V_target * e,
        # read and write of the rows that receive a gradient
        "grad_rows": 2 * live_rows * w.V_draft * e,
        "needed_target_rows": needed, "path_rows": path_rows, "live_grad_rows": live_rows,
    }


def timed_steps(p, data, n, stream, barrier, clocks=None):
    """n back-to-back steps bracketed by barrier + synchronize; returns (total ms, per-step ms,
    host time stamps of the region's start and end)."""
    ev0 = torch.cuda.Event(enable_timing=True)
    barrier()
    t0 = time.perf_counter()
    ev0.record(stream)
    marks = []
    for _ in range(n):
        p.step(data["draft"], data["target"], data["d2t"])
        marks.append(torch.cuda.Event(enable_timing=True))
        marks[-1].record(stream)
    barrier()
    t1 = time.perf_counter()
    per_step = [a.elapsed_time(b) for a, b in zip([ev0] + marks[:-1], marks)]
    return ev0.elapsed_time(marks[-1]), per_step, (t0, t1)


def by_clock(per_step, span, clocks, step_bytes):
    """Steps binned by the SM clock sampled while they ran (the device runs the queued steps
    back to back, so a sample's place between the region's host time stamps is its place in
    the step sequence).  Returns [{sm_mhz (bin centre), steps, ms_per_step, gbs}], fastest first."""
    if not clocks.samples:
        return []
    t0, t1 = span
    ends = np.cumsum(per_step) / max(sum(per_step), 1e-9)
    bins = {}
    for mhz, ts in zip(clocks.samples, clocks.stamps):
        if not (t0 <= ts <= t1):
            continue
        i = min(int(np.searchsorted(ends, (ts - t0) / (t1 - t0))), len(per_step) - 1)
        bins.setdefault(int(round(mhz / 50.0)) * 50, set()).add(i)
    out = []
    for mhz, steps in sorted(bins.items(), reverse=True):
        ms = statistics.mean(per_step[i] for i in steps)
        out.append({"sm_mhz": mhz, "steps": len(steps), "ms_per_step": ms,
                    "gbs": step_bytes / (ms * 1e-3) / 1e9})
    return out


def run_gpu(args, w, rank, world, local_rank):
    from paper_2509_22134_b200 import binding as gto
    from paper_2509_22134_b200 import synth
    from paper_2509_22134_b200.runner import GtoPass

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    b0 = shard_first_position(rank, w.B)
    data = synth.generate(w, dev, b0=b0)
    p = GtoPass(w, dev, flags=gto.GTO_FLAG_GRAD_LIVE_ROWS)
    p.grad.zero_()   # rows without a gradient are the caller's under GTO_FLAG_GRAD_LIVE_ROWS
    # the old-policy log-probabilities are an input of the gradient call: fix them once
    p.build_tree(data["draft"])
    p.tree_reward(data["target"], data["d2t"])
    p.set_old_logp_from_path(b0=b0)
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        p.step(data["draft"], data["target"], data["d2t"])
    assert p.status() == 0

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    stream = torch.cuda.current_stream(dev)
    # ---- (1) the headline region: K steps, the three calls and nothing else
    launches0 = p.launches()
    with ClockSampler(local_rank) as clocks:
        ms, per_step, _ = timed_steps(p, data, args.steps, stream, barrier)
    launches = p.launches() - launches0
    # ---- (2) the same with every launch bracketed by events: the per-kernel split.  The board
    #      idles for a moment first so that this region starts from the same power state as
    #      the first one (a few hundred ms of back-to-back steps already lower the clock).
    time.sleep(COOLDOWN_SECONDS)
    gto.gto_kernel_timing(p.ctx, True)
    for _ in range(3):
        p.step(data["draft"], data["target"], data["d2t"])
    gto.gto_kernel_times(p.ctx)
    with ClockSampler(local_rank) as split_clocks:
        ms_events, _, _ = timed_steps(p, data, args.steps, stream, barrier)
    ktimes = gto.gto_kernel_times(p.ctx)
    gto.gto_kernel_timing(p.ctx, False)
    # ---- (3) sustained: at least SUSTAINED_SECONDS of back-to-back steps, clocks sampled
    sustained = None
    if not args.no_sustained:
        n_sus = max(args.steps, int(math.ceil(SUSTAINED_SECONDS * 1e3 / (ms / args.steps))))
        with ClockSampler(local_rank) as sus_clocks:
            sus_ms, sus_steps, sus_span = timed_steps(p, data, n_sus, stream, barrier)
        sustained = (n_sus, sus_ms, sus_steps, sus_span, sus_clocks)
    assert p.status() == 0

    # ---- next-row kernel, timed on its own (not part of the step): token-level loss
    extras = {}
    if not args.no_extras:
        for _ in range(3):
            p.token_loss(data["draft"], data["target"], data["d2t"], 1.0 / w.B)
        t_ev0, t_ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        t_ev0.record(stream)
        for _ in range(args.steps):
            p.token_loss(data["draft"], data["target"], data["d2t"], 1.0 / w.B)
        t_ev1.record(stream)
        torch.cuda.synchronize(dev)
        tot, cnt = t_ev0.elapsed_time(t_ev1), args.steps
        tok_bytes = w.B * 3 * w.V_draft * w.elem_bytes   # draft row, mapped target logits, gradient row
        # what has to cross the memory bus: the mapped ids are spread over the whole target row
        tok_streamed = w.B * (2 * w.V_draft + w.V_target) * w.elem_bytes
        extras["token_loss"] = {"ms": tot / cnt, "algorithmic_bytes": tok_bytes,
                                "gbs": tok_bytes / (tot / cnt * 1e-3) / 1e9,
                                "streamed_bytes": tok_streamed,
                                "streamed_gbs": tok_streamed / (tot / cnt * 1e-3) / 1e9,
                                "note": "Eq. 13 on the B root rows, timed alone (not part of the step): "
                                        "back-to-back calls between two events (one launch per call), so the "
                                        "figure includes any host-side gap"}

    # ---- (4) end to end: host buffers, copies inside the timed region
    e2e = run_e2e(args, w, dev, b0, world) if not args.no_e2e else None
    if e2e is None:
        e2e = {"ms": float("nan"), "positions": 0, "h2d": 0, "d2h": 0, "positions_per_step": 0, "steps": 0,
               "pinned_h2d_gbs": None}

    sus_ms_all = sustained[1] if sustained else float("nan")
    ms, ms_events, e2e_ms, sus_ms_all = max_over_ranks([ms, ms_events, e2e["ms"], sus_ms_all], world, dev)
    if rank != 0:
        return

    alg = algorithmic_bytes(w, p)
    peak, peak_kind = measured_peak()
    kern = {}
    for name, (tot, cnt) in ktimes.items():
        if cnt:
            kern[name] = {"ms": tot / cnt, "launches_per_step": cnt / args.steps}
            if name in alg:
                kern[name]["gbs"] = alg[name] / (tot / cnt * 1e-3) / 1e9
    top = max((n for n in kern if n in alg), key=lambda n: kern[n]["ms"] * kern[n]["launches_per_step"])
    traffic = None
    if top in NCU_TRAFFIC:
        src, sha, per_row, v_cap = NCU_TRAFFIC[top]
        if _sha256(os.path.join(ROOT, src)) == sha:
            rows = {"draft_rows": w.G * w.B * w.R, "target_rows": alg["needed_target_rows"]}[top]
            v_now = {"draft_rows": w.V_draft, "target_rows": w.V_target}[top]
            traffic = per_row * rows * v_now / v_cap
    step_bytes = alg["draft_rows"] + alg["target_rows"] + alg["grad_rows"]
    step_s = ms * 1e-3 / args.steps
    roofline = {"bound": "hbm", "kernel": top, "achieved": kern[top]["gbs"], "peak": peak,
                "unit": "GB/s", "frac": kern[top]["gbs"] / peak, "peak_kind": f"of {peak_kind}",
                "traffic": traffic,
                "algorithmic_bytes_per_launch": alg[top],
                "timed_in": f"a second region of {args.steps} steps with every launch bracketed by CUDA "
                            f"events ({ms_events / args.steps:.4f} ms per step there), after "
                            f"{COOLDOWN_SECONDS} s of idling",
                "clocks": split_clocks.summary(),
                "pass": {"algorithmic_bytes_per_step": step_bytes,
                         "achieved": step_bytes / step_s / 1e9,
                         "frac": step_bytes / step_s / 1e9 / peak,
                         "frac_of_8000_nominal": step_bytes / step_s / 1e9 / 8000.0},
                "kernels": kern,
                "counts": {k: alg[k] for k in ("needed_target_rows", "path_rows", "live_grad_rows")}}
    line = {"metric": METRIC, "value": world * w.B * args.steps / (ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms / args.steps, "ms_per_step_median": statistics.median(per_step),
            "ms_per_step_min": min(per_step), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "storage_dtype": w.dtype, "data": "synthetic",
            "config": workload_config(w, world),
            "clocks": clocks.summary(),
            "e2e": {"value": world * e2e["positions"] / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                    "positions_per_step": e2e["positions_per_step"], "steps": e2e["steps"],
                    "pinned_h2d_gbs": e2e["pinned_h2d_gbs"]},
            "gpu_launches": launches,
            "roofline": roofline,
            "extras": extras}
    if sustained:
        n_sus, _, sus_steps, sus_span, sus_clocks = sustained
        sus_s = sus_ms_all * 1e-3 / n_sus
        cs = sus_clocks.summary()
        line["sustained"] = {"steps": n_sus, "seconds": sus_ms_all * 1e-3, "ms_per_step": sus_ms_all / n_sus,
                             "value": world * w.B / sus_s, "gbs": step_bytes / sus_s / 1e9,
                             "frac_of_measured": step_bytes / sus_s / 1e9 / peak,
                             "frac_of_8000_nominal": step_bytes / sus_s / 1e9 / 8000.0,
                             "sm_mhz_median": cs["sm_mhz"], "mem_mhz_median": cs["mem_mhz"],
                             "power_w_median": cs["power_w"], "reasons": cs["reasons"],
                             "by_clock": by_clock(sus_steps, sus_span, sus_clocks, step_bytes)}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"], line["parity"] = cpu_baseline_and_parity(w, data, p, b0)
    print(json.dumps(line), flush=True)


def run_e2e(args, w, dev, b0, world):
    """The same pass through the C ABI with the logits in pinned HOST memory: every step
    copies its positions' draft rows and the old-policy log-probabilities to the device,
    builds the trees, copies the target rows the trees need (gto_tree_reward_host), and
    reads the losses, rewards, advantages and accepted paths back.  The gradient stays on the device, where the
    draft model's backward pass consumes it."""
    from paper_2509_22134_b200 import synth
    from paper_2509_22134_b200.runner import GtoPass
    we = w.with_B(min(w.B, E2E_POSITIONS))
    data = synth.generate(we, dev, b0=b0)
    host = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v)
            for k, v in data.items() if k in ("draft", "target")}
    from paper_2509_22134_b200 import binding as gto
    p = GtoPass(we, dev, flags=gto.GTO_FLAG_GRAD_LIVE_ROWS)
    p.build_tree(data["draft"])
    p.tree_reward(data["target"], data["d2t"])
    p.set_old_logp_from_path(b0=b0)
    old_host = torch.empty(p.old_logp.shape, dtype=torch.float32, pin_memory=True).copy_(p.old_logp)
    back = {"loss": p.stats["loss"], "adv": p.stats["adv"], "ratio": p.stats["ratio"],
            "reward": p.reward["reward"], "path_len": p.reward["path_len"],
            "path_row": p.reward["path_row"], "path_token": p.reward["path_token"]}
    back_host = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in back.items()}
    h2d_fixed = host["draft"].numel() * host["draft"].element_size() + old_host.numel() * 4
    row_bytes = we.V_target * we.elem_bytes
    d2h = sum(t.numel() * t.element_size() for t in back.values())

    rows = [0]

    def step():
        data["draft"].copy_(host["draft"], non_blocking=True)
        p.old_logp.copy_(old_host, non_blocking=True)
        p.build_tree(data["draft"])
        # only the target rows the trees need cross the bus (gto_tree_reward_host)
        rows[0] = p.tree_reward_host(host["target"], data["target"], data["d2t"])
        p.surrogate_grad(data["draft"])
        for k, v in back.items():
            back_host[k].copy_(v, non_blocking=True)
        torch.cuda.current_stream(dev).synchronize()       # the caller reads the results

    steps = max(3, min(args.steps, 10))
    for _ in range(3):
        step()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the bus itself: one plain copy of the pinned draft buffer, for a ceiling beside the figure
    torch.cuda.synchronize(dev)
    ev0.record()
    data["draft"].copy_(host["draft"], non_blocking=True)
    ev1.record()
    torch.cuda.synchronize(dev)
    pinned_gbs = host["draft"].numel() * host["draft"].element_size() / (ev0.elapsed_time(ev1) * 1e-3) / 1e9
    if world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize(dev)
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    torch.cuda.synchronize(dev)
    ms = ev0.elapsed_time(ev1)
    p.close()
    del data, host
    torch.cuda.empty_cache()
    h2d = h2d_fixed + rows[0] * row_bytes   # + the row list read back (counted in d2h)
    d2h += 4 * (we.G * we.B * we.R + 1)
    return {"ms": ms, "positions": we.B * steps, "h2d": h2d, "d2h": d2h,
            "positions_per_step": we.B, "steps": steps, "pinned_h2d_gbs": pinned_gbs}


def spawn_ranks(n: int) -> int:
    """Started without a launcher: run this same command line as n ranks on this node (one per
    GPU, rank r on GPU r) under torch.distributed.run, and return its exit code."""
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="gto", choices=["gto", "reference"])
    ap.add_argument("--workload", type=int, default=2, help="index into the synthetic workloads")
    ap.add_argument("--positions", type=int, default=None, help="override B (a multiple of m)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the back-to-back region (profiling runs)")
    ap.add_argument("--no-extras", action="store_true", help="skip the token-loss timing (profiling runs)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 3 if args.impl == "reference" else 50
    if args.warmup is None:
        args.warmup = 1 if args.impl == "reference" else 5

    from paper_2509_22134_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.positions:
        w = w.with_B(args.positions)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, w, rank, world)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if not torch.cuda.is_available():
        raise SystemExit(f"bench.py: no CUDA device on rank {rank} (the GTO pass has no CPU path)")
    if torch.cuda.device_count() <= local_rank:
        raise SystemExit(f"bench.py: rank {rank} wants GPU {local_rank}, the node has {torch.cuda.device_count()}")
    if world > 1:
        torch.cuda.set_device(local_rank)
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_gpu(args, w, rank, world, local_rank)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
