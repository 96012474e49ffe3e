"""Benchmark of the GTO draft-tree pass (build tree -> Draft Tree Reward -> group surrogate
gradient) on synthetic logits at the LLaMA-3.1-8B shape.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload ID]

One step = one pass of the whole hot path over the batch of B positions resident in HBM.
With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs the same
number of its own positions (weak scaling); positions are independent, so no collective is
on the data path - only the timing barrier and the max-over-ranks reduction.

Prints ONE JSON line on rank 0.  `--impl reference` times the fp64 CPU oracle instead (on a
bounded sample per step), on rank 0 only.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
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

# DRAM traffic per processed row of the dominant kernels, from one ncu capture each
# (dram__bytes_read.sum + dram__bytes_write.sum over the launch / rows in the launch).  An
# entry is used only while the kernel source it was taken from is unchanged.
NCU_TRAFFIC = {
    # kernel: (source file, sha256 of that file at capture time, bytes per row, V of the capture)
    # from the ncu capture summarised under profiles/ (row pass, workload 2 shapes at B = 64)
    "draft_rows": ("paper_2509_22134_b200/csrc/row_reduce.cu",
                   "9b80b0d584d978fb10de3ec7706c5b4e528dccfda59000aa34ca2ccb52ccf1a2", (510916864 + 4050432) / 7808, 32000),
    "target_rows": ("paper_2509_22134_b200/csrc/row_reduce.cu",
                    "9b80b0d584d978fb10de3ec7706c5b4e528dccfda59000aa34ca2ccb52ccf1a2", (429946368 + 3444480) / 1673, 128256),
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
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
                mask = int(get_reasons(self._h))
                for bit, name in self._REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
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
                "samples": len(self.samples)}


# ------------------------------------------------------------------------ oracle legs
def _oracle_group_fn(w):
    """Returns f(draft_g, target_g, d2t, b0) running the oracle's whole pass on one group."""
    from oracle import gto_oracle as orc
    from paper_2509_22134_b200 import synth

    def run(draft_g, target_g, d2t, b0):
        def old_fn(path_logp, path_row, path_token, path_len):
            out = np.zeros_like(path_logp)
            for i in range(path_logp.shape[0]):
                out[i] = synth.old_logp_from_path(w, path_logp[i:i + 1], path_row[i:i + 1],
                                                  path_token[i:i + 1], path_len[i:i + 1], b0=b0 + i)[0]
            return out
        return orc.group_pass(draft_g, target_g, w.D, w.k, w.g, w.m, old_fn, d2t, w.eta,
                              delta=w.std_delta, eps=w.clip_eps, grad_scale=w.grad_scale)
    return run


def _sample_groups(w, n_groups, device):
    """Synthetic logits of the first n_groups groups, as host fp32 arrays (exact values)."""
    from paper_2509_22134_b200 import synth
    data = synth.generate(w.with_B(n_groups * w.m), device)
    draft = data["draft"].float().cpu().numpy()
    target = data["target"].float().cpu().numpy()
    d2t = None if data["d2t"] is None else data["d2t"].cpu().numpy().astype(np.int64)
    return draft, target, d2t


def cpu_baseline(w, device, budget_s=12.0, max_groups=4):
    """Oracle throughput on whole groups of the workload until ~budget_s of CPU work."""
    run = _oracle_group_fn(w)
    draft, target, d2t = _sample_groups(w, max_groups, device)
    torch.set_num_threads(1)
    done, t0 = 0, time.perf_counter()
    for gidx in range(max_groups):
        sl = slice(gidx * w.m, (gidx + 1) * w.m)
        run(draft[:, sl], target[:, sl], d2t, gidx * w.m)
        done += w.m
        if time.perf_counter() - t0 >= budget_s:
            break
    dt = time.perf_counter() - t0
    return {"value": done / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"first {done} positions ({done // w.m} groups of m={w.m}) of the workload, "
                      f"{dt:.1f} s, fp64 numpy, one host thread of {os.cpu_count()}"}


def run_reference(args, w, rank, world):
    """The oracle as the reference arm: one group of m positions per step, rank 0 only."""
    if rank != 0:
        return
    device = "cuda:0" if torch.cuda.is_available() else "cpu"
    run = _oracle_group_fn(w)
    n_groups = 2
    draft, target, d2t = _sample_groups(w, n_groups, device)
    torch.set_num_threads(1)

    def step(i):
        gidx = i % n_groups
        sl = slice(gidx * w.m, (gidx + 1) * w.m)
        run(draft[:, sl], target[:, sl], d2t, gidx * w.m)

    wall0 = time.perf_counter()
    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    done = 0
    for i in range(args.steps):
        step(i)
        done += 1
        if time.perf_counter() - wall0 > REFERENCE_BUDGET_S:   # keep the run to a few minutes
            break
    dt = time.perf_counter() - t0
    value = done * w.m / dt
    sample = (f"each step = one group of m={w.m} positions of the workload (groups 0..{n_groups - 1} "
              f"in turn), fp64 numpy, one host thread of {os.cpu_count()}")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": done, "steps_requested": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * dt / max(done, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
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


def run_gpu(args, w, rank, world, local_rank):
    from paper_2509_22134_b200 import binding as gto
    from paper_2509_22134_b200 import synth
    from paper_2509_22134_b200.runner import GtoPass

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    b0 = shard_first_position(rank, w.B)
    data = synth.generate(w, dev, b0=b0)
    p = GtoPass(w, dev, flags=gto.GTO_FLAG_GRAD_LIVE_ROWS)
    # the old-policy log-probabilities are an input of the gradient call: fix them once
    p.build_tree(data["draft"])
    p.tree_reward(data["target"], data["d2t"])
    p.set_old_logp_from_path(b0=b0)
    for _ in range(max(args.warmup, 3)):
        p.step(data["draft"], data["target"], data["d2t"])
    assert p.status() == 0

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    stream = torch.cuda.current_stream(dev)
    ev0 = torch.cuda.Event(enable_timing=True)
    gto.gto_kernel_timing(p.ctx, True)
    launches0 = p.launches()
    with ClockSampler(local_rank) as clocks:
        barrier()
        ev0.record(stream)
        marks = []
        for _ in range(args.steps):
            p.step(data["draft"], data["target"], data["d2t"])
            marks.append(torch.cuda.Event(enable_timing=True))
            marks[-1].record(stream)
        ev1 = marks[-1]
        barrier()
    ms = ev0.elapsed_time(ev1)
    per_step = [a.elapsed_time(b) for a, b in zip([ev0] + marks[:-1], marks)]
    ktimes = gto.gto_kernel_times(p.ctx)
    gto.gto_kernel_timing(p.ctx, False)
    launches = p.launches() - launches0
    assert p.status() == 0

    # ---- next-row kernel, timed on its own (not part of the step): token-level loss
    extras = {}
    if not args.no_e2e:
        gto.gto_kernel_timing(p.ctx, True)
        for _ in range(3):
            p.token_loss(data["draft"], data["target"], data["d2t"], 1.0 / w.B)
        gto.gto_kernel_times(p.ctx)
        for _ in range(args.steps):
            p.token_loss(data["draft"], data["target"], data["d2t"], 1.0 / w.B)
        tot, cnt = gto.gto_kernel_times(p.ctx)["token_loss"]
        gto.gto_kernel_timing(p.ctx, False)
        tok_bytes = w.B * 3 * w.V_draft * w.elem_bytes   # draft row, mapped target logits, gradient row
        extras["token_loss"] = {"ms": tot / cnt, "algorithmic_bytes": tok_bytes,
                                "gbs": tok_bytes / (tot / cnt * 1e-3) / 1e9,
                                "note": "Eq. 13 on the B root rows; the id-map gather touches "
                                        "nearly every 32-byte sector of the target row"}

    # ---- end to end: host buffers, copies inside the timed region
    e2e = run_e2e(args, w, dev, b0, world) if not args.no_e2e else None
    if e2e is None:
        e2e = {"ms": float("nan"), "positions": 0, "h2d": 0, "d2h": 0, "positions_per_step": 0, "steps": 0}

    ms, e2e_ms = max_over_ranks([ms, e2e["ms"]], world, dev)
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
                "pass": {"algorithmic_bytes_per_step": step_bytes,
                         "achieved": step_bytes / step_s / 1e9,
                         "frac": step_bytes / step_s / 1e9 / peak,
                         "frac_of_8000_nominal": step_bytes / step_s / 1e9 / 8000.0},
                "kernels": kern,
                "counts": {k: alg[k] for k in ("needed_target_rows", "path_rows", "live_grad_rows")}}
    line = {"metric": METRIC, "value": world * w.B * args.steps / (ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms / args.steps, "ms_per_step_median": statistics.median(per_step),
            "ms_per_step_min": min(per_step), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(w, world),
            "clocks": clocks.summary(),
            "e2e": {"value": world * e2e["positions"] / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                    "positions_per_step": e2e["positions_per_step"], "steps": e2e["steps"]},
            "gpu_launches": launches,
            "roofline": roofline,
            "extras": extras}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, dev)
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
            "positions_per_step": we.B, "steps": steps}


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
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the GTO pass has no CPU path)")
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
