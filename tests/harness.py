"""Runs the CUDA library on a synthetic workload and checks it against the oracle.

Shared by the GPU parity tests and the smoke check.  The only place where the product
package and the oracle meet.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle_tasks
from oracle import parallel as opar
from paper_2509_22134_b200 import synth
from paper_2509_22134_b200.runner import GtoPass


def gather_outputs(p: GtoPass, pos):
    """Library outputs restricted to the positions `pos`, as numpy arrays."""
    idx = torch.as_tensor(pos, device=p.device, dtype=torch.long)
    out = {}
    for name, t in p.tree.items():
        out[name] = t.index_select(1, idx).cpu().numpy()
    for name, t in p.reward.items():
        dim = 0 if name.startswith("path_") else 1
        out[name] = t.index_select(dim, idx).cpu().numpy()
    for name, t in p.stats.items():
        if name == "loss":
            groups = sorted(set(int(b) // p.w.m for b in pos))
            out[name] = t[torch.as_tensor(groups, device=p.device)].cpu().numpy()
        else:
            out[name] = t.index_select(0, idx).cpu().numpy()
    out["grad"] = p.grad.index_select(0, idx).float().cpu().numpy().astype(np.float64)
    return out


def run_pass(w: synth.Workload, device="cuda:0", data=None, **kw):
    if data is None:
        data = synth.generate(w, device)
    p = GtoPass(w, device, **kw)
    if kw.get("flags", 0) & 4:      # GTO_FLAG_GRAD_LIVE_ROWS: the other rows are the caller's
        p.grad.zero_()
    p.build_tree(data["draft"])
    p.tree_reward(data["target"], data["d2t"])
    p.set_old_logp_from_path()
    p.surrogate_grad(data["draft"])
    assert p.status() == 0, "device status word set"
    return p, data


def check_against_oracle(w: synth.Workload, p: GtoPass, data, groups, cfg_extra=None, workers=None):
    """Oracle comparison on the listed groups (each m consecutive positions).  With `workers`
    (an oracle.parallel.OracleWorkers) every group is checked on its own host core."""
    d2t = None if data["d2t"] is None else data["d2t"].cpu().numpy().astype(np.int64)

    def payload(gs):
        pos = [gidx * w.m + i for gidx in gs for i in range(w.m)]
        idx = torch.as_tensor(pos, device=p.device, dtype=torch.long)
        draft, dtag = opar.encode_logits(data["draft"].index_select(1, idx))
        target, ttag = opar.encode_logits(data["target"].index_select(1, idx))
        return dict(w=w, cfg_extra=cfg_extra, draft=draft, draft_tag=dtag, target=target,
                    target_tag=ttag, d2t=d2t, gpu=gather_outputs(p, pos), positions=pos)

    if workers is None or len(groups) == 1:
        return oracle_tasks.check_groups(**payload(list(groups)))
    reps, _ = workers.run("oracle_tasks", "check_groups", [payload([gidx]) for gidx in groups])
    return oracle_tasks.merge_reports(reps)
