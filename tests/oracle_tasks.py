"""Tasks the oracle worker processes run for the GPU parity tests: one call checks whole
groups of one workload against the library's outputs for the same positions."""
from __future__ import annotations

import numpy as np

from oracle import check as ocheck
from oracle import parallel as opar
from paper_2509_22134_b200 import synth


class Cfg:
    pass


def make_cfg(w: synth.Workload, extra=None):
    cfg = Cfg()
    for name in ("B", "G", "D", "k", "g", "m", "eta", "clip_eps", "std_delta", "grad_scale"):
        setattr(cfg, name, getattr(w, name))
    for key, val in (extra or {}).items():
        setattr(cfg, key, val)
    return cfg


def old_logp_fn(w: synth.Workload):
    """The old-policy log-probabilities of the accepted paths, as the harness defines them
    (an input of the method): the path's own values plus the seeded perturbation."""
    def fn(path_logp, path_row, path_token, path_len, positions):
        out = np.zeros_like(path_logp)
        for j, b in enumerate(positions):
            out[j] = synth.old_logp_from_path(w, path_logp[j:j + 1], path_row[j:j + 1],
                                              path_token[j:j + 1], path_len[j:j + 1], b0=b)[0]
        return out
    return fn


def check_groups(w, cfg_extra, draft, draft_tag, target, target_tag, d2t, gpu, positions):
    """oracle.check.check_positions on the given positions (whole groups)."""
    return ocheck.check_positions(make_cfg(w, cfg_extra), opar.decode_logits(draft, draft_tag),
                                  opar.decode_logits(target, target_tag), d2t, gpu, old_logp_fn(w),
                                  positions)


def merge_reports(reps):
    out = {}
    for rep in reps:
        for key, val in rep.items():
            if key.startswith("max_"):
                out[key] = max(out.get(key, 0.0), val)
            elif key.startswith("mean_"):
                out[key] = out.get(key, 0.0) + val * rep["positions"]
            else:
                out[key] = out.get(key, 0) + val
    for key in out:
        if key.startswith("mean_"):
            out[key] /= max(out["positions"], 1)
    return out
