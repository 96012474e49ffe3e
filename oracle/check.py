"""Element-by-element comparison of the CUDA library's outputs with the oracle
(test infrastructure only).  Receives plain numpy arrays; imports nothing of the
product path.

Tolerances: integer structure bit-exact; a structural mismatch is excused only when
the oracle's own ranking of that tree has a decision whose competing scores lie within
1e-6 (counted and reported); rewards and advantages 1e-4 relative; gradients 2e-3
absolute.
"""
from __future__ import annotations

import numpy as np

from . import gto_oracle as orc

TIE_TOL = 1e-6
REL_TOL = 1e-4
GRAD_ATOL = 2e-3
LSE_ATOL = 2e-6
CLIP_EDGE_TOL = 1e-6


def _close(a, b, rtol=REL_TOL, atol=0.0):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return np.all(np.abs(a - b) <= atol + rtol * np.maximum(1.0, np.abs(b)))


def check_positions(cfg, draft, target, d2t, gpu, old_logp_fn, positions):
    """Compare the library with the oracle on `positions` (whole groups).

    cfg: object with B, G, D, k, g, m, eta, clip_eps, std_delta, grad_scale (+ optional
    agg, unbiased, debias).  draft: [G, n, D, k, V_d], target: [G, n, R, V_t] (any float
    dtype holding the stored logits exactly) for the n listed positions, d2t: int array or None.  gpu: dict of numpy
    arrays of the library's outputs restricted to the same positions (leading G where the
    library has it), grad [n, D, V_d] float64, loss [n/m].
    old_logp_fn(path_logp[n,D], path_row, path_token, path_len, positions) -> [n, D].
    Returns a report dict; raises AssertionError on any mismatch outside the tolerances.
    """
    G, D, k, g, m = cfg.G, cfg.D, cfg.k, cfg.g, cfg.m
    n = len(positions)
    assert n % m == 0
    agg = getattr(cfg, "agg", orc.AGG_LSE)
    rep = dict(positions=n, trees=G * n, near_tie_trees=0, clip_edge=0, ill_conditioned_groups=0,
               max_lse_err=0.0, max_reward_rel=0.0, max_adv_err=0.0, max_grad_err=0.0,
               mean_path_len=0.0, mean_needed_rows=0.0)
    fwd = []
    excused = np.zeros(n, dtype=bool)
    for i in range(n):
        d_i = np.asarray(draft[:, i], dtype=np.float64)
        t_i = np.asarray(target[:, i], dtype=np.float64)
        f = orc.position_forward(d_i, t_i, D, k, g, d2t, cfg.eta, agg, getattr(cfg, "all_nodes", False))
        fwd.append(f)
        for t in range(G):
            tr = f["trees"][t]
            same = all(np.array_equal(gpu[name][t, i], getattr(tr, attr)) for name, attr in
                       [("node_token", "token"), ("node_parent", "parent"), ("node_depth", "depth"),
                        ("node_ctx_row", "ctx_row"), ("node_slot", "slot"), ("node_pool", "pool")])
            if not same:
                gap = min(tr.cut_gaps)
                assert gap < TIE_TOL, (f"tree structure mismatch at position {positions[i]} tree {t} "
                                       f"with smallest decision gap {gap}")
                rep["near_tie_trees"] += 1
                excused[i] = True
                continue
            # ancestor mask
            W = gpu["node_mask"].shape[-1]
            bits = np.zeros((g, g), dtype=bool)
            for a_ in range(g):
                bits[:, a_] = (gpu["node_mask"][t, i, :, a_ // 64].astype(np.uint64) >> np.uint64(a_ % 64)) & np.uint64(1)
            assert np.array_equal(bits, tr.mask), f"mask mismatch at {positions[i]} tree {t}"
            err = np.max(np.abs(gpu["row_lse"][t, i] - tr.row_lse))
            rep["max_lse_err"] = max(rep["max_lse_err"], float(err))
            assert err <= LSE_ATOL, f"draft lse error {err} at {positions[i]}"
            assert _close(gpu["node_logp"][t, i], tr.logp, rtol=0, atol=1e-5)
            assert _close(gpu["node_score"][t, i], tr.score, rtol=0, atol=1e-5)
            rw = f["rewards"][t]
            used = ~np.isnan(rw["row_lse_t"])
            assert np.array_equal(np.isnan(gpu["row_lse_t"][t, i]), ~used)
            assert np.all(gpu["row_argmax_t"][t, i][~used] == -1)
            err = np.max(np.abs(gpu["row_lse_t"][t, i][used] - rw["row_lse_t"][used]))
            rep["max_lse_err"] = max(rep["max_lse_err"], float(err))
            assert err <= LSE_ATOL, f"target lse error {err} at {positions[i]}"
            want_am = [orc.argmax_low(t_i[t, r]) for r in np.flatnonzero(used)]
            assert np.array_equal(gpu["row_argmax_t"][t, i][used], want_am)
            rep["mean_needed_rows"] += used.sum() / (G * n)
            assert _close(gpu["node_ptarget"][t, i], rw["p"], rtol=REL_TOL, atol=1e-12)
            assert _close(gpu["node_pathprod"][t, i], rw["Pp"], rtol=REL_TOL, atol=1e-12)
            assert _close(gpu["node_L"][t, i], rw["Lc"])
            rel = abs(gpu["reward"][t, i] - rw["r"]) / max(1.0, abs(rw["r"]))
            rep["max_reward_rel"] = max(rep["max_reward_rel"], float(rel))
            assert rel <= REL_TOL, f"reward {gpu['reward'][t, i]} vs {rw['r']}"
            assert _close(gpu["etree"][t, i], rw["etree"])
            assert gpu["n_leaves"][t, i] == len(rw["leaves"])
        if excused[i]:
            continue
        path = f["path"]
        l = len(path["nodes"])
        rep["mean_path_len"] += l / n
        assert gpu["path_len"][i] == l, f"path length {gpu['path_len'][i]} vs {l} at {positions[i]}"
        assert list(gpu["path_node"][i][:l]) == path["nodes"]
        assert list(gpu["path_row"][i][:l]) == path["rows"]
        assert list(gpu["path_token"][i][:l]) == path["tokens"]
        assert np.all(gpu["path_node"][i][l:] == -1)
        assert _close(gpu["path_logp"][i][:l], path["logp"], rtol=0, atol=1e-5)

    # ---- groups: Eq. 9-12 and the gradient
    for g0 in range(0, n, m):
        idx = list(range(g0, g0 + m))
        if excused[idx].any():
            continue
        r_cur = np.array([fwd[i]["rewards"][0]["r"] for i in idx])
        r_ref = np.array([fwd[i]["rewards"][1]["r"] for i in idx])
        R, A = orc.group_advantages(r_cur, r_ref, m, cfg.std_delta,
                                    unbiased=getattr(cfg, "unbiased", False),
                                    debias=getattr(cfg, "debias", True))
        if np.std(R) < 1e-4:
            rep["ill_conditioned_groups"] += 1
            continue
        path_len = np.array([len(fwd[i]["path"]["nodes"]) for i in idx])
        path_logp = np.zeros((m, D))
        path_row = np.full((m, D), -1, dtype=np.int64)
        path_tok = np.full((m, D), -1, dtype=np.int64)
        for j, i in enumerate(idx):
            l = path_len[j]
            path_logp[j, :l] = fwd[i]["path"]["logp"]
            path_row[j, :l] = fwd[i]["path"]["rows"]
            path_tok[j, :l] = fwd[i]["path"]["tokens"]
        old = old_logp_fn(path_logp, path_row, path_tok, path_len, [positions[i] for i in idx])
        sur = orc.clipped_surrogate(path_logp, old, path_len, A, m, cfg.clip_eps, cfg.grad_scale)
        assert _close(gpu["R"][idx], R, rtol=REL_TOL)
        adv_err = np.max(np.abs(gpu["adv"][idx] - A) / np.maximum(1.0, np.abs(A)))
        rep["max_adv_err"] = max(rep["max_adv_err"], float(adv_err))
        assert adv_err <= REL_TOL, f"advantage error {adv_err}"
        assert _close(gpu["ratio"][idx], sur["ratio"])
        edge = np.minimum(np.abs(sur["ratio"] - (1 + cfg.clip_eps)),
                          np.abs(sur["ratio"] - (1 - cfg.clip_eps))) < CLIP_EDGE_TOL
        rep["clip_edge"] += int(edge.sum())
        if edge.any():
            continue
        assert np.array_equal(gpu["active"][idx].astype(bool), sur["active"])
        assert _close(gpu["coeff"][idx], sur["coeff"], rtol=REL_TOL, atol=1e-9)
        assert _close(gpu["loss"][g0 // m], sur["loss"][0], rtol=REL_TOL, atol=1e-9)
        for j, i in enumerate(idx):
            l = path_len[j]
            d_i = np.asarray(draft[0, i], dtype=np.float64)
            rows = [d_i[orc.draft_slot_of_row(int(r), k)] for r in path_row[j, :l]]
            lse = [fwd[i]["trees"][0].row_lse[r] for r in path_row[j, :l]]
            want = orc.surrogate_grad_rows(rows, lse, list(path_tok[j, :l]), sur["coeff"][j], D,
                                           draft.shape[-1])
            err = float(np.max(np.abs(gpu["grad"][i] - want)))
            rep["max_grad_err"] = max(rep["max_grad_err"], err)
            assert err <= GRAD_ATOL, f"gradient error {err} at position {positions[i]}"
    return rep
