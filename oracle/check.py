"""Element-by-element comparison of the CUDA library's outputs with the oracle
(test infrastructure only).  Receives plain numpy arrays; imports nothing of the
product path.

Tolerances: integer structure bit-exact; a structural mismatch is excused only when the
ranking decision that was resolved differently (a layer's frontier ranking, or the top-g
cut) has competing oracle scores within 1e-6 (counted and reported); rewards, target
probabilities and path products 1e-4 relative; advantages 1e-4 of max(1, |A|) (they amplify
a reward error by 1 / std(R), so groups with std(R) < 1e-4 are reported as ill-conditioned
and skipped); gradients 2e-3 absolute.
"""
from __future__ import annotations

import numpy as np

from . import gto_oracle as orc

TIE_TOL = 1e-6
REL_TOL = 1e-4
GRAD_ATOL = 2e-3
LSE_ATOL = 2e-6
CLIP_EDGE_TOL = 1e-6


SCORE_ATOL = 0.5 * TIE_TOL   # scores this close to the oracle's keep every decision whose gap is >= TIE_TOL


def _close(a, b, rtol=REL_TOL, atol=0.0):
    """|a - b| <= atol + rtol |b|, element by element (a true relative bound)."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return np.all(np.abs(a - b) <= atol + rtol * np.abs(b))


def _exchange_gap(tr, their_pool):
    """Largest oracle score gap between a candidate only the oracle selected and one only the
    other side selected.  inf where the index decides on every implementation: the same
    parent and the same logit, or a candidate against its own descendant."""
    ours, theirs = set(int(p) for p in tr.pool), set(int(p) for p in their_pool)
    worst = 0.0
    for a in ours - theirs:
        for b in theirs - ours:
            if b < 0 or b >= len(tr.cand_score):
                return np.inf
            gap = float(tr.cand_score[a] - tr.cand_score[b])
            if gap == 0.0 and tr.cand_parent[a] == tr.cand_parent[b]:
                return np.inf
            up = int(tr.cand_parent[b])
            while up >= 0:
                if up == a:
                    return np.inf
                up = int(tr.cand_parent[up])
            worst = max(worst, abs(gap))
    return worst if (ours - theirs) and (theirs - ours) else np.inf


def differing_decisions(tr, got):
    """Which ranking decisions of the oracle's tree `tr` the other side resolved differently,
    with the oracle's score gap at each.  got: dict of the other side's node lists (pool, slot,
    token, depth).  Looks at the shallowest depth whose selected nodes differ (deeper
    differences follow from it): a node that is selected on one side only is the top-g cut,
    and the gap reported is the largest one between a candidate only the oracle kept and one
    only the other side kept (the candidates that were actually exchanged: the oracle's own
    neighbour across the cut can be a sibling with the same logit, which nobody confuses);
    a node selected on both sides with another frontier slot is that layer's ranking, and
    the gap reported is the largest one any moved candidate crossed (between its rank on
    the two sides; two separate exchanges in one layer do not span what lies between them).
    Returns a list of (decision name, gap); empty if no ranking decision explains the
    difference (then it is a plain error)."""
    k = tr.k
    out = []
    for d in range(1, tr.D + 1):
        mine = {int(p): (int(s), int(t)) for p, s, t, dd in zip(tr.pool, tr.slot, tr.token, tr.depth) if dd == d}
        theirs = {int(p): (int(s), int(t)) for p, s, t, dd in
                  zip(got["pool"], got["slot"], got["token"], got["depth"]) if dd == d}
        if mine == theirs:
            continue
        if set(mine) != set(theirs):
            out.append(("top-g cut", _exchange_gap(tr, got["pool"])))
        both = [p for p in mine if p in theirs]
        if any(mine[p][1] != theirs[p][1] for p in both):
            return []                          # same candidate, other token: not a ranking matter
        moved = [p for p in both if mine[p][0] != theirs[p][0]]
        if moved:
            if d not in tr.layer_gaps:
                return []
            rank = lambda s_: k if s_ < 0 else s_
            worst = 0.0
            for p in moved:        # a candidate crossed every rank between its two places
                lo, hi = sorted((rank(mine[p][0]), rank(theirs[p][0])))
                worst = max(worst, float(max(tr.layer_gaps[d][lo:hi], default=np.inf)))
            out.append((f"frontier ranking of depth {d}", worst))
        break
    return out


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
               max_lse_err=0.0, max_score_err=0.0, max_reward_rel=0.0, max_adv_err=0.0, max_grad_err=0.0,
               mean_path_len=0.0, mean_needed_rows=0.0)
    fwd = []
    excused = np.zeros(n, dtype=bool)
    for i in range(n):
        d_i = np.asarray(draft[:, i], dtype=np.float64)
        t_i = np.asarray(target[:, i], dtype=np.float64)
        f = orc.position_forward(d_i, t_i, D, k, g, d2t, cfg.eta, agg, getattr(cfg, "all_nodes", False),
                                 getattr(cfg, "expected_path", False))
        fwd.append(f)
        for t in range(G):
            tr = f["trees"][t]
            same = all(np.array_equal(gpu[name][t, i], getattr(tr, attr)) for name, attr in
                       [("node_token", "token"), ("node_parent", "parent"), ("node_depth", "depth"),
                        ("node_ctx_row", "ctx_row"), ("node_slot", "slot"), ("node_pool", "pool")])
            if not same:
                why = differing_decisions(tr, dict(pool=gpu["node_pool"][t, i], slot=gpu["node_slot"][t, i],
                                                   token=gpu["node_token"][t, i], depth=gpu["node_depth"][t, i]))
                assert why and all(gap < TIE_TOL for _, gap in why), (
                    f"tree structure mismatch at position {positions[i]} tree {t}: {why or 'no ranking decision differs'}")
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
            # an fp32 output: besides the 1e-5 of the row's log-sum-exp, its own rounding (2^-24
            # relative) counts once |log p| reaches the hundreds (heavy-tailed fp32 logits)
            assert _close(gpu["node_logp"][t, i], tr.logp, rtol=2.0 ** -23, atol=1e-5)
            err = np.max(np.abs(gpu["node_score"][t, i] - tr.score))
            rep["max_score_err"] = max(rep["max_score_err"], float(err))
            assert err <= 1e-5, f"score error {err} at {positions[i]}"
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
            # stored as fp32: values below the smallest normal number may flush
            assert _close(gpu["node_ptarget"][t, i], rw["p"], atol=1e-37)
            assert _close(gpu["node_pathprod"][t, i], rw["Pp"], atol=1e-37)
            assert _close(gpu["node_L"][t, i], rw["Lc"], atol=1e-37)
            rel = abs(gpu["reward"][t, i] - rw["r"]) / max(1e-7, abs(rw["r"]))
            rep["max_reward_rel"] = max(rep["max_reward_rel"], float(rel))
            assert rel <= REL_TOL, f"reward {gpu['reward'][t, i]} vs {rw['r']}"
            assert _close(gpu["etree"][t, i], rw["etree"], atol=1e-37)
            assert gpu["n_leaves"][t, i] == len(rw["leaves"])
        if excused[i]:
            continue
        path = f["path"]
        l = len(path["nodes"])
        rep["mean_path_len"] += l / n
        if getattr(cfg, "expected_path", False) and list(gpu["path_node"][i][:gpu["path_len"][i]]) != path["nodes"]:
            # the arg-max over L is a floating-point decision: another sequence is excused only if
            # its L is within the tie window of the best one
            rw0 = f["rewards"][0]
            other = int(gpu["path_node"][i][gpu["path_len"][i] - 1]) if gpu["path_len"][i] > 0 else -1
            assert other in [int(x) for x in rw0["leaves"]] and \
                rw0["Lc"][path["nodes"][-1]] - rw0["Lc"][other] < TIE_TOL, f"sequence choice at {positions[i]}"
            rep["near_tie_trees"] += 1
            excused[i] = True
            continue
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
        # a difference of two rewards: relative to the rewards, not to the difference
        assert np.all(np.abs(gpu["R"][idx] - R) <= REL_TOL * np.maximum(np.abs(r_cur), np.abs(r_ref)))
        adv_err = np.max(np.abs(gpu["adv"][idx] - A) / np.maximum(1.0, np.abs(A)))
        rep["max_adv_err"] = max(rep["max_adv_err"], float(adv_err))
        assert adv_err <= REL_TOL, f"advantage error {adv_err}"
        assert _close(gpu["ratio"][idx], sur["ratio"])          # s > 0: a relative bound
        edge = np.minimum(np.abs(sur["ratio"] - (1 + cfg.clip_eps)),
                          np.abs(sur["ratio"] - (1 - cfg.clip_eps))) < CLIP_EDGE_TOL
        rep["clip_edge"] += int(edge.sum())
        if edge.any():
            continue
        assert np.array_equal(gpu["active"][idx].astype(bool), sur["active"])
        # coefficients and the group loss are sums over advantages: 1e-4 of the advantages' scale
        scale = REL_TOL * float(np.max(np.abs(A) * sur["ratio"])) / m
        assert _close(gpu["coeff"][idx], sur["coeff"], rtol=REL_TOL, atol=abs(cfg.grad_scale) * scale)
        assert _close(gpu["loss"][g0 // m], sur["loss"][0], rtol=REL_TOL, atol=m * scale)
        for j, i in enumerate(idx):
            l = path_len[j]
            d_i = np.asarray(draft[0, i], dtype=np.float64)
            rows = [d_i[orc.draft_slot_of_row(int(r), k)] for r in path_row[j, :l]]
            lse = [fwd[i]["trees"][0].row_lse[r] for r in path_row[j, :l]]
            want = orc.surrogate_grad_rows(rows, lse, list(path_tok[j, :l]), sur["coeff"][j], D,
                                           draft.shape[-1])
            err = float(np.max(np.abs(gpu["grad"][i] - want)))
            rep["max_grad_err"] = max(rep["max_grad_err"], err)
            # 2e-3 absolute is stated for grad_scale = 1; entries scale with it
            assert err <= GRAD_ATOL * abs(cfg.grad_scale), f"gradient error {err} at position {positions[i]}"
    return rep
