"""Plain fp64 CPU oracle of the GTO draft-tree pass (test infrastructure only).

Everything here is written out from the paper's definitions, one position and one
tree at a time, with numpy for the V-wide reductions and plain Python loops for the
tree logic.  Nothing is blocked, fused or reordered, so each function can be read
against the passage it cites.  Inputs are the logits *as stored* (bf16 or fp32
values converted exactly to float64).

Steps and the passages they follow:

  lse_and_topk          Sec. 3.1 (i): the distribution each expansion draws from
  build_tree            Sec. 3.1 (i) layer-wise expansion, (ii) global prune/re-rank,
                        Fig. 1 caption (path confidence = product of edge probabilities)
  target_node_probs     Sec. 3.1, the factor T(x_{t+k} | ...) of Eq. 4
  tree_reward           Sec. 3.1 Eq. 3-5 (expected acceptance length, smooth max)
  longest_accepted      Sec. 3.2 "longest accepted sequence", App. A case (b) (greedy target)
  most_expected_sequence  the other reading of that phrase: the sequence with the largest L_i
  group_advantages      Sec. 3.2 Eq. 9-10 (debias, standardise)
  clipped_surrogate     Sec. 3.2 Eq. 11-12 (length-normalised ratio, PPO clip)
  surrogate_grad_rows   derivative of Eq. 12 with respect to the draft logits
  token_loss            Sec. 3.2 Eq. 13 and App. B: teacher-to-student cross-entropy per prefix

Readings fixed where the paper is silent (all listed in the design notes):
  * global acceptance score = sum of draft log-probabilities along the path;
  * every tie is broken toward the lower index (token id, layer candidate index,
    pool index, target id);
  * the prune pool is every candidate node (k at depth 1, k*k at each later depth);
    g counts nodes and excludes the root; nodes are listed in ascending pool index;
  * the sequences S_i of Eq. 2 are the root-to-leaf paths of the selected tree;
  * "accepted" means greedy (temperature 0) verification; the bonus token is not counted;
  * std is the population std; groups are consecutive blocks of m positions;
  * advantages and the old-policy log-probabilities are constants for the gradient;
  * with a reduced draft vocabulary the target distribution of the token-level loss is
    renormalised over the mapped ids.

Pins (tests/test_oracle_*.py): naive long-double log-sum-exp, brute-force sort,
an independent path-enumerating tree builder, special cases k=1 / D=1 / g=P, the
Fig. 1 worked example, exact enumeration and Monte-Carlo of target roll-outs, the
single-chain one-hot case, Eq. (1) bounds, scipy z-score, finite differences and
autograd for the gradient.  Conventions with no counterpart to check against
(node order, leaf definition of S_i, clip-edge equality) are "parity unpinned"
with respect to the authors' code.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

AGG_LSE = 0   # Eq. 5 (default)
AGG_MAX = 1   # Sec. 4.2 "Max"
AGG_MEAN = 2  # Sec. 4.2 "Sum (Average)"


# --------------------------------------------------------------------------- O1
def lse_and_topk(z, k):
    """Log-sum-exp of one logit row and its k best tokens.

    Sec. 3.1 (i): each frontier node proposes its k most probable tokens under the
    draft distribution softmax(z).  Returns (lse, ids[k], logp[k]) where
    logp = z[ids] - lse and ids are ordered by (value descending, id ascending).
    """
    z = np.asarray(z, dtype=np.float64)
    zmax = np.max(z)
    lse = zmax + np.log(np.sum(np.exp(z - zmax)))
    order = np.argsort(-z, kind="stable")  # stable: equal values keep ascending id
    ids = order[:k].astype(np.int64)
    return float(lse), ids, z[ids] - lse


def argmax_low(z):
    """Index of the largest entry, lowest index on ties (greedy target token)."""
    z = np.asarray(z)
    return int(np.flatnonzero(z == np.max(z))[0])


# ------------------------------------------------------------------------ O2-O4
@dataclass
class DraftTree:
    """The pruned draft tree of one position (g nodes, root excluded)."""
    D: int
    k: int
    g: int
    token: np.ndarray      # [g] draft-vocabulary id of the node's token
    parent: np.ndarray     # [g] list position of the parent node, -1 = child of the root
    depth: np.ndarray      # [g] 1..D
    ctx_row: np.ndarray    # [g] context row the token was proposed from (0 = root)
    slot: np.ndarray       # [g] frontier slot of the node at its depth, -1 if never expanded
    pool: np.ndarray       # [g] pool index (depth-major candidate number)
    logp: np.ndarray       # [g] draft log-probability of the edge into the node
    score: np.ndarray      # [g] global acceptance score = sum of logp on the path
    mask: np.ndarray       # [g,g] bool, mask[n,a] = a is n or an ancestor of n
    row_lse: np.ndarray    # [R] draft log-sum-exp of every context row
    cut_gaps: list = field(default_factory=list)  # smallest score gap behind each layer ranking and the top-g cut
    layer_gaps: dict = field(default_factory=dict)  # depth d -> gaps between ranks (r, r+1), r < k, of layer d's ranking
    cand_score: np.ndarray = None   # [P] score of every candidate of the pool, selected or not
    cand_parent: np.ndarray = None  # [P] pool index of every candidate's parent, -1 = child of the root


def context_row(d, j, k):
    """Row index of frontier slot j at depth d (d = 0 is the root)."""
    return 0 if d == 0 else 1 + (d - 1) * k + j


def draft_slot_of_row(r, k):
    """Inverse of context_row: (d, j) such that the draft tensor [D, k, V] holds context
    row r at [d, j] (row 0 is the root at [0, 0]; [0, 1:] holds no context)."""
    return (0, 0) if r == 0 else (1 + (r - 1) // k, (r - 1) % k)


def _decision_gap(pool, a, b):
    """Score gap between two candidates that a ranking decision separates (a ranked first).
    Two cases are decided by the index on every implementation and are not fragile, so they
    report inf: two children of one parent with the same logit (their scores are the same
    sum), and a candidate against its own descendant (a log-probability is never positive,
    so the descendant cannot score higher, and on a tie the ancestor has the lower index)."""
    gap = pool[a]["score"] - pool[b]["score"]
    if gap == 0.0 and pool[a]["parent_pool"] == pool[b]["parent_pool"]:
        return np.inf
    up = pool[b]["parent_pool"]
    while up >= 0:
        if up == a:
            return np.inf
        up = pool[up]["parent_pool"]
    return gap


def build_tree(draft, D, k, g):
    """Decoding-time tree policy G of Sec. 3.1 on one position.

    draft: [D, k, V] logits; draft[0, 0] is the root context, draft[d, j] (d >= 1) is
    the context reached through frontier slot j of depth d; draft[0, 1:] is unused.

    (i) Layer-wise expansion: at depth 1 the root's k best tokens are the candidates
    and all become frontier slots.  At depth d >= 2 every frontier node of depth d-1
    proposes its k best tokens; candidate q = j*k + c has score
    score(frontier j) + logp(c | context j).  While d < D the k best candidates of
    the layer (score descending, q ascending) become the next frontier, slot = rank.
    (ii) Global prune: all k + (D-1)*k*k candidates are re-ranked by
    (score descending, pool index ascending) and the best g kept.
    """
    R = 1 + (D - 1) * k
    P = k + (D - 1) * k * k
    assert 1 <= g <= P
    row_lse = np.full(R, np.nan)
    pool = []          # pool[p] = dict(score, logp, depth, ctx_row, token, parent_pool)
    slot_of = {}       # pool index -> frontier slot
    cut_gaps = []
    layer_gaps = {}

    lse, ids, lp = lse_and_topk(draft[0, 0], k)
    row_lse[0] = lse
    for c in range(k):
        pool.append(dict(score=lp[c], logp=lp[c], depth=1, ctx_row=0,
                         token=int(ids[c]), parent_pool=-1))
    frontier = list(range(k)) if D > 1 else []   # pool indices, in slot order
    for j, p in enumerate(frontier):
        slot_of[p] = j

    for d in range(2, D + 1):
        base = k + (d - 2) * k * k
        for j, fp in enumerate(frontier):
            row = context_row(d - 1, j, k)
            lse, ids, lp = lse_and_topk(draft[d - 1, j], k)
            row_lse[row] = lse
            for c in range(k):
                pool.append(dict(score=pool[fp]["score"] + lp[c], logp=lp[c], depth=d,
                                 ctx_row=row, token=int(ids[c]), parent_pool=fp))
        if d < D:
            layer = list(range(base, base + k * k))
            layer.sort(key=lambda p: (-pool[p]["score"], p))
            frontier = layer[:k]
            # slots are ranks, so every adjacent pair down to the cut is a decision
            layer_gaps[d] = [_decision_gap(pool, layer[r], layer[r + 1])
                             for r in range(min(k, len(layer) - 1))]
            cut_gaps.append(min(layer_gaps[d], default=np.inf))
            for j, p in enumerate(frontier):
                slot_of[p] = j
    assert len(pool) == P

    ranked = sorted(range(P), key=lambda p: (-pool[p]["score"], p))
    cut_gaps.append(_decision_gap(pool, ranked[g - 1], ranked[g]) if P > g else np.inf)
    selected = sorted(ranked[:g])
    pos = {p: n for n, p in enumerate(selected)}

    token = np.array([pool[p]["token"] for p in selected], dtype=np.int64)
    depth = np.array([pool[p]["depth"] for p in selected], dtype=np.int64)
    ctx = np.array([pool[p]["ctx_row"] for p in selected], dtype=np.int64)
    logp = np.array([pool[p]["logp"] for p in selected], dtype=np.float64)
    score = np.array([pool[p]["score"] for p in selected], dtype=np.float64)
    slot = np.array([slot_of.get(p, -1) for p in selected], dtype=np.int64)
    parent = np.empty(g, dtype=np.int64)
    mask = np.zeros((g, g), dtype=bool)
    for n, p in enumerate(selected):
        pp = pool[p]["parent_pool"]
        if pp < 0:
            parent[n] = -1
        else:
            # a parent scores at least as high as its child and has the lower pool
            # index, so it is always selected with it
            parent[n] = pos[pp]
            mask[n] = mask[parent[n]]
        mask[n, n] = True
    return DraftTree(D=D, k=k, g=g, token=token, parent=parent, depth=depth, ctx_row=ctx,
                     slot=slot, pool=np.array(selected, dtype=np.int64), logp=logp,
                     score=score, mask=mask, row_lse=row_lse, cut_gaps=cut_gaps,
                     layer_gaps=layer_gaps,
                     cand_score=np.array([c["score"] for c in pool], dtype=np.float64),
                     cand_parent=np.array([c["parent_pool"] for c in pool], dtype=np.int64))


# ------------------------------------------------------------------------ O5-O6
def target_node_probs(tree, target, d2t=None):
    """p_n = T(token_n | context of n): softmax of the node's context row of the
    target logits at the node's token (mapped to the target vocabulary by d2t).

    target: [R, V_t].  Returns (p[g], row_lse_t[R] with NaN for rows no node uses).
    """
    g = tree.g
    p = np.empty(g)
    lse_t = np.full(target.shape[0], np.nan)
    for n in range(g):
        r = int(tree.ctx_row[n])
        if np.isnan(lse_t[r]):
            z = np.asarray(target[r], dtype=np.float64)
            zmax = np.max(z)
            lse_t[r] = zmax + np.log(np.sum(np.exp(z - zmax)))
        tok = int(tree.token[n]) if d2t is None else int(d2t[int(tree.token[n])])
        p[n] = np.exp(float(target[r][tok]) - lse_t[r])
    return p, lse_t


def tree_reward(tree, p, eta=1.0, agg=AGG_LSE, all_nodes=False):
    """Draft Tree Reward, Eq. 3-5.

    Pp_n = product of p along the root-to-n path (Eq. 4), Lc_n = sum of Pp over the
    path (Eq. 3 for the sequence ending at n).  The sequences S_i are the
    root-to-leaf paths (leaf = selected node without a selected child), and
    r = (1/eta) log sum_i exp(eta L_i) (Eq. 5), or the Max / Average of Sec. 4.2.
    With all_nodes the sequences are the root-to-node paths of every selected node (the
    other reading of "N candidate sequences of length l_i <= d").
    Returns dict(r, Pp, Lc, leaves, etree) with etree = sum_n Pp_n (the exact
    expected number of accepted tokens when the target samples at temperature 1).
    """
    g = tree.g
    Pp = np.empty(g)
    Lc = np.empty(g)
    has_child = np.zeros(g, dtype=bool)
    for n in range(g):          # parents precede children in the list
        a = int(tree.parent[n])
        if a < 0:
            Pp[n] = p[n]
            Lc[n] = Pp[n]
        else:
            has_child[a] = True
            Pp[n] = p[n] * Pp[a]
            Lc[n] = Lc[a] + Pp[n]
    leaves = np.arange(g) if all_nodes else np.flatnonzero(~has_child)
    L = Lc[leaves]
    if agg == AGG_LSE:
        M = np.max(eta * L)
        r = (M + np.log(np.sum(np.exp(eta * L - M)))) / eta
    elif agg == AGG_MAX:
        r = np.max(L)
    elif agg == AGG_MEAN:
        r = np.mean(L)
    else:
        raise ValueError("unknown aggregation")
    return dict(r=float(r), Pp=Pp, Lc=Lc, leaves=leaves, etree=float(np.sum(Pp)))


# --------------------------------------------------------------------------- O7
def longest_accepted(tree, target, d2t=None):
    """Longest accepted sequence of the tree under greedy target verification.

    Start at the root context; the target's greedy token there is the arg-max of the
    context's target row (lowest id on ties).  If a selected child of the current node
    carries that token the walk moves to it, otherwise it stops.  A node that was
    never expanded (slot -1, or depth D) has no children, so the walk ends there.
    Returns dict(nodes, rows, tokens, logp): list positions, the context row of each
    step (the draft row that produced the token), the draft tokens and their draft
    log-probabilities.
    """
    k = tree.k
    children = {}
    for n in range(tree.g):
        children.setdefault(int(tree.parent[n]), []).append(n)
    nodes, rows, toks, lps = [], [], [], []
    cur, row = -1, 0
    while True:
        a = argmax_low(target[row])
        nxt = None
        for n in children.get(cur, []):
            t = int(tree.token[n]) if d2t is None else int(d2t[int(tree.token[n])])
            if t == a:
                nxt = n
                break
        if nxt is None:
            break
        assert int(tree.ctx_row[nxt]) == row
        nodes.append(nxt)
        rows.append(row)
        toks.append(int(tree.token[nxt]))
        lps.append(float(tree.logp[nxt]))
        if tree.slot[nxt] < 0 or tree.depth[nxt] >= tree.D:
            break
        cur, row = nxt, context_row(int(tree.depth[nxt]), int(tree.slot[nxt]), k)
    return dict(nodes=nodes, rows=rows, tokens=toks, logp=lps)


def most_expected_sequence(tree, Lc, leaves):
    """The other reading of "longest accepted sequence" (Sec. 3.2): instead of verifying
    greedily, take the candidate sequence S_i whose expected acceptance length L_i (Eq. 3) is
    the largest - the lowest list position on ties - and return it whole, root to its last
    node, in the form longest_accepted uses.  Lc, leaves: from tree_reward.
    """
    leaves = [int(n) for n in leaves]
    best = leaves[0]
    for n in leaves[1:]:
        if Lc[n] > Lc[best]:
            best = n
    chain = []
    n = best
    while n >= 0:
        chain.append(n)
        n = int(tree.parent[n])
    chain.reverse()
    return dict(nodes=chain, rows=[int(tree.ctx_row[n]) for n in chain],
                tokens=[int(tree.token[n]) for n in chain], logp=[float(tree.logp[n]) for n in chain])


# --------------------------------------------------------------------------- O8
def group_advantages(r_cur, r_ref, m, delta=1e-6, unbiased=False, debias=True):
    """Eq. 9: R_i = r(T_i) - r(T_i under the reference draft); Eq. 10: standardise R
    within each block of m consecutive positions, A = (R - mean) / (std + delta),
    std being the population standard deviation (divide by m).
    Returns (R[B], A[B]).
    """
    r_cur = np.asarray(r_cur, dtype=np.float64)
    r_ref = np.asarray(r_ref, dtype=np.float64)
    B = r_cur.shape[0]
    assert B % m == 0
    R = r_cur - r_ref if debias else r_cur.copy()
    A = np.empty(B)
    for k0 in range(0, B, m):
        grp = R[k0:k0 + m]
        mean = np.sum(grp) / m
        var = np.sum((grp - mean) ** 2) / ((m - 1) if (unbiased and m > 1) else m)
        A[k0:k0 + m] = (grp - mean) / (np.sqrt(var) + delta)
    return R, A


# --------------------------------------------------------------------------- O9
def clipped_surrogate(path_logp, old_logp, path_len, adv, m, eps=0.2, grad_scale=1.0):
    """Eq. 11-12 for a batch of B positions grouped in blocks of m.

    path_logp, old_logp: [B, D] per-token log-probabilities of the longest accepted
    sequence under the current and the old / reference draft (entries >= path_len
    are ignored).  s_i = exp((sum cur - sum old) / max(l_i, 1));
    loss_k = -(1/m) sum_i min(s_i A_i, clip(s_i, 1-eps, 1+eps) A_i).
    The term of position i has a non-zero derivative iff the unclipped branch is the
    minimum: (A >= 0 and s <= 1+eps) or (A < 0 and s >= 1-eps).
    Returns dict(ratio[B], active[B], loss[B/m], coeff[B]) where coeff_i multiplies
    d(log M(token_j | ctx_j))/dz for every step j < l_i of position i:
    coeff_i = grad_scale * (-1/m) * A_i * s_i / max(l_i, 1) if active else 0.
    """
    path_logp = np.asarray(path_logp, dtype=np.float64)
    old_logp = np.asarray(old_logp, dtype=np.float64)
    B = path_logp.shape[0]
    s = np.empty(B)
    active = np.zeros(B, dtype=bool)
    coeff = np.zeros(B)
    loss = np.zeros(B // m)
    for i in range(B):
        l = int(path_len[i])
        diff = float(np.sum(path_logp[i, :l]) - np.sum(old_logp[i, :l]))
        s[i] = np.exp(diff / max(l, 1))
        clipped = min(max(s[i], 1.0 - eps), 1.0 + eps)
        loss[i // m] += -(1.0 / m) * min(s[i] * adv[i], clipped * adv[i])
        active[i] = (adv[i] >= 0 and s[i] <= 1.0 + eps) or (adv[i] < 0 and s[i] >= 1.0 - eps)
        if active[i]:
            coeff[i] = grad_scale * (-1.0 / m) * adv[i] * s[i] / max(l, 1)
    return dict(ratio=s, active=active, loss=loss, coeff=coeff)


def surrogate_grad_rows(draft_rows, row_lse, tokens, coeff, D, V):
    """Gradient of the summed group losses with respect to the draft logits of the
    rows on one position's longest accepted sequence.

    d log softmax(z)[tok] / dz = onehot(tok) - softmax(z), so step j receives
    coeff * (onehot(token_j) - softmax(draft_rows[j])).  Rows j >= len(tokens) are 0.
    draft_rows: list of [V] logit rows (the context rows of the path); row_lse: their
    log-sum-exp.  Returns [D, V].
    """
    out = np.zeros((D, V))
    for j, tok in enumerate(tokens):
        z = np.asarray(draft_rows[j], dtype=np.float64)
        softmax = np.exp(z - row_lse[j])
        out[j] = -coeff * softmax
        out[j, tok] += coeff
    return out


# ------------------------------------------------------------------ whole passes
def position_forward(draft_b, target_b, D, k, g, d2t=None, eta=1.0, agg=AGG_LSE, all_nodes=False,
                     expected_path=False):
    """Trees, rewards and the longest accepted sequence of one position.

    draft_b: [G, D, k, V_d], target_b: [G, R, V_t] with G = 2 (0 = current draft,
    1 = frozen reference draft).  expected_path selects most_expected_sequence instead of the
    greedy walk.  Returns dict(trees, probs, rewards, path).
    """
    G = draft_b.shape[0]
    trees, probs, rewards = [], [], []
    for t in range(G):
        tree = build_tree(draft_b[t], D, k, g)
        p, lse_t = target_node_probs(tree, target_b[t], d2t)
        rw = tree_reward(tree, p, eta, agg, all_nodes)
        rw["p"] = p
        rw["row_lse_t"] = lse_t
        trees.append(tree)
        probs.append(p)
        rewards.append(rw)
    if expected_path:
        path = most_expected_sequence(trees[0], rewards[0]["Lc"], rewards[0]["leaves"])
    else:
        path = longest_accepted(trees[0], target_b[0], d2t)
    return dict(trees=trees, rewards=rewards, path=path)


def group_pass(draft_g, target_g, D, k, g, m, old_logp_fn, d2t=None, eta=1.0, agg=AGG_LSE,
               delta=1e-6, eps=0.2, grad_scale=1.0, unbiased=False, debias=True, all_nodes=False,
               expected_path=False):
    """The whole pass of Algorithm 1's inner loop on ONE group of m positions: trees and
    rewards of both drafts, the longest accepted sequences, Eq. 9-12 and the gradient rows.
    Sequences the functions above; adds no arithmetic of its own.

    draft_g: [G, m, D, k, V_d], target_g: [G, m, R, V_t].
    old_logp_fn(path_logp[m,D], path_row[m,D], path_token[m,D], path_len[m]) -> [m, D]:
    the old-policy log-probabilities of the accepted tokens (an input of the method).
    Returns dict(fwd, R, A, path_len, path_logp, path_row, path_token, old, sur, grad[m,D,V_d]).
    """
    V = draft_g.shape[-1]
    fwd = [position_forward(np.asarray(draft_g[:, i], dtype=np.float64),
                            np.asarray(target_g[:, i], dtype=np.float64), D, k, g, d2t, eta, agg,
                            all_nodes, expected_path)
           for i in range(m)]
    r_cur = np.array([f["rewards"][0]["r"] for f in fwd])
    r_ref = np.array([f["rewards"][1]["r"] for f in fwd])
    R, A = group_advantages(r_cur, r_ref, m, delta, unbiased=unbiased, debias=debias)
    path_len = np.array([len(f["path"]["nodes"]) for f in fwd])
    path_logp = np.zeros((m, D))
    path_row = np.full((m, D), -1, dtype=np.int64)
    path_tok = np.full((m, D), -1, dtype=np.int64)
    for i, f in enumerate(fwd):
        l = path_len[i]
        path_logp[i, :l] = f["path"]["logp"]
        path_row[i, :l] = f["path"]["rows"]
        path_tok[i, :l] = f["path"]["tokens"]
    old = old_logp_fn(path_logp, path_row, path_tok, path_len)
    sur = clipped_surrogate(path_logp, old, path_len, A, m, eps, grad_scale)
    grad = np.zeros((m, D, V))
    for i, f in enumerate(fwd):
        l = path_len[i]
        d_i = np.asarray(draft_g[0, i], dtype=np.float64)          # [D, k, V] of the current draft
        rows = [d_i[draft_slot_of_row(int(r), k)] for r in path_row[i, :l]]
        lse = [f["trees"][0].row_lse[r] for r in path_row[i, :l]]
        grad[i] = surrogate_grad_rows(rows, lse, list(path_tok[i, :l]), sur["coeff"][i], D, V)
    return dict(fwd=fwd, R=R, A=A, path_len=path_len, path_logp=path_logp, path_row=path_row,
                path_token=path_tok, old=old, sur=sur, grad=grad)


# ------------------------------------------------------------------ token-level loss
def token_loss(z_draft, z_target, d2t=None):
    """Token-level loss of Eq. 13 / App. B for one teacher-forced prefix: the cross-entropy
    H(p_T, p_M) = -sum_v p_T(v) log p_M(v) from the target's next-token distribution to the
    draft's, and its derivative with respect to the draft logits, p_M - p_T.

    z_draft: [V_d] draft logits of the prefix; z_target: [V_t] target logits of the same
    prefix.  With a reduced draft vocabulary (d2t: draft id -> target id) the target
    distribution is the softmax of the target logits at the mapped ids only, so that both
    distributions live on the draft vocabulary (the paper sums over one common vocabulary).
    Returns (H, grad[V_d]).
    """
    zd = np.asarray(z_draft, dtype=np.float64)
    zt = np.asarray(z_target, dtype=np.float64)
    if d2t is not None:
        zt = zt[np.asarray(d2t, dtype=np.int64)]
    assert zd.shape == zt.shape
    md, mt = np.max(zd), np.max(zt)
    log_pm = zd - (md + np.log(np.sum(np.exp(zd - md))))
    log_pt = zt - (mt + np.log(np.sum(np.exp(zt - mt))))
    p_t = np.exp(log_pt)
    H = -float(np.sum(p_t * log_pm))
    return H, np.exp(log_pm) - p_t


# ------------------------------------------------------------------ grouping
def sample_groups(s, m, K, u):
    """SampleGroups of Algorithm 1 under the constraints of Eq. 6-7: K non-overlapping
    groups of m adjacent positions of a sequence of length s, start indices 1-based with
    1 <= t_k <= s - m + 1 and t_{k+1} >= t_k + m.  The paper does not say how the starts
    are drawn; here the K uniforms u in [0, 1) are turned into K independent integer offsets
    in [0, s - K m], sorted, and the k-th (0-based) is shifted by k m.  Every admissible
    placement can occur; its probability is proportional to the number of orderings of its
    offsets (placements with equal offsets, i.e. groups back to back, are rarer).
    Returns the start indices t_1 < ... < t_K.
    """
    assert K >= 0 and m >= 1 and K * m <= s
    free = s - K * m
    gaps = sorted(min(int(np.floor(float(x) * (free + 1))), free) for x in u[:K])
    return [1 + gp + i * m for i, gp in enumerate(gaps)]
