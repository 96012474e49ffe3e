"""The comparison harness itself (oracle/check.py): a structural mismatch is excused only by
the ranking decision that was actually resolved differently, never by an unrelated near tie."""
import numpy as np
import pytest

from oracle import check as ocheck
from oracle import gto_oracle as orc

D, K, G_NODES, V = 4, 3, 12, 12


def lists(tree):
    return dict(pool=tree.pool, slot=tree.slot, token=tree.token, depth=tree.depth)


def candidate_site(tree_draft, tree, node):
    """(d, j, token) of the draft logit that feeds the edge into `node`."""
    d, j = orc.draft_slot_of_row(int(tree.ctx_row[node]), K)
    return d, j, int(tree.token[node])


def find_case(kind):
    """A random tree plus a copy of its logits with ONE logit raised just enough to flip one
    decision: two adjacent frontier ranks of a layer, or the top-g cut."""
    for seed in range(200):
        rng = np.random.default_rng(seed)
        draft = rng.normal(size=(D, K, V)) * 2.0
        tr = orc.build_tree(draft, D, K, G_NODES)
        if kind == "layer":
            d = 2 + seed % (D - 2)
            nodes = [n for n in range(tr.g) if tr.depth[n] == d and tr.slot[n] >= 0]
            by_slot = {int(tr.slot[n]): n for n in nodes}
            pairs = [r for r in range(K - 1) if r in by_slot and r + 1 in by_slot]
            if not pairs:
                continue
            r = pairs[0]
            lower = by_slot[r + 1]
            gap = tr.layer_gaps[d][r]
            site = candidate_site(draft, tr, lower)
            p_edge = np.exp(tr.logp[lower])
        else:
            gap = tr.cut_gaps[-1]
            # the best unselected candidate: rebuild with one more node to learn where it sits
            bigger = orc.build_tree(draft, D, K, G_NODES + 1)
            extra = [n for n in range(bigger.g) if bigger.pool[n] not in set(tr.pool)]
            if len(extra) != 1:
                continue
            site = candidate_site(draft, bigger, extra[0])
            p_edge = np.exp(bigger.logp[extra[0]])
            d, r = None, None
        if not (1e-3 < gap < 0.3):
            continue
        bumped = draft.copy()
        bumped[site] += gap * 1.2 / (1.0 - p_edge)     # raises the edge's log-probability by 1.2 gap
        other = orc.build_tree(bumped, D, K, G_NODES)
        if kind == "layer":
            # keep the case only if the bump did exactly what was meant: same nodes down to
            # depth d, with the slots of the two chosen nodes exchanged
            upto = lambda t: {int(p): int(s) for p, s, dd in zip(t.pool, t.slot, t.depth) if dd <= d}
            want = upto(tr)
            a, b = int(tr.pool[by_slot[r]]), int(tr.pool[lower])
            want[a], want[b] = want[b], want[a]
            if upto(other) != want:
                continue
        else:
            if len(set(other.pool) - set(tr.pool)) != 1 or not np.array_equal(
                    other.slot[np.isin(other.pool, tr.pool)], tr.slot[np.isin(tr.pool, other.pool)]):
                continue
        why = ocheck.differing_decisions(tr, lists(other))
        return tr, other, why, gap, d
    raise AssertionError("no case found")


def test_a_flipped_frontier_ranking_is_named_with_its_own_gap():
    tr, other, why, gap, d = find_case("layer")
    assert len(why) == 1 and why[0][0] == f"frontier ranking of depth {d}"
    assert why[0][1] == pytest.approx(gap, rel=1e-12)
    assert min(tr.cut_gaps) <= gap          # an unrelated, smaller gap may exist: it must not excuse


def test_a_flipped_top_g_cut_is_named_with_its_own_gap():
    tr, other, why, gap, _ = find_case("cut")
    assert why == [("top-g cut", pytest.approx(gap, rel=1e-12))]


def test_the_cut_gap_is_taken_between_the_candidates_that_were_exchanged():
    """The oracle's neighbour across the cut is a sibling with the same logit (decided by the
    index everywhere, gap inf); the other side kept the next candidate instead, which scores
    just below: the decision that differs is that one, with its own finite gap."""
    for seed in range(2000):
        rng = np.random.default_rng(seed)
        draft = np.round(rng.normal(size=(D, K, V)) * 2.0 * 4) / 4       # a coarse grid: equal logits occur
        tr = orc.build_tree(draft, D, K, G_NODES)
        if tr.cut_gaps[-1] != np.inf:
            continue
        ranked = sorted(range(len(tr.cand_score)), key=lambda p: (-tr.cand_score[p], p))
        x, x2, y = ranked[G_NODES - 1], ranked[G_NODES], ranked[G_NODES + 1]
        if tr.cand_parent[x] != tr.cand_parent[x2] or tr.cand_score[x] != tr.cand_score[x2]:
            continue
        gap = tr.cand_score[x] - tr.cand_score[y]
        up, related = int(tr.cand_parent[y]), False
        while up >= 0:
            related |= up in (x, x2)
            up = int(tr.cand_parent[up])
        if related or tr.cand_parent[y] == tr.cand_parent[x] or not (1e-3 < gap < 0.3):
            continue
        # raise the logit behind y just enough for it to pass x (and x's twin)
        bigger = orc.build_tree(draft, D, K, G_NODES + 2)
        at = [n for n in range(bigger.g) if int(bigger.pool[n]) == y]
        if len(at) != 1:
            continue
        site = candidate_site(draft, bigger, at[0])
        bumped = draft.copy()
        bumped[site] += gap * 1.2 / (1.0 - np.exp(bigger.logp[at[0]]))
        other = orc.build_tree(bumped, D, K, G_NODES)
        if set(int(p) for p in other.pool) != (set(int(p) for p in tr.pool) - {x}) | {y}:
            continue
        why = ocheck.differing_decisions(tr, lists(other))
        assert why and why[0][0] == "top-g cut" and why[0][1] == pytest.approx(gap, rel=1e-12)
        return
    raise AssertionError("no case found")


def test_two_separate_exchanges_in_one_layer_do_not_span_the_ranks_between_them():
    rng = np.random.default_rng(3)
    for _ in range(200):
        tr = orc.build_tree(rng.normal(size=(D, K, V)) * 2.0, D, K, G_NODES)
        d = 2
        at = {int(tr.slot[n]): n for n in range(tr.g) if tr.depth[n] == d and tr.slot[n] >= 0}
        if len(at) == K:
            break
    # hand-made gaps between the ranks (0,1), (1,2), (2,3) of the layer: tiny, large, tiny
    other = lists(tr)
    other["slot"] = tr.slot.copy()
    other["slot"][at[0]], other["slot"][at[1]] = 1, 0
    saved = tr.layer_gaps[d]
    tr.layer_gaps[d] = [1e-9, 5.0, 2e-9][:len(saved)] + list(saved[3:])
    why = ocheck.differing_decisions(tr, other)
    assert why == [(f"frontier ranking of depth {d}", 1e-9)]
    # a candidate that moved from rank 0 to rank 2 did cross the large gap
    other["slot"][at[0]], other["slot"][at[1]], other["slot"][at[2]] = 2, 0, 1
    why = ocheck.differing_decisions(tr, other)
    assert why == [(f"frontier ranking of depth {d}", 5.0)]


def test_identical_trees_and_plain_errors():
    rng = np.random.default_rng(7)
    tr = orc.build_tree(rng.normal(size=(D, K, V)) * 2.0, D, K, G_NODES)
    assert ocheck.differing_decisions(tr, lists(tr)) == []
    wrong = lists(tr)
    wrong["token"] = tr.token.copy()
    wrong["token"][3] += 1                  # same candidate, another token: no ranking explains it
    assert ocheck.differing_decisions(tr, wrong) == []


def test_relative_bound_has_no_floor():
    assert ocheck._close([1.00005e-3], [1e-3])
    assert not ocheck._close([1.1e-3], [1e-3])          # 10 % off on a small probability
    assert not ocheck._close([2e-9], [1e-9])
