"""The pins must be sensitive: plausible mistakes planted IN THE ORACLE (a dropped factor, a
wrong sign, a wrong tie-break, a sample instead of a population statistic, a transposed
operand) have to make at least one pin fail.  Each case swaps one oracle function for a
mutant and re-runs the pins that cover it."""
import numpy as np
import pytest

from oracle import gto_oracle as orc

import test_oracle_group as tg
import test_oracle_pass as tp
import test_oracle_reward as tr
import test_oracle_rows as trow
import test_oracle_token_loss as tt
import test_oracle_tree as ttree


def fails(fn, *args):
    try:
        fn(*args)
    except AssertionError:
        return True
    return False


def test_reward_dropped_path_product(monkeypatch):
    real = orc.tree_reward

    def mutant(tree, p, eta=1.0, agg=orc.AGG_LSE, all_nodes=False):
        out = real(tree, p, eta, agg, all_nodes)
        # Eq. 3 with the edge probability instead of the product along the path
        Lc = np.empty(tree.g)
        for n in range(tree.g):
            a = int(tree.parent[n])
            Lc[n] = p[n] + (Lc[a] if a >= 0 else 0.0)
        L = Lc[out["leaves"]]
        out = dict(out, Lc=Lc, r=float(np.log(np.sum(np.exp(eta * L))) / eta))
        return out
    monkeypatch.setattr(orc, "tree_reward", mutant)
    assert fails(tr.test_sequence_length_is_expected_leading_matches_by_enumeration, 0)
    assert fails(tr.test_single_chain_one_hot_reward_counts_matching_tokens, 3) or \
        fails(tr.test_sequence_length_by_monte_carlo)


def test_reward_missing_one_over_eta(monkeypatch):
    real = orc.tree_reward

    def mutant(tree, p, eta=1.0, agg=orc.AGG_LSE, all_nodes=False):
        out = real(tree, p, eta, agg, all_nodes)
        if agg == orc.AGG_LSE:
            out = dict(out, r=out["r"] * eta)
        return out
    monkeypatch.setattr(orc, "tree_reward", mutant)
    assert fails(tr.test_eta_limits_and_variants)


def test_target_probability_ignores_the_id_map(monkeypatch):
    real = orc.target_node_probs
    monkeypatch.setattr(orc, "target_node_probs", lambda tree, target, d2t=None: real(tree, target, None))
    assert fails(tr.test_reduced_vocabulary_map_is_used_for_the_gather)


def test_walk_that_follows_the_draft_instead_of_the_greedy_target(monkeypatch):
    def mutant(tree, target, d2t=None):
        # always step to the first selected child: never consults the target
        nodes, rows, toks, lps = [], [], [], []
        cur, row = -1, 0
        while True:
            kids = [n for n in range(tree.g) if int(tree.parent[n]) == cur]
            if not kids:
                break
            n = kids[0]
            nodes.append(n); rows.append(row); toks.append(int(tree.token[n])); lps.append(float(tree.logp[n]))
            if tree.slot[n] < 0 or tree.depth[n] >= tree.D:
                break
            cur, row = n, orc.context_row(int(tree.depth[n]), int(tree.slot[n]), tree.k)
        return dict(nodes=nodes, rows=rows, tokens=toks, logp=lps)
    monkeypatch.setattr(orc, "longest_accepted", mutant)
    assert any(fails(tr.test_greedy_path_length_is_max_L_for_one_hot_targets, s) for s in range(6))
    assert fails(tr.test_walk_stops_at_unexpanded_node_and_on_mismatch)


def test_topk_ties_to_the_higher_index(monkeypatch):
    def mutant(z, k):
        z = np.asarray(z, dtype=np.float64)
        lse = np.max(z) + np.log(np.sum(np.exp(z - np.max(z))))
        order = np.argsort(-z[::-1], kind="stable")
        ids = (len(z) - 1 - order)[:k].astype(np.int64)
        return float(lse), ids, z[ids] - lse
    monkeypatch.setattr(orc, "lse_and_topk", mutant)
    assert fails(trow.test_topk_is_full_sort_with_low_index_ties) or \
        fails(trow.test_topk_constant_row_gives_first_ids)
    assert fails(ttree.test_ties_go_to_the_lower_index)


def test_lse_without_the_max_term(monkeypatch):
    def mutant(z, k):
        z = np.asarray(z, dtype=np.float64)
        lse = np.log(np.sum(np.exp(z - np.max(z))))          # forgot to add the max back
        ids = np.argsort(-z, kind="stable")[:k].astype(np.int64)
        return float(lse), ids, z[ids] - lse
    monkeypatch.setattr(orc, "lse_and_topk", mutant)
    assert fails(trow.test_lse_matches_naive_long_double, 512, 2.5)


def test_advantages_with_the_sample_std(monkeypatch):
    real = orc.group_advantages
    monkeypatch.setattr(orc, "group_advantages",
                        lambda rc, rr, m, delta=1e-6, unbiased=False, debias=True:
                        real(rc, rr, m, delta, True, debias))
    assert fails(tg.test_advantages_match_scipy_zscore_and_sum_to_zero)


def test_advantages_without_the_reference_reward(monkeypatch):
    real = orc.group_advantages
    monkeypatch.setattr(orc, "group_advantages",
                        lambda rc, rr, m, delta=1e-6, unbiased=False, debias=True:
                        real(rc, rr, m, delta, unbiased, False))
    assert fails(tg.test_advantages_match_scipy_zscore_and_sum_to_zero) or \
        fails(tg.test_advantages_special_cases)


def test_surrogate_with_the_wrong_sign_or_a_missing_length_normalisation(monkeypatch):
    real = orc.clipped_surrogate

    def flipped(*a, **kw):
        out = real(*a, **kw)
        return dict(out, coeff=-out["coeff"])
    monkeypatch.setattr(orc, "clipped_surrogate", flipped)
    assert fails(tg.test_gradient_matches_autograd_and_finite_differences, 0)

    def unnormalised(path_logp, old_logp, path_len, adv, m, eps=0.2, grad_scale=1.0):
        out = real(path_logp, old_logp, path_len, adv, m, eps, grad_scale)
        return dict(out, coeff=out["coeff"] * np.maximum(np.asarray(path_len), 1))
    monkeypatch.setattr(orc, "clipped_surrogate", unnormalised)
    assert fails(tg.test_gradient_matches_autograd_and_finite_differences, 1)


def test_gradient_rows_without_the_one_hot_term(monkeypatch):
    def mutant(draft_rows, row_lse, tokens, coeff, D, V):
        out = np.zeros((D, V))
        for j, _ in enumerate(tokens):
            out[j] = -coeff * np.exp(np.asarray(draft_rows[j], dtype=np.float64) - row_lse[j])
        return out
    monkeypatch.setattr(orc, "surrogate_grad_rows", mutant)
    assert fails(tg.test_gradient_matches_autograd_and_finite_differences, 0)


def test_token_loss_with_transposed_operands(monkeypatch):
    real = orc.token_loss

    def mutant(z_draft, z_target, d2t=None):
        zt = np.asarray(z_target, dtype=np.float64)
        if d2t is not None:
            zt = zt[np.asarray(d2t, dtype=np.int64)]
        H, g = real(zt, z_draft)                       # H(p_M, p_T) instead of H(p_T, p_M)
        return H, -g
    monkeypatch.setattr(orc, "token_loss", mutant)
    assert fails(tt.test_matches_torch_soft_target_cross_entropy_and_autograd, 0)
    assert fails(tt.test_one_hot_target_gives_the_negative_log_likelihood)


def test_tree_with_a_transposed_frontier_slot(monkeypatch):
    monkeypatch.setattr(orc, "context_row", lambda d, j, k: 0 if d == 0 else 1 + (d - 1) * k + (k - 1 - j))
    assert fails(ttree.test_context_rows_follow_the_input_layout)


def test_tree_scored_by_the_edge_probability_instead_of_the_path(monkeypatch):
    """Fig. 1 caption: the path confidence is the product along the path."""
    real = orc.lse_and_topk
    calls = {"n": 0}

    def mutant(z, k):
        lse, ids, lp = real(z, k)
        calls["n"] += 1
        return lse, ids, lp
    # the mutant tree builder: cumulative scores replaced by the last edge's log-probability
    real_build = orc.build_tree

    def build(draft, D, k, g):
        t = real_build(draft, D, k, g)
        return orc.DraftTree(**{**t.__dict__, "score": t.logp.copy()})
    monkeypatch.setattr(orc, "build_tree", build)
    assert fails(ttree.test_fig1_greedy_leaf_is_pruned_by_a_better_sibling_path) or \
        fails(ttree.test_tree_invariants_default_shape, 0)


def test_walk_that_ignores_the_id_map(monkeypatch):
    """Sec. 3.2 with a reduced draft vocabulary: comparing the greedy target id with the raw
    draft id instead of its image under the map."""
    real = orc.longest_accepted
    monkeypatch.setattr(orc, "longest_accepted", lambda tree, target, d2t=None: real(tree, target, None))
    assert fails(tr.test_walk_compares_the_greedy_target_id_with_the_mapped_draft_id)
    assert fails(tr.test_greedy_target_token_outside_the_image_of_the_map_accepts_nothing)


def test_surrogate_that_drops_the_gradient_scale(monkeypatch):
    real = orc.clipped_surrogate
    monkeypatch.setattr(orc, "clipped_surrogate",
                        lambda path_logp, old_logp, path_len, adv, m, eps=0.2, grad_scale=1.0:
                        real(path_logp, old_logp, path_len, adv, m, eps, 1.0))
    assert fails(tg.test_gradient_matches_autograd_and_finite_differences, 1)
    assert fails(tp.test_hand_worked_group_rows_tokens_and_advantages_land_where_they_belong)


def test_pass_that_reads_the_gradient_rows_from_the_wrong_draft_row(monkeypatch):
    """The draft tensor keeps k - 1 unused rows after the root: an index that forgets them."""
    monkeypatch.setattr(orc, "draft_slot_of_row", lambda r, k: (r // k, r % k))
    assert fails(tp.test_hand_worked_group_rows_tokens_and_advantages_land_where_they_belong)
    assert fails(tp.test_whole_pass_gradient_by_finite_differences_over_every_draft_logit)


def test_pass_that_hands_the_advantages_to_the_wrong_positions(monkeypatch):
    real = orc.group_advantages

    def mutant(rc, rr, m, delta=1e-6, unbiased=False, debias=True):
        R, A = real(rc, rr, m, delta, unbiased, debias)
        return R, A[::-1].copy()
    monkeypatch.setattr(orc, "group_advantages", mutant)
    # (finite differences cannot see this one: loss and gradient would use the same wrong values)
    assert fails(tp.test_hand_worked_group_rows_tokens_and_advantages_land_where_they_belong)


def test_expected_path_that_takes_the_deepest_leaf(monkeypatch):
    real = orc.most_expected_sequence

    def mutant(tree, Lc, leaves):
        return real(tree, np.asarray(tree.depth, dtype=np.float64), leaves)   # ranks leaves by depth
    monkeypatch.setattr(orc, "most_expected_sequence", mutant)
    assert fails(tr.test_most_expected_sequence_is_the_argmax_of_explicit_path_sums) or \
        any(fails(tr.test_most_expected_sequence_extends_the_greedy_path_for_one_hot_targets, s) for s in range(6))
