"""Pins for the oracle's glue: position_forward / group_pass sequence the pinned functions
(Algorithm 1's inner loop) and decide WHICH draft row, token, advantage and position each
gradient row belongs to.  A hand-worked group fixes those by explicit indices, and central
finite differences of the whole pass over every draft logit fix them again without
reference to any index arithmetic."""
import numpy as np
import pytest
from scipy.special import softmax

from oracle import gto_oracle as orc

M, D, K, V, G_NODES = 2, 2, 2, 4, 4
SCALE = 0.5 / 16          # omega / K of App. B


def worked_group(pad=np.nan):
    """Two positions, D = 2, k = 2, V = 4, g = 4 of the 6 candidates.

    Position 0 (current draft): the root row proposes tokens 0 and 1 (slots 0, 1).  The greedy
    target takes token 1, so the walk continues in the context of slot 1 - context row 2,
    stored at draft[.., 1, 1, :] - where the draft proposes 2 and 3 and the target takes 2.
    Accepted path: tokens (1, 2) from context rows (0, 2).  Scores: token 0 -0.38, its child 0
    -1.12, token 1 -1.38, path 1-2 -1.46: those four are kept.
    Position 1: the root proposes 1 and 2; the target takes 1 (slot 0, context row 1, stored at
    draft[.., 1, 0, :]); there the target takes 3, which the draft (0 and 1) does not offer.  Accepted path: token (1) from context row (0)."""
    draft = np.zeros((2, M, D, K, V))
    draft[0, 0, 0, 0] = [3, 2, 0, 0]
    draft[0, 0, 1, 0] = [1, 0, 0, 0]
    draft[0, 0, 1, 1] = [0, 0, 4, 1]
    draft[0, 1, 0, 0] = [0, 5, 1, 0]
    draft[0, 1, 1, 0] = [2.2, 2.1, 2, 0]
    draft[0, 1, 1, 1] = [0, 1, 0, 3]
    # the frozen reference draft: other rows, so that the debiased rewards differ
    draft[1, 0, 0, 0] = [0, 0, 3, 2]
    draft[1, 0, 1, 0] = [0, 2, 0, 0]
    draft[1, 0, 1, 1] = [1, 0, 0, 2]
    draft[1, 1, 0, 0] = [1, 4, 0, 0]
    draft[1, 1, 1, 0] = [0, 0, 0, 2]
    draft[1, 1, 1, 1] = [2, 0, 1, 0]
    draft += 1e-3 * np.arange(V)[::-1]        # no exact ties: a small step never changes a tree
    target = np.zeros((2, M, 1 + (D - 1) * K, V))
    target[:, 0, 0] = [0, 2.0, 0.5, 0]        # position 0, root: greedy token 1
    target[:, 0, 1] = [1.5, 0, 0, 0.2]
    target[:, 0, 2] = [0, 0.3, 1.7, 0]        # context of slot 1: greedy token 2
    target[:, 1, 0] = [0.1, 1.2, 0.9, 0]      # position 1, root: greedy token 1
    target[:, 1, 1] = [0, 0.4, 0, 1.1]        # context of slot 0: greedy token 3 (not offered)
    target[:, 1, 2] = [0.6, 0, 0, 0]
    draft[:, :, 0, 1] = pad                   # no context lives in [.., 0, 1:, :]
    old = np.array([[-1.6, -0.2], [-0.1, 0.0]])   # old-policy log-probabilities of the paths
    return draft, target, old


def run(draft, target, old, **kw):
    return orc.group_pass(draft, target, D, K, G_NODES, M, lambda *a: old, delta=1e-6, eps=0.2,
                          grad_scale=SCALE, **kw)


def test_hand_worked_group_rows_tokens_and_advantages_land_where_they_belong():
    draft, target, old = worked_group()
    out = run(draft, target, old)
    assert list(out["path_len"]) == [2, 1]
    assert out["path_row"].tolist() == [[0, 2], [0, -1]]
    assert out["path_token"].tolist() == [[1, 2], [1, -1]]
    lp = lambda z, t: z[t] - np.log(np.sum(np.exp(z)))
    want_logp = [[lp(draft[0, 0, 0, 0], 1), lp(draft[0, 0, 1, 1], 2)], [lp(draft[0, 1, 0, 0], 1), 0.0]]
    assert np.allclose(out["path_logp"], want_logp, atol=1e-12)
    # Eq. 9-10 on the two positions: with m = 2 the standardised values are +-1 (up to delta),
    # signed by which position gained more over its reference tree
    r = np.array([[f["rewards"][t]["r"] for t in range(2)] for f in out["fwd"]])
    Rdeb = r[:, 0] - r[:, 1]
    assert np.allclose(out["R"], Rdeb, atol=1e-15)
    half = abs(Rdeb[0] - Rdeb[1]) / 2
    assert np.allclose(out["A"], np.sign(Rdeb - Rdeb.mean()) * half / (half + 1e-6), atol=1e-12)
    # Eq. 11: length-normalised ratios; both inside the clip range here
    s = np.exp([(want_logp[0][0] + want_logp[0][1] - old[0].sum()) / 2, want_logp[1][0] - old[1, 0]])
    assert np.allclose(out["sur"]["ratio"], s, atol=1e-12)
    assert out["sur"]["active"].all() and np.all(np.abs(s - 1) < 0.2)
    coeff = SCALE * (-1.0 / M) * out["A"] * s / np.array([2, 1])
    # the gradient rows, by explicit position in the draft tensor
    want = np.zeros((M, D, V))
    want[0, 0] = coeff[0] * (np.eye(V)[1] - softmax(draft[0, 0, 0, 0]))
    want[0, 1] = coeff[0] * (np.eye(V)[2] - softmax(draft[0, 0, 1, 1]))
    want[1, 0] = coeff[1] * (np.eye(V)[1] - softmax(draft[0, 1, 0, 0]))
    assert np.allclose(out["grad"], want, atol=1e-12)
    assert np.all(out["grad"][1, 1] == 0.0)
    assert out["sur"]["loss"][0] == pytest.approx(-(s * out["A"]).sum() / M, abs=1e-12)


def test_whole_pass_gradient_by_finite_differences_over_every_draft_logit():
    """The summed group loss is a smooth function of the current draft's logits while the
    trees stay the same; its derivative must be the reported rows scattered to the draft rows
    their path_row names, and zero everywhere else (also on the rows of the reference draft)."""
    draft, target, old = worked_group(pad=0.0)
    base = run(draft, target, old)
    h = 1e-6

    def total(dr):
        out = run(dr, target, old)
        for f, f0 in zip(out["fwd"], base["fwd"]):          # the step is small: same trees
            assert all(np.array_equal(a.pool, b.pool) and np.array_equal(a.token, b.token)
                       for a, b in zip(f["trees"], f0["trees"]))
        return SCALE * out["sur"]["loss"].sum()

    scattered = np.zeros_like(draft)
    for i in range(M):
        for j in range(base["path_len"][i]):
            r = int(base["path_row"][i, j])
            d, slot = (0, 0) if r == 0 else (1 + (r - 1) // K, (r - 1) % K)
            scattered[0, i, d, slot] = base["grad"][i, j]
    for idx in np.ndindex(draft.shape):
        up, dn = draft.copy(), draft.copy()
        up[idx] += h
        dn[idx] -= h
        fd = (total(up) - total(dn)) / (2 * h)
        assert abs(fd - scattered[idx]) < 1e-8, (idx, fd, scattered[idx])


def test_position_forward_uses_each_trees_own_rows():
    """Tree t is built from draft[t] and scored on target[t]; the accepted path is walked on
    the current draft's tree (t = 0) with the current target rows."""
    draft, target, _ = worked_group(pad=0.0)
    target = target.copy()
    target[1] = target[1][:, :, ::-1]                      # the reference tree sees other rows
    f = orc.position_forward(draft[:, 0], target[:, 0], D, K, G_NODES)
    for t in range(2):
        tree = orc.build_tree(draft[t, 0], D, K, G_NODES)
        assert np.array_equal(f["trees"][t].token, tree.token)
        p, _ = orc.target_node_probs(tree, target[t, 0])
        assert f["rewards"][t]["r"] == orc.tree_reward(tree, p)["r"]
    assert f["path"] == orc.longest_accepted(f["trees"][0], target[0, 0])
    assert f["path"] != orc.longest_accepted(f["trees"][0], target[1, 0])
