"""Pins for the Draft Tree Reward (Eq. 3-5) and the greedy accepted path."""
import itertools

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import gto_oracle as orc
from test_oracle_tree import node_paths


def tiny_case(seed, V=3, D=3, k=2, g=5, scale=1.5):
    rng = np.random.default_rng(seed)
    draft = rng.normal(size=(D, k, V)) * scale
    target = rng.normal(size=(1 + (D - 1) * k, V)) * scale
    tree = orc.build_tree(draft, D, k, g)
    return draft, target, tree


def rollout_dist(tree, target, prefix):
    """Target next-token distribution after `prefix` (a tuple of tokens): the tree's
    own context row while the prefix is the root or an expanded tree node, else any
    fixed distribution (uniform) - it cannot change a match count any more."""
    V = target.shape[1]
    if len(prefix) == 0:
        return softmax(target[0])
    paths = node_paths(tree)
    if prefix in paths:
        n = paths.index(prefix)
        if tree.slot[n] >= 0 and tree.depth[n] < tree.D:
            return softmax(target[orc.context_row(int(tree.depth[n]), int(tree.slot[n]), tree.k)])
    return np.full(V, 1.0 / V)


def lcp(a, b):
    n = 0
    for x, y in zip(a, b):
        if x != y:
            break
        n += 1
    return n


@pytest.mark.parametrize("seed", range(4))
def test_sequence_length_is_expected_leading_matches_by_enumeration(seed):
    """Eq. 3: L_i is the expected number of leading tokens of S_i that a target
    roll-out reproduces.  Enumerate every roll-out of length D."""
    draft, target, tree = tiny_case(seed)
    p, _ = orc.target_node_probs(tree, target)
    rw = orc.tree_reward(tree, p)
    paths = node_paths(tree)
    V, D = target.shape[1], tree.D
    exp_match = np.zeros(tree.g)
    exp_max = 0.0
    total = 0.0
    leaves = [paths[i] for i in rw["leaves"]]
    for x in itertools.product(range(V), repeat=D):
        pr = 1.0
        for u in range(D):
            pr *= rollout_dist(tree, target, x[:u])[x[u]]
        total += pr
        for n in range(tree.g):
            exp_match[n] += pr * lcp(x, paths[n])
        exp_max += pr * max(lcp(x, s) for s in leaves)
    assert abs(total - 1.0) < 1e-12
    assert np.allclose(exp_match, rw["Lc"], atol=1e-12)
    # exact tree acceptance: E[max_i matches] = sum_n Pp_n, between max L and sum L
    assert abs(exp_max - rw["etree"]) < 1e-12
    L = rw["Lc"][rw["leaves"]]
    assert L.max() - 1e-12 <= rw["etree"] <= L.sum() + 1e-12
    # Eq. 5 with eta = 1 and the App. A Eq. (1) bounds
    assert abs(rw["r"] - logsumexp(L)) < 1e-12
    assert L.max() <= rw["r"] <= L.max() + np.log(len(L)) + 1e-12


def test_sequence_length_by_monte_carlo():
    draft, target, tree = tiny_case(11, V=4, D=3, k=2, g=6)
    p, _ = orc.target_node_probs(tree, target)
    rw = orc.tree_reward(tree, p)
    paths = node_paths(tree)
    rng = np.random.default_rng(0)
    n_roll = 100000
    counts = np.zeros((n_roll, tree.g))
    for i in range(n_roll):
        x = ()
        for u in range(tree.D):
            q = rollout_dist(tree, target, x)
            x = x + (int(rng.choice(len(q), p=q)),)
        counts[i] = [lcp(x, s) for s in paths]
    mean = counts.mean(axis=0)
    sem = counts.std(axis=0) / np.sqrt(n_roll) + 1e-9
    assert np.all(np.abs(mean - rw["Lc"]) < 4.5 * sem)


@pytest.mark.parametrize("n_match", [0, 1, 3, 5])
def test_single_chain_one_hot_reward_counts_matching_tokens(n_match):
    """k = 1, g = D: the tree is one chain; with one-hot target rows the reward is
    the number of leading draft tokens equal to the target's tokens."""
    rng = np.random.default_rng(n_match)
    D, V = 5, 20
    draft = rng.normal(size=(D, 1, V))
    tree = orc.build_tree(draft, D, 1, D)
    target = np.full((D, V), -1000.0)
    for d in range(D):
        tok = int(tree.token[d])
        hot = tok if d < n_match else (tok + 1) % V
        target[d, hot] = 1000.0
    p, _ = orc.target_node_probs(tree, target)
    rw = orc.tree_reward(tree, p)
    assert rw["r"] == pytest.approx(float(n_match), abs=1e-12)
    assert len(rw["leaves"]) == 1
    path = orc.longest_accepted(tree, target)
    assert len(path["nodes"]) == n_match
    assert path["nodes"] == list(range(n_match))


def test_eta_limits_and_variants():
    draft, target, tree = tiny_case(5, V=6, D=4, k=3, g=12)
    p, _ = orc.target_node_probs(tree, target)
    L = orc.tree_reward(tree, p)["Lc"][orc.tree_reward(tree, p)["leaves"]]
    assert orc.tree_reward(tree, p, eta=200.0)["r"] == pytest.approx(L.max(), abs=2e-2)
    small = 1e-5
    assert orc.tree_reward(tree, p, eta=small)["r"] - np.log(len(L)) / small == pytest.approx(L.mean(), abs=1e-3)
    assert orc.tree_reward(tree, p, agg=orc.AGG_MAX)["r"] == L.max()
    assert orc.tree_reward(tree, p, agg=orc.AGG_MEAN)["r"] == pytest.approx(L.mean())
    for eta in (0.5, 1.0, 3.0):
        r = orc.tree_reward(tree, p, eta=eta)["r"]
        assert L.max() <= r <= L.max() + np.log(len(L)) / eta + 1e-12
        assert r == pytest.approx(logsumexp(eta * L) / eta)


def test_reduced_vocabulary_map_is_used_for_the_gather():
    rng = np.random.default_rng(3)
    D, k, g, Vd, Vt = 3, 2, 5, 4, 9
    d2t = np.array([1, 4, 6, 8])
    draft = rng.normal(size=(D, k, Vd))
    target = rng.normal(size=(1 + (D - 1) * k, Vt))
    tree = orc.build_tree(draft, D, k, g)
    p, lse_t = orc.target_node_probs(tree, target, d2t)
    for n in range(g):
        r = int(tree.ctx_row[n])
        assert p[n] == pytest.approx(softmax(target[r])[d2t[tree.token[n]]])
    assert np.all(np.isnan(lse_t) == ~np.isin(np.arange(target.shape[0]), tree.ctx_row))


@pytest.mark.parametrize("seed", range(6))
def test_greedy_path_length_is_max_L_for_one_hot_targets(seed):
    """App. A case (b): at temperature 0 each L_i is the common-prefix length with
    the greedy target trajectory and the accepted length is max_i L_i."""
    rng = np.random.default_rng(50 + seed)
    D, k, g, V = 4, 3, 14, 8
    draft = rng.normal(size=(D, k, V)) * 2
    tree = orc.build_tree(draft, D, k, g)
    R = 1 + (D - 1) * k
    greedy = rng.integers(0, V, size=R)
    # make the target agree with the draft's best token on most rows so paths are long
    for r in range(R):
        d, j = (0, 0) if r == 0 else (1 + (r - 1) // k, (r - 1) % k)
        if rng.random() < 0.8:
            greedy[r] = int(np.argsort(-draft[d, j])[rng.integers(0, 2)])
    target = np.full((R, V), -1000.0)
    target[np.arange(R), greedy] = 1000.0
    p, _ = orc.target_node_probs(tree, target)
    rw = orc.tree_reward(tree, p)
    L = rw["Lc"][rw["leaves"]]
    path = orc.longest_accepted(tree, target)
    assert np.allclose(L, np.round(L))
    assert len(path["nodes"]) == int(round(L.max()))
    # the path is parent-linked with depths 1..l and the reported rows are the contexts
    for j, n in enumerate(path["nodes"]):
        assert tree.depth[n] == j + 1
        assert tree.parent[n] == (path["nodes"][j - 1] if j else -1)
        assert path["rows"][j] == tree.ctx_row[n]
        assert greedy[path["rows"][j]] == tree.token[n]
        assert path["logp"][j] == tree.logp[n]


def test_walk_stops_at_unexpanded_node_and_on_mismatch():
    D, k, V = 3, 2, 4
    draft = np.zeros((D, k, V))
    draft[0, 0] = [5, 4, 0, 0]
    draft[1, 0] = [0, 0, 5, 4]
    draft[1, 1] = [-9, -9, -9, -9.5]
    draft[2, 0] = [1, 0, 0, 0]
    draft[2, 1] = [1, 0, 0, 0]
    tree = orc.build_tree(draft, D, k, 4)
    target = np.zeros((1 + (D - 1) * k, V))
    target[0, 0] = 9        # accepts token 0 at depth 1
    target[1, 3] = 9        # greedy token 3 under slot 0: child (token 3) selected?
    path = orc.longest_accepted(tree, target)
    toks = [int(tree.token[n]) for n in path["nodes"]]
    assert toks[0] == 0
    assert all(tree.parent[b] == a for a, b in zip(path["nodes"], path["nodes"][1:]))
    target[0] = 0
    target[0, 2] = 9        # greedy token not among the root's children
    assert orc.longest_accepted(tree, target)["nodes"] == []


def _worked_tree_with_id_map():
    """D = 3, k = 2, draft vocabulary 4 mapped into a target vocabulary of 9 by (1, 4, 6, 8).
    Worked by hand: the root proposes tokens 0 and 1 (slots 0, 1); under token 0 the draft
    proposes 2 and 3, which outrank both children of token 1 and become slots 0 and 1 of
    depth 2 (context rows 3 and 4); the six best candidates are the pool indices
    0, 1, 2, 3, 6 (path 0-2-0) and 8 (path 0-3-1), listed in that order."""
    D, k = 3, 2
    d2t = np.array([1, 4, 6, 8])
    draft = np.zeros((D, k, 4))
    draft[0, 0] = [5, 4, 0, 0]
    draft[0, 1] = np.nan                       # no context lives here
    draft[1, 0] = [0, 0, 5, 4]
    draft[1, 1] = [-9, -9, -9, -9.5]
    draft[2, 0] = [1, 0, 0, 0]
    draft[2, 1] = [0, 3, 0, 0]
    tree = orc.build_tree(draft, D, k, 6)
    assert list(tree.pool) == [0, 1, 2, 3, 6, 8]
    assert list(tree.token) == [0, 1, 2, 3, 0, 1]
    return tree, d2t


def test_walk_compares_the_greedy_target_id_with_the_mapped_draft_id():
    """Sec. 3.2 / App. A case (b) with a reduced draft vocabulary: the target's greedy token
    is a TARGET id, a child matches when the image of its draft id under the map equals it.
    The greedy ids are chosen so that a walk that compared raw draft ids would go elsewhere:
    at the root the target picks id 1 = map(0), and a child with draft id 1 exists too."""
    tree, d2t = _worked_tree_with_id_map()
    target = np.full((5, 9), -50.0)
    target[0, 1] = 50.0          # map(0): accept token 0 (list position 0)
    target[1, 8] = 50.0          # map(3) in the context of token 0: accept 0-3 (position 3, slot 1)
    target[4, 4] = 50.0          # map(1) in context row 4 = slot 1 of depth 2: accept 0-3-1 (position 5)
    target[2, 4] = 50.0          # rows the walk must not consult
    target[3, 1] = 50.0
    path = orc.longest_accepted(tree, target, d2t)
    assert path["nodes"] == [0, 3, 5]
    assert path["rows"] == [0, 1, 4]
    assert path["tokens"] == [0, 3, 1]           # draft ids, not target ids
    assert path["logp"] == pytest.approx([5 - np.log(np.exp(5) + np.exp(4) + 2),
                                          4 - np.log(np.exp(5) + np.exp(4) + 2),
                                          3 - np.log(np.exp(3) + 3)], abs=1e-12)
    # the identity map on a shared vocabulary is the same thing as no map
    same = orc.longest_accepted(tree, target[:, :4] + 0.0, np.arange(4))
    assert same == orc.longest_accepted(tree, target[:, :4] + 0.0, None)


def test_greedy_target_token_outside_the_image_of_the_map_accepts_nothing():
    """A target id no draft id maps to cannot be drafted: the walk stops, also when a child
    happens to carry that number as its draft id."""
    tree, d2t = _worked_tree_with_id_map()
    target = np.full((5, 9), -50.0)
    target[0, 0] = 50.0          # target id 0 is not in (1, 4, 6, 8); draft id 0 is a child of the root
    assert orc.longest_accepted(tree, target, d2t)["nodes"] == []
    target[0] = -50.0
    target[0, 1] = 50.0          # accept token 0 ...
    target[1, 2] = 50.0          # ... then target id 2: unmapped, while draft id 2 is a child there
    assert orc.longest_accepted(tree, target, d2t)["nodes"] == [0]


def test_all_nodes_variant_sums_over_every_root_to_node_sequence():
    """Independent restatement: walk every node's path with explicit products."""
    draft, target, tree = tiny_case(11, V=6, D=4, k=3, g=12)
    p, _ = orc.target_node_probs(tree, target)
    Ls = []
    for n in range(tree.g):
        chain, x = [], n
        while x >= 0:
            chain.append(x)
            x = int(tree.parent[x])
        chain.reverse()
        Ls.append(sum(np.prod([p[a] for a in chain[:j + 1]]) for j in range(len(chain))))
    got = orc.tree_reward(tree, p, eta=1.3, all_nodes=True)
    assert got["r"] == pytest.approx(logsumexp(1.3 * np.array(Ls)) / 1.3, rel=1e-12)
    assert len(got["leaves"]) == tree.g
    assert got["r"] >= orc.tree_reward(tree, p, eta=1.3)["r"]     # a superset of sequences
    assert orc.tree_reward(tree, p, agg=orc.AGG_MAX, all_nodes=True)["r"] == \
        orc.tree_reward(tree, p, agg=orc.AGG_MAX)["r"]            # the longest paths end in leaves


@pytest.mark.parametrize("seed", range(6))
def test_most_expected_sequence_extends_the_greedy_path_for_one_hot_targets(seed):
    """App. A case (b): with one-hot target rows L_i is the length of the prefix S_i shares with
    the greedy target trajectory, so a sequence of largest L_i starts with the whole greedy
    accepted path and its L equals the accepted length."""
    rng = np.random.default_rng(80 + seed)
    D, k, g, V = 4, 3, 14, 8
    draft = rng.normal(size=(D, k, V)) * 2
    tree = orc.build_tree(draft, D, k, g)
    R = 1 + (D - 1) * k
    greedy = np.array([int(np.argsort(-draft[orc.draft_slot_of_row(r, k)])[rng.integers(0, 2)]) for r in range(R)])
    target = np.full((R, V), -1000.0)
    target[np.arange(R), greedy] = 1000.0
    p, _ = orc.target_node_probs(tree, target)
    rw = orc.tree_reward(tree, p)
    walk = orc.longest_accepted(tree, target)
    best = orc.most_expected_sequence(tree, rw["Lc"], rw["leaves"])
    l = len(walk["nodes"])
    assert best["nodes"][:l] == walk["nodes"] and best["rows"][:l] == walk["rows"]
    assert rw["Lc"][best["nodes"][-1]] == pytest.approx(l, abs=1e-12)
    assert best["nodes"][-1] in rw["leaves"]
    # parent-linked from the root, one node per depth
    assert [int(tree.depth[n]) for n in best["nodes"]] == list(range(1, len(best["nodes"]) + 1))
    assert all(tree.parent[b] == a for a, b in zip(best["nodes"], best["nodes"][1:]))
    assert tree.parent[best["nodes"][0]] == -1


def test_most_expected_sequence_is_the_argmax_of_explicit_path_sums():
    """Independent restatement: every leaf's L by explicit products along its path; the first
    leaf of largest L wins; tokens, rows and log-probabilities are those of its path."""
    draft, target, tree = tiny_case(11, V=6, D=4, k=3, g=12)
    p, _ = orc.target_node_probs(tree, target)
    rw = orc.tree_reward(tree, p)
    chains = {}
    for n in rw["leaves"]:
        chain, x = [], int(n)
        while x >= 0:
            chain.append(x)
            x = int(tree.parent[x])
        chains[int(n)] = chain[::-1]
    L = {n: sum(np.prod([p[a] for a in c[:j + 1]]) for j in range(len(c))) for n, c in chains.items()}
    want = max(sorted(L), key=lambda n: (L[n], -n))
    got = orc.most_expected_sequence(tree, rw["Lc"], rw["leaves"])
    assert got["nodes"] == chains[want]
    assert got["tokens"] == [int(tree.token[n]) for n in chains[want]]
    assert got["rows"] == [int(tree.ctx_row[n]) for n in chains[want]]
    assert got["logp"] == [float(tree.logp[n]) for n in chains[want]]
    # not simply the deepest or the first leaf
    assert len({len(c) for c in chains.values()}) > 1
    # an exact tie goes to the lower list position
    Lc = rw["Lc"].copy()
    a, b = sorted(chains)[:2]
    Lc[a] = Lc[b] = Lc.max() + 1.0
    assert orc.most_expected_sequence(tree, Lc, rw["leaves"])["nodes"][-1] == a
