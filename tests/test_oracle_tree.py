"""Pins for the oracle's tree policy (layer-wise expansion, global top-g prune)."""
import os

import numpy as np
import pytest
from scipy.special import softmax

from oracle import gto_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def node_paths(tree):
    """Token path (root excluded) of every node, through the parent links."""
    out = []
    for n in range(tree.g):
        p, a = [], n
        while a >= 0:
            p.append(int(tree.token[a]))
            a = int(tree.parent[a])
        out.append(tuple(reversed(p)))
    return out


def enumerate_tree(draft, D, k, g):
    """Independent statement of the tree policy in probability space: candidates are
    explicit token paths with confidence = product of edge probabilities; numpy
    lexsort does the ranking.  Only meant for inputs without exact ties."""
    conf = {}                      # path -> confidence
    probs = softmax(draft[0, 0])
    best = np.lexsort((np.arange(probs.size), -probs))[:k]
    frontier = [(int(t),) for t in best]          # slot order = rank order
    for t in best:
        conf[(int(t),)] = probs[t]
    for d in range(2, D + 1):
        layer = []
        for j, path in enumerate(frontier):
            probs = softmax(draft[d - 1, j])
            for t in np.lexsort((np.arange(probs.size), -probs))[:k]:
                child = path + (int(t),)
                conf[child] = conf[path] * probs[t]
                layer.append(child)
        c = np.array([conf[p] for p in layer])
        frontier = [layer[i] for i in np.lexsort((np.arange(len(layer)), -c))[:k]]
    paths = list(conf)
    c = np.array([conf[p] for p in paths])
    keep = np.argsort(-c, kind="stable")[:g]
    return {paths[i]: conf[paths[i]] for i in keep}


@pytest.mark.parametrize("V,D,k,g,seed", [(6, 3, 2, 5, 0), (8, 3, 3, 9, 1), (5, 4, 2, 7, 2),
                                          (8, 2, 3, 4, 3), (7, 3, 3, 21, 4), (16, 4, 3, 10, 5)])
def test_tree_matches_independent_enumeration(V, D, k, g, seed):
    rng = np.random.default_rng(seed)
    draft = rng.normal(size=(D, k, V)) * 2.0
    tree = orc.build_tree(draft, D, k, g)
    want = enumerate_tree(draft, D, k, g)
    got = dict(zip(node_paths(tree), np.exp(tree.score)))
    assert set(got) == set(want)
    for p in want:
        assert abs(got[p] - want[p]) < 1e-12


def check_invariants(tree, draft):
    g, k, D = tree.g, tree.k, tree.D
    # parents precede children; depth and context rows are consistent
    for n in range(g):
        a = int(tree.parent[n])
        assert a < n
        if a < 0:
            assert tree.depth[n] == 1 and tree.ctx_row[n] == 0
        else:
            assert tree.depth[n] == tree.depth[a] + 1
            assert tree.slot[a] >= 0
            assert tree.ctx_row[n] == orc.context_row(int(tree.depth[a]), int(tree.slot[a]), k)
            assert tree.score[n] <= tree.score[a]
            assert abs(tree.score[n] - (tree.score[a] + tree.logp[n])) < 1e-12
        assert np.array_equal(np.flatnonzero(tree.mask[n]),
                              sorted(set([n]) | set(np.flatnonzero(tree.mask[a]) if a >= 0 else [])))
    assert np.all(np.diff(tree.pool) > 0)
    # at most k expanded nodes per depth, and distinct slots
    for d in range(1, D + 1):
        s = tree.slot[(tree.depth == d) & (tree.slot >= 0)]
        assert len(s) <= k and len(set(s)) == len(s)
    # edge log-probabilities are the draft log-softmax of the context row at the token
    for n in range(g):
        r = int(tree.ctx_row[n])
        d, j = (0, 0) if r == 0 else (1 + (r - 1) // k, (r - 1) % k)
        z = draft[d, j]
        assert abs(tree.logp[n] - (z[tree.token[n]] - np.log(np.sum(np.exp(z))))) < 1e-10


@pytest.mark.parametrize("seed", range(5))
def test_tree_invariants_default_shape(seed):
    rng = np.random.default_rng(100 + seed)
    D, k, g, V = 7, 10, 60, 200
    draft = rng.normal(size=(D, k, V)) * 2.5
    tree = orc.build_tree(draft, D, k, g)
    check_invariants(tree, draft)
    assert tree.g == 60 and len(tree.cut_gaps) == (D - 2) + 1


def test_k1_is_the_greedy_chain():
    rng = np.random.default_rng(7)
    D, V = 5, 30
    draft = rng.normal(size=(D, 1, V))
    tree = orc.build_tree(draft, D, 1, D)
    assert list(tree.token) == [int(np.argmax(draft[d, 0])) for d in range(D)]
    assert list(tree.parent) == [-1, 0, 1, 2, 3]
    assert list(tree.depth) == [1, 2, 3, 4, 5]


def test_depth1_is_the_rows_topg():
    rng = np.random.default_rng(8)
    draft = rng.normal(size=(1, 6, 50))
    tree = orc.build_tree(draft, 1, 6, 4)
    assert list(tree.token) == list(np.argsort(-draft[0, 0], kind="stable")[:4])
    assert np.all(tree.parent == -1) and np.all(tree.slot == -1)


def test_g_equal_pool_keeps_everything():
    rng = np.random.default_rng(9)
    D, k, V = 3, 3, 12
    draft = rng.normal(size=(D, k, V))
    P = k + (D - 1) * k * k
    tree = orc.build_tree(draft, D, k, P)
    assert list(tree.pool) == list(range(P))
    check_invariants(tree, draft)


def test_ties_go_to_the_lower_index():
    # constant rows: every candidate of a layer ties; ranks must follow the index
    D, k, V = 3, 2, 4
    draft = np.zeros((D, k, V))
    tree = orc.build_tree(draft, D, k, 5)
    # depth 1: tokens 0,1; depth 2 candidates all tie -> frontier = q 0,1 (children of slot 0)
    # global: depth-1 nodes (log 1/4), then depth-2 in pool order (log 1/16) x3
    assert list(tree.pool) == [0, 1, 2, 3, 4]
    assert list(tree.parent) == [-1, -1, 0, 0, 1]
    assert list(tree.token) == [0, 1, 0, 1, 0]
    assert list(tree.slot) == [0, 1, 0, 1, -1]


def read_fig1():
    edges, conf, kept, pruned = {}, {}, [], []
    with open(os.path.join(GOLDEN, "fig1_example.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split(";")]
            if parts[0] == "kept":
                kept = parts[1:]
            elif parts[0] == "pruned":
                pruned = parts[1:]
            elif len(parts) == 4:
                edges[(parts[0], parts[1])] = float(parts[2])
            else:
                conf[parts[0]] = float(parts[1])
    return edges, conf, kept, pruned


def test_fig1_greedy_leaf_is_pruned_by_a_better_sibling_path():
    """Fig. 1 caption (a): confidence is the product of edge probabilities, and the
    greedy leaf (0.36) loses to the sibling path (0.38) under top-4 re-ranking."""
    edges, conf, kept, pruned = read_fig1()
    vocab = ["is", "has", "a", "the", "to", "been"]
    tid = {w: i for i, w in enumerate(vocab)}
    V, D, k = len(vocab), 2, 2
    tiny = 1e-12

    def row(ctx):
        p = np.full(V, tiny)
        for (c, w), pr in edges.items():
            if c == ctx:
                p[tid[w]] = pr
        return np.log(p / p.sum())

    draft = np.zeros((D, k, V))
    draft[0, 0] = row("It")
    # depth-1 frontier: slot 0 = "is" (0.6), slot 1 = "has" (0.4)
    draft[1, 0] = row("It is")
    draft[1, 1] = row("It has")
    tree = orc.build_tree(draft, D, k, 3)       # 4 nodes with the root = 3 without
    names = {" ".join(["It"] + [vocab[t] for t in p]): s
             for p, s in zip(node_paths(tree), np.exp(tree.score))}
    assert set(names) == set(kept)
    for p in pruned:
        assert p not in names
    for name, c in conf.items():
        if name in names:
            assert abs(names[name] - c) < 1e-9
    # the greedy path is exactly the pruned one
    greedy = ["It", vocab[int(np.argmax(draft[0, 0]))]]
    greedy.append(vocab[int(np.argmax(draft[1, 0]))])
    assert " ".join(greedy) == pruned[0]
    # and it would have scored the printed 0.36
    assert abs(edges[("It", "is")] * edges[("It is", "a")] - conf["It is a"]) < 1e-12


def test_context_rows_follow_the_input_layout():
    """Row 0 is the root context, row 1 + (d-1)k + j the context reached through frontier slot j
    of depth d (the layout of the target tensor [R, V] with R = 1 + (D-1)k): written out for
    D = 3, k = 2."""
    assert [orc.context_row(0, 0, 2)] + [orc.context_row(d, j, 2) for d in (1, 2) for j in (0, 1)] == \
        [0, 1, 2, 3, 4]
    D, k, V = 3, 2, 4
    draft = np.full((D, k, V), -20.0)
    draft[0, 0, [2, 1]] = [3.0, 2.0]            # root: token 2 (slot 0), token 1 (slot 1)
    draft[1, 0, [0, 3]] = [1.0, 0.5]            # under slot 0 of depth 1
    draft[1, 1, [3, 0]] = [1.0, 0.9]            # under slot 1 of depth 1
    draft[2, 0, [1, 2]] = [0.2, 0.1]            # contexts of depth 2, slots 0 and 1
    draft[2, 1, [1, 2]] = [0.2, 0.1]
    tree = orc.build_tree(draft, D, k, 10)      # g = P: every candidate
    assert list(tree.depth) == [1, 1, 2, 2, 2, 2, 3, 3, 3, 3]
    assert list(tree.ctx_row) == [0, 0, 1, 1, 2, 2, 3, 3, 4, 4]
    assert list(tree.token[:6]) == [2, 1, 0, 3, 3, 0]
    # depth-2 frontier: the two best of the four by cumulative score are both under token 2
    assert list(tree.slot[:6]) == [0, 1, 0, 1, -1, -1]
    assert list(tree.parent) == [-1, -1, 0, 0, 1, 1, 2, 2, 3, 3]
