"""Pins for the oracle's continuous verification tree (Section 3.2, Figure 3).

Expected values come from the example the paper describes (tests/golden/figure3_tree.txt), from an independent Python
construction of the same "vertical first, then horizontal" shape (workloads.tree_from_branching, which shares no code
with the oracle) combined with a library sort, and from structural facts any such tree must satisfy."""
import os

import numpy as np
import pytest

import oracle
from paper_2506_14158_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "figure3_tree.txt")


def _random_probs(rng, B, T, V):
    x = rng.standard_normal((B, T, V)) * 2
    e = np.exp(x - x.max(-1, keepdims=True))
    return (e / e.sum(-1, keepdims=True)).astype(np.float32)


def test_the_example_of_figure_3():
    nodes = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    words = [w for w, _, _ in nodes]
    V, T = len(words), len(words)
    # a drafter whose distributions rank the continuations as the figure does; every other token gets less mass
    q = np.full((1, T, V), 1e-3, dtype=np.float32)
    bfs = {}  # the figure lists the nodes breadth-first: node index = line number
    for i, (w, p, rank) in enumerate(nodes):
        bfs[w] = i
    for w, p, rank in nodes[1:]:
        q[0, bfs[p], words.index(w)] = 0.6 / int(rank)
    r = oracle.build_tree(q, [2, 3], [words.index("The")])
    assert r["n_nodes"][0] == 9
    got = [(words[r["tokens"][0, i]], "-" if r["parent"][0, i] < 0 else words[r["tokens"][0, r["parent"][0, i]]]) for i in range(9)]
    assert got == [(w, p) for w, p, _ in nodes]
    assert r["position"][0].tolist() == [0, 1, 1, 2, 2, 2, 2, 2, 2]


@pytest.mark.parametrize("branching,T", [((3, 2, 1), 15), ((4, 3, 2, 2, 1), 26), ((2, 2, 2, 2), 31), ((2, 2, 2, 2), 20),
                                         ((1, 1, 1, 1, 1), 6), ((5,), 6), ((8, 1), 128), ((3, 3, 3), 4), ((2, 3), 1)])
def test_shape_and_tokens_match_an_independent_construction(branching, T):
    rng = np.random.default_rng(len(branching) * 100 + T)
    B, V = 3, 97
    q = _random_probs(rng, B, T, V)
    root = rng.integers(0, V, B).astype(np.int32)
    L = np.array([0, 1000, 77], dtype=np.int32)
    r = oracle.build_tree(q, branching, root, L)
    want_parent = W.tree_from_branching(branching, T)  # python lists, written separately from the oracle
    n = len(want_parent)
    depth = W.tree_depths(want_parent)
    for b in range(B):
        assert r["n_nodes"][b] == n
        np.testing.assert_array_equal(r["parent"][b, :n], want_parent)
        assert (r["parent"][b, n:] == -1).all() and (r["tokens"][b, n:] == 0).all()
        np.testing.assert_array_equal(r["position"][b, :n], L[b] + depth)
        assert r["tokens"][b, 0] == root[b]
        for u in range(n):
            kids = W.children_of(want_parent, u)
            top = np.argsort(-q[b, u].astype(np.float64), kind="stable")[: len(kids)]  # library sort, ties to the lower index
            np.testing.assert_array_equal(r["tokens"][b, kids], top)


def test_structural_invariants():
    rng = np.random.default_rng(9)
    for _ in range(30):
        D = int(rng.integers(1, 7))
        branching = [int(x) for x in rng.integers(1, 5, D)]
        T = int(rng.integers(1, 129))
        q = _random_probs(rng, 1, T, 50)
        r = oracle.build_tree(q, branching, [7])
        n = int(r["n_nodes"][0])
        par, tok = r["parent"][0, :n], r["tokens"][0, :n]
        assert par[0] == -1 and all(0 <= par[i] < i for i in range(1, n))          # topological, root first
        assert all(par[i] <= par[i + 1] for i in range(1, n - 1))                    # breadth-first: siblings contiguous
        depth = W.tree_depths(par)
        assert depth.max(initial=0) <= D and all(depth[i] <= depth[i + 1] for i in range(n - 1))
        full = 1 + sum(int(np.prod(branching[: l + 1])) for l in range(D))
        assert n == min(T, full)
        for u in range(n):
            kids = W.children_of(par, u)
            assert len(kids) <= (branching[depth[u]] if depth[u] < D else 0)
            if kids:
                assert tok[kids[0]] == int(np.argmax(q[0, u]))                       # first sibling = the top-1 choice
                assert len(set(tok[kids].tolist())) == len(kids)                     # alternatives are distinct tokens
                p = q[0, u, tok[kids]]
                assert all(p[j] >= p[j + 1] for j in range(len(kids) - 1))           # in rank order
                rest = np.delete(q[0, u], tok[kids])
                assert rest.size == 0 or rest.max() <= p[-1]                         # nothing more probable was left out
        if n == full and D > 0:  # untruncated: the vertical chain of top-1 choices reaches depth D
            u = 0
            for _l in range(D):
                u = W.children_of(par, u)[0]
            assert depth[u] == D


def test_chain_and_star_reduce_to_argmax_and_topk():
    rng = np.random.default_rng(3)
    q = _random_probs(rng, 2, 6, 40)
    r = oracle.build_tree(q, [1, 1, 1, 1, 1], [5, 6])
    for b in range(2):
        assert r["parent"][b].tolist() == [-1, 0, 1, 2, 3, 4]
        assert r["tokens"][b, 1:].tolist() == [int(np.argmax(q[b, i])) for i in range(5)]
    r = oracle.build_tree(q, [5], [5, 6])
    for b in range(2):
        assert r["parent"][b].tolist() == [-1, 0, 0, 0, 0, 0]
        assert r["tokens"][b, 1:].tolist() == np.argsort(-q[b, 0], kind="stable")[:5].tolist()


def test_equal_probabilities_go_to_the_lower_token():
    q = np.zeros((1, 4, 10), dtype=np.float32)
    q[0, 0, [7, 2, 5]] = 0.25   # three equal maxima
    q[0, 0, 9] = 0.25
    r = oracle.build_tree(q, [3], [0])
    assert r["tokens"][0].tolist() == [0, 2, 5, 7]


def test_bad_arguments():
    q = np.full((1, 3, 4), 0.25, dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.build_tree(q, [0], [0])       # a node must get at least one child
    with pytest.raises(ValueError):
        oracle.build_tree(q, [5], [0])       # more alternatives than tokens
