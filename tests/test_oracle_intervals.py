"""Pins of the checker's interval form of the tree mask (App. A.1): the ancestor relation read off
the labels must be the transitive closure of parent[] (computed here by walking up the tree),
closed forms for chains and stars, and the way back."""
import numpy as np

import oracle
from paper_2408_00264_b200 import workloads as W


def ancestors_by_walking(par):
    n = len(par)
    m = np.zeros((n, n), bool)
    for i in range(n):
        j = i
        while j >= 0:
            m[i, j] = True
            j = par[j]
    return m


def test_labels_give_the_ancestor_relation_and_the_way_back():
    rng = np.random.default_rng(7)
    for n in (1, 2, 5, 17, 64, 128):
        trees = [W.tree_random(n, 6, rng) for _ in range(6)] + [W.tree_chain(n), W.tree_star(n), W.tree_forest(n)]
        par = np.stack(trees).astype(np.int32)
        tin, tout, st = oracle.tree_to_intervals(par)
        assert (st == 0).all()
        for b in range(len(par)):
            want = ancestors_by_walking(par[b])
            got = (tin[b][None, :] <= tin[b][:, None]) & (tin[b][:, None] < tout[b][None, :])
            assert np.array_equal(got, want)
            assert sorted(tin[b].tolist()) == list(range(n))          # a depth-first numbering
        back, st2 = oracle.tree_from_intervals(tin, tout)
        assert (st2 == 0).all() and np.array_equal(back, par)


def test_closed_forms_and_malformed_input():
    n = 9
    tin, tout, _ = oracle.tree_to_intervals(W.tree_chain(n)[None])
    assert tin[0].tolist() == list(range(n)) and tout[0].tolist() == [n] * n
    tin, tout, _ = oracle.tree_to_intervals(W.tree_star(n)[None])
    assert tin[0].tolist() == list(range(n)) and tout[0].tolist() == [n] + list(range(2, n + 1))
    tin, tout, _ = oracle.tree_to_intervals(W.tree_forest(n)[None])
    assert tout[0].tolist() == list(range(1, n + 1))
    _, _, st = oracle.tree_to_intervals(np.array([[-1, 2, 0]], np.int32))
    assert st.tolist() == [7]
    # labels that are no forest in topological order
    bad = [([0, 1, 1], [3, 2, 3]),      # two nodes with the same tin
           ([0, 1, 2], [3, 3, 2]),      # an empty interval
           ([0, 1, 2], [2, 3, 3]),      # overlap without nesting: [0,2) and [1,3)
           ([1, 0, 2], [2, 3, 3])]      # node 1 would be the parent of node 0
    for ti, to in bad:
        par, st = oracle.tree_from_intervals(np.array([ti]), np.array([to]))
        assert st.tolist() == [7] and (par == -1).all()
    # any strictly nested labelling works, not only the canonical one
    par, st = oracle.tree_from_intervals(np.array([[10, 20, 40, 25]]), np.array([[100, 35, 50, 30]]))
    assert st.tolist() == [0] and par[0].tolist() == [-1, 0, 0, 1]
