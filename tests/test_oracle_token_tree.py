"""Pins of the token-tree checker (Sec. 2.1, caption of Fig. 2: speculations merged by prefix
matching) against the definition taken another way: sets of paths, hand-made trees, special cases."""
import numpy as np

from paper_2408_00264_b200 import workloads as W


def paths_of(tokens, parent, n):
    out = {}
    for i in range(1, n):
        path, j = [], i
        while j > 0:
            path.append(int(tokens[j]))
            j = int(parent[j])
        out[i] = tuple(reversed(path))
    return out


def test_hand_made_example(oracle):
    # speculations a-b-c, a-b-d, a-e, f, a-b-c (again) after root r: 6 distinct prefixes
    # depth 1: a (first in candidate 0), f (candidate 3); depth 2: a-b (0), a-e (2);
    # depth 3: a-b-c (0), a-b-d (1)
    a, b, c, d, e, f, r = 10, 11, 12, 13, 14, 15, 99
    cand = np.full((1, 5, 3), -1, dtype=np.int32)
    seqs = [[a, b, c], [a, b, d], [a, e], [f], [a, b, c]]
    for i, s in enumerate(seqs):
        cand[0, i, :len(s)] = s
    lens = np.array([[len(s) for s in seqs]], dtype=np.int32)
    tok, par, n, node_of, st = oracle.build_token_tree(np.array([r]), cand, lens, 10)
    assert st[0] == 0 and n[0] == 7
    assert tok[0].tolist() == [r, a, f, b, e, c, d, -1, -1, -1]
    assert par[0].tolist() == [-1, 0, 0, 1, 1, 3, 3, 0, 0, 0]
    assert node_of[0, 0].tolist() == [1, 3, 5] and node_of[0, 4].tolist() == [1, 3, 5]
    assert node_of[0, 1].tolist() == [1, 3, 6] and node_of[0, 2].tolist() == [1, 4, -1]
    assert node_of[0, 3].tolist() == [2, -1, -1]


def test_nodes_are_exactly_the_distinct_prefixes(oracle):
    root, cand, lens = W.make_candidates(6, 24, 6, 5, seed=3)
    tok, par, n, node_of, st = oracle.build_token_tree(root, cand, lens, 128)
    assert (st == 0).all()
    for b in range(6):
        want = {tuple(int(t) for t in cand[b, c, :d + 1]) for c in range(24) for d in range(int(lens[b, c]))}
        got = paths_of(tok[b], par[b], int(n[b]))
        assert set(got.values()) == want and len(got) == len(want)       # no prefix twice
        assert tok[b, 0] == root[b] and par[b, 0] == -1
        assert all(par[b, i] < i for i in range(1, int(n[b])))            # topological
        depth = [len(got[i]) for i in range(1, int(n[b]))]
        assert depth == sorted(depth)                                     # by depth first
        for p in range(int(n[b])):                                        # distinct sibling tokens
            kids = [int(tok[b, i]) for i in range(1, int(n[b])) if par[b, i] == p]
            assert len(kids) == len(set(kids))
        for c in range(24):                                               # every candidate is a path
            for d in range(6):
                i = int(node_of[b, c, d])
                if d >= lens[b, c]:
                    assert i == -1
                else:
                    assert got[i] == tuple(int(t) for t in cand[b, c, :d + 1])
        assert (tok[b, int(n[b]):] == -1).all() and (par[b, int(n[b]):] == 0).all()


def test_special_cases(oracle):
    # one candidate: a chain; candidates with distinct first tokens: disjoint chains under the root
    cand = np.array([[[5, 6, 7, 8]]], dtype=np.int32)
    tok, par, n, _, st = oracle.build_token_tree(np.array([1]), cand, np.array([[4]]), 8)
    assert n[0] == 5 and par[0, :5].tolist() == [-1, 0, 1, 2, 3] and tok[0, :5].tolist() == [1, 5, 6, 7, 8]
    cand = np.array([[[1, 9], [2, 9], [3, 9]]], dtype=np.int32)
    tok, par, n, _, st = oracle.build_token_tree(np.array([0]), cand, np.array([[2, 2, 2]]), 8)
    assert n[0] == 7 and par[0, :7].tolist() == [-1, 0, 0, 0, 1, 2, 3]
    # repeating every candidate changes nothing; empty candidates add nothing
    root, cand, lens = W.make_candidates(2, 10, 5, 4, seed=8)
    a = oracle.build_token_tree(root, cand, lens, 64)
    cand2 = np.concatenate([cand, cand, np.full((2, 3, 5), -1, np.int32)], axis=1)
    lens2 = np.concatenate([lens, lens, np.zeros((2, 3), np.int32)], axis=1)
    b = oracle.build_token_tree(root, cand2, lens2, 64)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])
    assert np.array_equal(b[3][:, :10], a[3]) and np.array_equal(b[3][:, 10:20], a[3])
    # too many nodes or a bad length: flagged, bare root
    tok, par, n, node_of, st = oracle.build_token_tree(root, cand, lens, 3)
    assert (st == 7).all() and (n == 1).all() and (node_of == -1).all() and (tok[:, 1:] == -1).all()
    lens_bad = lens.copy(); lens_bad[1, 0] = 6
    st = oracle.build_token_tree(root, cand, lens_bad, 64)[4]
    assert st.tolist() == [0, 7]


def test_tree_feeds_the_walk(oracle):
    # the arrays, padding included, are a valid tree for the acceptance walk: following candidate
    # c's tokens as the target's choices accepts exactly candidate c's nodes
    root, cand, lens = W.make_candidates(3, 12, 5, 6, seed=21)
    cap = 64
    tok, par, n, node_of, st = oracle.build_token_tree(root, cand, lens, cap)
    for b in range(3):
        c = int(np.argmax(lens[b]))
        L = int(lens[b, c])
        ids = np.full((1, cap), 10 ** 6, dtype=np.int32)            # a token nobody drafted
        chain = [0] + [int(x) for x in node_of[b, c, :L]]
        for j in range(L):
            ids[0, chain[j]] = cand[b, c, j]
        alen, aidx, nxt, wst = oracle.accept_walk(par[b:b + 1], tok[b:b + 1], ids, 8)
        assert wst[0] == 0 and alen[0] == L + 1 and aidx[0, :L + 1].tolist() == chain
