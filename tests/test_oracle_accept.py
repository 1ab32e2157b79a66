"""Pins for the checker's per-node argmax, greedy acceptance walk and KV commit."""
import itertools

import numpy as np
import pytest

from paper_2408_00264_b200 import workloads as W


# ---------------------------------------------------------------- argmax (greedy target, T=0)
def test_argmax_matches_numpy_first_occurrence(oracle):
    rng = np.random.default_rng(1)
    bits = W.f32_to_bf16_bits(rng.standard_normal((37, 1003)).astype(np.float32))
    ld = 1008
    lg = np.zeros((37, ld), np.uint16)
    lg[:, :1003] = bits
    lg[:, 1003:] = W.f32_to_bf16_bits(np.full((37, 5), 100.0, np.float32))  # padding is ignored
    got = oracle.argmax(lg, 1003)
    assert np.array_equal(got, np.argmax(W.bf16_bits_to_f64(bits), axis=1))


def test_argmax_ties_signed_zero_and_edges(oracle):
    V = 64
    base = W.f32_to_bf16_bits(np.full((6, V), -1.0, np.float32))
    one = W.f32_to_bf16_bits(np.array([1.0], np.float32))[0]
    base[0, [9, 3, 50]] = one                  # exact tie: lowest index wins
    base[1, V - 1] = one                       # maximum in the last column
    base[2, 0] = one                           # maximum in the first column
    base[3, :] = 0x8000                        # all -0.0 ...
    base[3, 7] = 0x0000                        # ... and one +0.0: equal, so index 0 wins
    base[4, :] = 0xFF80                        # all -inf: first index
    base[5, 20] = 0x0000
    base[5, 10] = 0x8000                       # -0.0 before +0.0 above negatives: index 10
    got = oracle.argmax(base, V)
    assert got.tolist() == [3, V - 1, 0, 0, 0, 10]


def test_argmax_recovers_planted_winner(oracle):
    w = W.generate(W.small_config(batch=2, n_nodes=16, vocab=777))
    assert np.array_equal(oracle.argmax(w.logits, 777), w.winner)


# ---------------------------------------------------------------- greedy walk
def brute_force_accept(parent, tokens, ids):
    """Enumerate every root-to-leaf path; the accepted prefix of a path ends at the first edge
    whose child token differs from the target's choice at its parent; keep the longest."""
    n = len(parent)
    kids = {i: [c for c in range(n) if parent[c] == i] for i in range(n)}
    leaves = [i for i in range(n) if not kids[i]]
    best = [0]
    for leaf in leaves:
        p = []
        j = leaf
        while j >= 0:
            p.append(j)
            j = parent[j]
        p = p[::-1]
        k = 1
        while k < len(p) and tokens[p[k]] == ids[p[k - 1]]:
            k += 1
        if k > len(best):
            best = p[:k]
    return best


def test_walk_equals_brute_force_on_tiny_trees(oracle):
    rng = np.random.default_rng(7)
    for trial in range(300):
        n = int(rng.integers(1, 13))
        parent = W.tree_random(n, 5, rng)
        vocab = 12                                  # small vocabulary: many chance agreements
        tokens = W._draw_tokens(parent, vocab, rng)
        ids = rng.integers(0, vocab, size=n).astype(np.int32)
        alen, aidx, nxt, st = oracle.accept_walk(parent[None], tokens[None], ids[None], 13)
        ref = brute_force_accept(parent, tokens, ids)
        assert st[0] == 0 and alen[0] == len(ref)
        assert aidx[0, : len(ref)].tolist() == ref and (aidx[0, len(ref):] == -1).all()
        assert nxt[0] == ids[ref[-1]]


def test_walk_closed_forms(oracle):
    n = 9
    parent = W.tree_chain(n)[None]
    tokens = np.arange(100, 100 + n, dtype=np.int32)[None]
    ids = np.full((1, n), 5, np.int32)
    ids[0, :-1] = tokens[0, 1:]                      # every edge agrees
    alen, aidx, nxt, st = oracle.accept_walk(parent, tokens, ids, n)
    assert alen[0] == n and aidx[0].tolist() == list(range(n)) and nxt[0] == 5
    ids2 = np.full((1, n), 7, np.int32)              # nothing agrees: only the root
    alen, aidx, nxt, _ = oracle.accept_walk(parent, tokens, ids2, n)
    assert alen[0] == 1 and aidx[0, 0] == 0 and (aidx[0, 1:] == -1).all() and nxt[0] == 7
    for k in range(0, n - 1):                         # k agreeing edges, then a miss
        ids3 = ids.copy()
        ids3[0, k] = 999
        alen, aidx, nxt, _ = oracle.accept_walk(parent, tokens, ids3, n)
        assert alen[0] == k + 1 and nxt[0] == 999


def test_walk_planted_workload_follows_winners(oracle):
    w = W.generate(W.small_config(batch=4, n_nodes=40, vocab=900, p_accept=0.9))
    alen, aidx, nxt, st = oracle.accept_walk(w.parent, w.tokens, w.winner, w.path_cap)
    assert (st == 0).all() and (alen >= 1).all()
    for b in range(4):
        pth = aidx[b, : alen[b]]
        assert pth[0] == 0
        for a, c in zip(pth[:-1], pth[1:]):
            assert w.parent[b, c] == a and w.tokens[b, c] == w.winner[b, a]
        last = pth[-1]
        kids = np.flatnonzero(w.parent[b] == last)
        assert w.winner[b, last] not in w.tokens[b, kids]
        assert nxt[b] == w.winner[b, last]


def test_walk_error_status(oracle):
    parent = np.array([[-1, 0, 1, 2], [-1, 0, -1, 1], [0, 0, 1, 2], [-1, 0, 3, 1]], np.int32)
    tokens = np.array([[1, 2, 3, 4]] * 4, np.int32)
    ids = np.array([[2, 3, 4, 9]] * 4, np.int32)
    alen, aidx, nxt, st = oracle.accept_walk(parent, tokens, ids, 3)   # path of 4 > capacity 3
    assert st[0] != 0 and alen[0] == 0 and (aidx[0] == -1).all() and nxt[0] == -1
    assert (st[1:] != 0).all() and (alen[1:] == 0).all()
    alen, aidx, nxt, st = oracle.accept_walk(parent[:1], tokens[:1], ids[:1], 4)
    assert st[0] == 0 and alen[0] == 4


# ---------------------------------------------------------------- commit
@pytest.mark.parametrize("paged", [False, True])
def test_commit_rows_and_everything_else_untouched(oracle, paged):
    w = W.generate(W.small_config(batch=3, n_q_heads=4, n_kv_heads=2, ctx=(10, 130), n_nodes=12,
                                  vocab=300, paged=paged, p_accept=0.9))
    ids = oracle.argmax(w.logits, w.cfg.vocab)
    alen, aidx, nxt, _ = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    kc, vc, new_len, st = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen,
                                           w.ctx_len, block_table=w.block_table)
    assert (st == 0).all() and np.array_equal(new_len, w.ctx_len + alen)
    exp_k, exp_v = w.k_cache.copy(), w.v_cache.copy()
    for b in range(3):
        for j in range(alen[b]):
            t = int(w.ctx_len[b]) + j
            if paged:
                exp_k[w.block_table[b, t // 64], t % 64] = w.k_tree[b, aidx[b, j]]
                exp_v[w.block_table[b, t // 64], t % 64] = w.v_tree[b, aidx[b, j]]
            else:
                exp_k[b, t] = w.k_tree[b, aidx[b, j]]
                exp_v[b, t] = w.v_tree[b, aidx[b, j]]
    assert np.array_equal(kc, exp_k) and np.array_equal(vc, exp_v)
    assert not np.array_equal(kc, w.k_cache)


def test_commit_then_decode_equals_decode_on_appended_path(oracle):
    # Equivalence requirement of Sec. 2.1: after the step, attention for a brand-new token over
    # the committed cache equals attention over context + accepted path.
    w = W.generate(W.small_config(batch=2, n_q_heads=4, n_kv_heads=2, ctx=(5, 90), n_nodes=14,
                                  vocab=200, p_accept=0.95))
    ids = oracle.argmax(w.logits, w.cfg.vocab)
    alen, aidx, _, _ = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    assert alen.max() >= 2
    kc, vc, new_len, _ = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen,
                                          w.ctx_len)
    one = W.generate(W.small_config(batch=2, n_q_heads=4, n_kv_heads=2, ctx=1, n_nodes=1,
                                    vocab=16, seed=5))
    root = np.array([[-1]] * 2, np.int32)
    after = oracle.tree_attn(one.q, kc, vc, one.k_tree, one.v_tree, root, new_len, w.scale)[0]
    for b in range(2):
        # the same new token appended as a child of the last accepted node of the old tree
        n_acc = int(alen[b])
        pth = aidx[b, :n_acc]
        q2 = np.concatenate([w.q[b:b + 1, pth], one.q[b:b + 1]], axis=1)
        k2 = np.concatenate([w.k_tree[b:b + 1, pth], one.k_tree[b:b + 1]], axis=1)
        v2 = np.concatenate([w.v_tree[b:b + 1, pth], one.v_tree[b:b + 1]], axis=1)
        par = np.arange(-1, n_acc, dtype=np.int32)[None]
        before = oracle.tree_attn(q2, w.k_cache[b:b + 1], w.v_cache[b:b + 1], k2, v2, par,
                                  w.ctx_len[b:b + 1], w.scale)[0]
        np.testing.assert_allclose(after[b, 0], before[0, n_acc], rtol=1e-13, atol=1e-15)


def test_commit_capacity_errors(oracle):
    w = W.generate(W.small_config(batch=2, n_q_heads=2, n_kv_heads=1, ctx=20, n_nodes=4, vocab=50))
    aidx = np.array([[0, 1, 2], [0, 3, -1]], np.int32)
    alen = np.array([3, 2], np.int32)
    ctx = np.array([w.cap_tokens - 2, 20], np.int32)     # sequence 0 would overflow its rows
    kc, vc, new_len, st = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen,
                                           ctx)
    assert st[0] != 0 and st[1] == 0 and new_len.tolist() == [w.cap_tokens - 2, 22]
    assert np.array_equal(kc[0], w.k_cache[0]) and np.array_equal(vc[0], w.v_cache[0])
    assert np.array_equal(kc[1, 20], w.k_tree[1, 0]) and np.array_equal(kc[1, 21], w.k_tree[1, 3])
    bad = np.array([[0, 9, 2], [0, 3, -1]], np.int32)    # node index outside the tree
    st = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, bad, alen,
                          np.array([3, 3], np.int32))[3]
    assert st[0] != 0 and st[1] == 0
