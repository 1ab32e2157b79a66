"""Input generators: tree shapes, sibling distinctness, planted winners, paging tables."""
import numpy as np
import pytest

from paper_2408_00264_b200 import workloads as W


def test_topn_level_sizes():
    # Level populations of the static trees (root + the N-1 best-scored nodes).
    exp = {"C1": [1, 3, 4, 4, 4], "C2": [1, 4, 8, 11, 15, 15, 10],
           "C5": [1, 6, 12, 17, 23, 21, 16, 16, 16]}
    for k, lv in exp.items():
        c = W.CONFIGS[k]
        p = W.tree_topn(c.branching, c.n_nodes)
        assert np.bincount(W.tree_depths(p)).tolist() == lv
        assert p[0] == -1 and all(0 <= p[i] < i for i in range(1, len(p)))
        assert W.tree_depths(p).max() == c.max_depth


def test_topn_bfs_variant_and_random_tree():
    p = W.tree_topn((4, 2, 1, 1), 16, order="bfs")
    assert np.bincount(W.tree_depths(p)).tolist() == [1, 4, 8, 3]
    rng = np.random.default_rng(3)
    for _ in range(20):
        p = W.tree_random(64, 6, rng)
        assert p[0] == -1 and all(0 <= p[i] < i for i in range(1, 64))
        assert W.tree_depths(p).max() <= 6


def test_generate_small_properties():
    cfg = W.small_config(batch=3, n_nodes=20, vocab=500, ctx=(5, 90), paged=True)
    w = W.generate(cfg)
    B, N = cfg.batch, cfg.n_nodes
    assert w.q.shape == (B, N, cfg.n_q_heads, 128) and w.q.dtype == np.uint16
    assert w.logits.shape[2] % 8 == 0
    vals = W.bf16_bits_to_f64(w.logits[..., : cfg.vocab])
    for b in range(B):
        for p in range(N):
            kids = np.flatnonzero(w.parent[b] == p)
            assert len(set(w.tokens[b, kids].tolist())) == len(kids)
        for i in range(N):
            row = vals[b, i].copy()
            top = row[w.winner[b, i]]
            row[w.winner[b, i]] = -np.inf
            assert top - row.max() >= cfg.margin       # unique maximum with the stated margin
            assert top - row.max() < cfg.margin + 0.07  # and no more than one bf16 step above it
    # paging: every sequence owns distinct valid pages covering ctx_len + N tokens
    used = w.block_table[w.block_table >= 0]
    assert len(set(used.tolist())) == len(used) and used.max() < w.n_pages
    for b in range(B):
        need = (int(w.ctx_len[b]) + N + 63) // 64
        assert (w.block_table[b, :need] >= 0).all() and (w.block_table[b, need:] == -1).all()
    assert w.path_cap == max(W.tree_depths(w.parent[b]).max() for b in range(B)) + 1
    w2 = W.generate(cfg)
    assert np.array_equal(w.q, w2.q) and np.array_equal(w.logits, w2.logits)
    assert np.array_equal(w.parent, w2.parent) and np.array_equal(w.block_table, w2.block_table)


def test_c3_algorithmic_bytes_formula():
    c = W.CONFIGS["C3"]
    row = c.n_kv_heads * 128 * 2
    kv = c.batch * 4096 * row * 2
    assert kv == 67108864
    assert c.batch * c.n_nodes * c.vocab * 2 == 65667072


def test_shard_sequences_partition():
    for B in (1, 4, 7, 32):
        for world in (1, 2, 3, 8):
            got = [i for r in range(world) for i in W.shard_sequences(B, r, world)]
            assert got == list(range(B))
