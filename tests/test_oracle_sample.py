"""Pins of the CPU checker's stochastic acceptance (temperature > 0).

The paper adopts its baseline's tree sampling algorithm and prints no formula (Sec. 4.1, Table 1
lower half), so nothing here compares the checker with itself: the pins are what the mathematics
fixes.  Speculative sampling must leave the target's distribution untouched, hence the probability
of every outcome (accepted path, next token) is the product of the target's conditional
probabilities along it - a closed form that knows nothing of the accept/reject sequence.
"""
import itertools

import numpy as np
import pytest

import oracle
from paper_2408_00264_b200 import workloads as W


def bits(x):
    b = W.f32_to_bf16_bits(np.atleast_1d(np.asarray(x, np.float32)))
    return int(b[0]) if np.ndim(x) == 0 else b


def softmax64(row_bits, temperature=1.0):
    x = W.bf16_bits_to_f64(row_bits) / temperature
    e = np.exp(x - x.max())
    return e / e.sum()


def outcome_probabilities(parent, tokens, logits_bits, temperature):
    """{(path tuple, next token): probability}: the target's conditionals multiplied along the path
    (written from the theorem, not from the algorithm).  A path ends at a node when the emitted
    token is none of its children's tokens."""
    n = len(parent)
    out = {}

    def rec(node, path, prob):
        p = softmax64(logits_bits[node], temperature)
        kids = [c for c in range(node + 1, n) if parent[c] == node]
        taken = set()
        for c in kids:
            if tokens[c] in taken:
                continue
            taken.add(tokens[c])
            rec(c, path + (c,), prob * p[tokens[c]])
        for v in range(len(p)):
            if v not in taken and p[v] > 0:
                out[(path, v)] = out.get((path, v), 0.0) + prob * p[v]
    rec(0, (0,), 1.0)
    return out


@pytest.mark.parametrize("seed,temperature", [(0, 1.0), (1, 1.0), (2, 0.7), (3, 1.6)])
def test_outcomes_follow_the_targets_distribution(seed, temperature):
    rng = np.random.default_rng(100 + seed)
    n, vocab, ld, draws = 6, 5, 8, 120_000
    parent = np.array([-1, 0, 0, 1, 1, 2], np.int32) if seed % 2 == 0 else np.array([-1, 0, 1, 2, 0, 0], np.int32)
    tokens = np.zeros(n, np.int32)
    for node in range(n):   # distinct tokens among siblings
        sib = [c for c in range(n) if parent[c] == node]
        tokens[sib] = rng.permutation(vocab)[:len(sib)]
    lg = np.zeros((n, ld), np.uint16)
    lg[:, :vocab] = bits(rng.normal(0, 1.5, size=(n, vocab)))
    lg[:, vocab:] = 0x7F00   # padding beyond the vocabulary must be ignored
    expect = outcome_probabilities(parent, tokens, lg[:, :vocab], temperature)
    assert abs(sum(expect.values()) - 1.0) < 1e-12
    u = rng.random((draws, n + 1), dtype=np.float32)
    alen, aidx, nxt, status, _ = oracle.accept_sample(np.broadcast_to(lg, (draws, n, ld)), vocab,
                                                      np.broadcast_to(parent, (draws, n)),
                                                      np.broadcast_to(tokens, (draws, n)), u, temperature, n)
    assert (status == 0).all() and (alen >= 1).all()
    counts = {}
    for i in range(draws):
        key = (tuple(int(x) for x in aidx[i, :alen[i]]), int(nxt[i]))
        counts[key] = counts.get(key, 0) + 1
    assert set(counts) <= set(expect), "an outcome of probability zero was produced"
    chi2, dof = 0.0, 0
    for key, pr in expect.items():
        e = pr * draws
        if e < 5:
            continue
        chi2 += (counts.get(key, 0) - e) ** 2 / e
        dof += 1
    # chi-square with dof degrees of freedom: mean dof, variance 2 dof; five standard deviations
    assert chi2 < dof + 5.0 * np.sqrt(2.0 * dof), (chi2, dof)
    # the first emitted token alone (accepted child's token or the drawn one): the root's softmax
    first = np.where(alen > 1, tokens[aidx[:, 1].clip(0)], nxt)
    freq = np.bincount(first, minlength=vocab) / draws
    p0 = softmax64(lg[0, :vocab], temperature)
    assert np.abs(freq - p0).max() < 5.0 * np.sqrt(0.25 / draws)


def test_low_temperature_is_the_greedy_walk():
    for seed in range(20):
        cfg = W.small_config(batch=3, n_nodes=12, vocab=50, seed=W.BASE_SEED + 900 + seed)
        w = W.generate(cfg)   # every row has a winner that leads by at least 0.5
        ids = oracle.argmax(w.logits, cfg.vocab)
        alen, aidx, nxt, st = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
        u = np.random.default_rng(seed).random((3, 13), dtype=np.float32)
        a2, i2, n2, s2, _ = oracle.accept_sample(w.logits, cfg.vocab, w.parent, w.tokens, u, 1e-3, w.path_cap)
        assert np.array_equal(alen, a2) and np.array_equal(aidx, i2) and np.array_equal(nxt, n2)
        assert np.array_equal(st, s2)


def test_certain_and_impossible_drafts_and_the_final_draw():
    n, vocab, ld = 5, 16, 16
    parent = np.array([[-1, 0, 1, 2, 3]], np.int32)          # a chain
    tokens = np.array([[3, 7, 1, 9, 4]], np.int32)
    lg = np.full((1, n, ld), bits(-60.0), np.uint16)
    for node in range(n - 1):                                # each node is sure of its child's token
        lg[0, node, tokens[0, node + 1]] = bits(60.0)
    lg[0, n - 1, 11] = bits(60.0)
    u = np.full((1, n + 1), 0.999999, np.float32)
    alen, aidx, nxt, st, _ = oracle.accept_sample(lg, vocab, parent, tokens, u, 1.0, n)
    assert alen.tolist() == [n] and aidx[0].tolist() == [0, 1, 2, 3, 4] and nxt.tolist() == [11]
    # a drafted token the target gives no probability: never accepted, never drawn afterwards
    lg2 = np.zeros((1, 2, ld), np.uint16)                    # uniform target ...
    lg2[0, 0, 5] = 0xFF80                                    # ... except token 5: -inf
    for uu in np.linspace(0.0, 0.9999, 37, dtype=np.float32):
        a, i, nx, s, _ = oracle.accept_sample(lg2, vocab, np.array([[-1, 0]], np.int32), np.array([[2, 5]], np.int32),
                                              np.array([[0.0, 0.0, uu]], np.float32), 1.0, 2)
        assert a.tolist() == [1] and nx[0] != 5
        # the remaining 15 tokens are equally likely: the draw is the inverse of the running sum
        rest = [v for v in range(vocab) if v != 5]
        assert nx[0] == rest[min(14, int(np.floor(float(uu) * 15 + 1e-9)))]
    # the accept test is strict: u = p exactly is a rejection, anything below it an acceptance
    lg3 = np.zeros((1, 2, ld), np.uint16)
    lg3[0, :, 2:vocab] = 0xFF80                              # two tokens of probability 1/2 each
    par, tok = np.array([[-1, 0]], np.int32), np.array([[0, 1]], np.int32)
    a, _, nx, _, mg = oracle.accept_sample(lg3, vocab, par, tok, np.array([[0, 0.5, 0.3]], np.float32), 1.0, 2)
    assert a.tolist() == [1] and nx.tolist() == [0] and mg[0, 0] == 0.0
    a, _, _, _, mg = oracle.accept_sample(lg3, vocab, par, tok, np.array([[0, 0.4990, 0.3]], np.float32), 1.0, 2)
    assert a.tolist() == [2] and abs(mg[0, 0] - 0.001) < 1e-6


def test_rejected_tokens_are_struck_before_the_next_sibling():
    # three children carrying tokens of probability 1/2, 1/4, 1/8 (and 1/8 left): after the first
    # is rejected the second is accepted below 1/2, after both below 1/2 again
    vocab, ld = 4, 8
    row = bits(np.log([0.5, 0.25, 0.125, 0.125]))
    lg = np.zeros((1, 4, ld), np.uint16)
    lg[0, :, :vocab] = row
    lg[0, :, vocab:] = 0xFF80
    par = np.array([[-1, 0, 0, 0]], np.int32)
    tok = np.array([[0, 0, 1, 2]], np.int32)
    def run(u1, u2, u3, uf):
        a, i, nx, _, _ = oracle.accept_sample(lg, vocab, par, tok, np.array([[0, u1, u2, u3, uf]], np.float32), 1.0, 2)
        return int(a[0]), int(i[0, 1]), int(nx[0])
    assert run(0.49, 0.9, 0.9, 0.0)[:2] == (2, 1)
    assert run(0.51, 0.49, 0.9, 0.0)[:2] == (2, 2)           # 0.25 / (1 - 0.5) = 0.5
    assert run(0.51, 0.51, 0.49, 0.0)[:2] == (2, 3)          # 0.125 / (1 - 0.75) = 0.5
    assert run(0.51, 0.51, 0.51, 0.7) == (1, -1, 3)          # only token 3 is left


def test_malformed_trees_are_reported():
    lg = np.zeros((2, 3, 8), np.uint16)
    par = np.array([[-1, 0, 1], [-1, 2, 0]], np.int32)       # second: parent after child
    tok = np.zeros((2, 3), np.int32)
    u = np.zeros((2, 4), np.float32)
    a, i, nx, st, _ = oracle.accept_sample(lg, 8, par, tok, u, 1.0, 3)
    assert st.tolist() == [0, 7] and a[1] == 0 and nx[1] == -1 and (i[1] == -1).all()
