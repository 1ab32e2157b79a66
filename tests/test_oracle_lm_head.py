"""Pins of the LM-head + greedy-choice checker (Sec. 3.1 + Sec. 4.2) against things it does not
compute itself: a float64 library matrix product, a closed form, and planted rounding ties."""
import numpy as np

from paper_2408_00264_b200 import workloads as W


def bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_logits_equal_a_library_matrix_product(oracle):
    h, w, _ = W.make_lm_head(9, 192, 700, seed=11, planted=0.0)
    ids, z = oracle.lm_head_argmax(h, w, want_logits=True)
    ref = W.bf16_bits_to_f64(h) @ W.bf16_bits_to_f64(w).T
    assert np.abs(z - ref).max() < 1e-12
    # wherever the best logit leads by more than a bf16 step the choice is numpy's
    top2 = np.sort(ref, axis=1)[:, -2:]
    clear = (top2[:, 1] - top2[:, 0]) > np.abs(top2[:, 1]) * 2.0 ** -6
    assert clear.any()
    assert np.array_equal(ids[clear], ref.argmax(axis=1)[clear])
    sel = np.array([7, 0, 3], dtype=np.int32)
    assert np.array_equal(oracle.lm_head_argmax(h, w, rows=sel), ids[sel])


def test_one_hot_weights_pick_the_largest_hidden_entry(oracle):
    # weight row v = unit vector e_(perm[v]): logit[v] = hidden[perm[v]] exactly
    K, V = 64, 64
    rng = np.random.default_rng(5)
    perm = rng.permutation(K)
    w = np.zeros((V, K), dtype=np.float32)
    w[np.arange(V), perm] = 1.0
    hid = W.bf16_bits_to_f32(bits(rng.standard_normal((5, K))))
    ids = oracle.lm_head_argmax(bits(hid), bits(w))
    expect = np.array([int(np.argmax(hid[r, perm])) for r in range(5)])
    assert np.array_equal(ids, expect)


def test_equal_rows_and_rounding_ties_go_to_the_lowest_index(oracle):
    hid = bits([[1.0, 1.0]])
    # logits 1 + 2^-9 and 1 + 3 * 2^-10 both round to bf16 1.0: the first wins although the
    # second is larger before rounding
    w = bits([[1.0, 2.0 ** -9], [1.0, 3 * 2.0 ** -10]])
    ids, z = oracle.lm_head_argmax(hid, w, want_logits=True)
    assert z[0, 1] > z[0, 0] and ids[0] == 0
    # a logit that survives the rounding beats them
    w3 = bits([[1.0, 2.0 ** -9], [1.0, 3 * 2.0 ** -10], [1.0, 2.0 ** -7], [1.0, 2.0 ** -7]])
    assert oracle.lm_head_argmax(hid, w3)[0] == 2
    # negative logits and an all-equal row
    assert oracle.lm_head_argmax(bits([[-1.0, 0.0]]), bits([[2.0, 0.0], [1.0, 0.0], [1.0, 5.0]]))[0] == 1
    assert oracle.lm_head_argmax(bits([[0.0, 0.0]]), bits([[2.0, 1.0], [1.0, 3.0]]))[0] == 0


def test_planted_winner_is_found(oracle):
    h, w, win = W.make_lm_head(12, 128, 3000, seed=3)
    assert np.array_equal(oracle.lm_head_argmax(h, w), win)
