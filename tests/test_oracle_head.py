"""Pins of the checker's draft-head step against a float64 torch restatement written separately
(library linear layers, library cosine similarity, library top-k), and special cases."""
import numpy as np
import torch

import oracle
from paper_2408_00264_b200 import workloads as W


def t64(bits):
    return torch.from_numpy(W.bf16_bits_to_f64(np.asarray(bits)))


def torch_head_step(h, e, wts, k_top, eps=1e-5):
    F = torch.nn.functional
    h, e = t64(h), t64(e)
    R, H = h.shape
    nh = wts["n_heads"]
    x = h * torch.rsqrt(h.pow(2).mean(-1, keepdim=True) + eps) * t64(wts["norm1"])
    q = F.linear(x, t64(wts["wq"]), t64(wts["bq"]))
    k = F.linear(e, t64(wts["wk"]), t64(wts["bk"]))
    v = F.linear(e, t64(wts["wv"]), t64(wts["bv"]))
    att = F.cosine_similarity(q.view(-1, H // nh), k.view(-1, H // nh), dim=-1).view(R, nh, 1)
    a = h + (v.view(R, nh, H // nh) * att).view(R, H)
    p = F.linear(torch.cat([a, e], dim=1), t64(wts["wfc"]), t64(wts["bfc"]))
    y = p * torch.rsqrt(p.pow(2).mean(-1, keepdim=True) + eps) * t64(wts["norm2"])
    logits = F.linear(y, t64(wts["lm_head"]))
    vals, ids = torch.topk(logits, k_top, dim=-1)
    return p.numpy(), ids.numpy(), vals.numpy(), logits.numpy()


def test_head_step_equals_the_library_restatement():
    for seed, (R, H, nh, V, k) in enumerate([(3, 64, 4, 500, 5), (1, 128, 8, 1000, 8), (5, 96, 3, 333, 1)]):
        h, e, wts = W.make_draft_head(R, H, nh, V, seed=seed + 1)
        p, ids, vals, logits = oracle.draft_head_step(h, e, wts, k)
        p2, ids2, vals2, logits2 = torch_head_step(h, e, wts, k)
        assert np.allclose(p, p2, rtol=1e-11, atol=1e-11)
        assert np.allclose(logits, logits2, rtol=1e-10, atol=1e-10)
        assert np.array_equal(ids, ids2) and np.allclose(vals, vals2, rtol=1e-10, atol=1e-10)
        assert (np.diff(vals, axis=1) <= 0).all()


def test_special_cases():
    R, H, nh, V = 2, 32, 4, 40
    h, e, wts = W.make_draft_head(R, H, nh, V, seed=9)
    one = W.f32_to_bf16_bits(np.array([1.0], np.float32))[0]
    # k = q (same projection, e = RMSNorm(h)): every gate is 1, a = h + v
    wts2 = dict(wts)
    wts2["wk"], wts2["bk"] = wts["wq"], wts["bq"]
    wts2["norm1"] = np.full(H, one, np.uint16)
    h64 = W.bf16_bits_to_f64(h)
    xn = h64 / np.sqrt((h64 * h64).mean(-1, keepdims=True) + 1e-5)
    e2 = W.f32_to_bf16_bits(xn.astype(np.float32))
    # (e2 is xn rounded to bf16, so q and k differ by that rounding only: gates within 1e-4 of 1)
    wts2["wfc"] = np.zeros((H, 2 * H), np.uint16)
    wts2["wfc"][np.arange(H), np.arange(H)] = one            # the projector passes `a` through
    wts2["bfc"] = np.zeros(H, np.uint16)
    p, _, _, _ = oracle.draft_head_step(h, e2, wts2, 1)
    v = W.bf16_bits_to_f64(e2) @ W.bf16_bits_to_f64(wts["wv"]).T + W.bf16_bits_to_f64(wts["bv"])
    assert np.abs(p - (h64 + v)).max() < 2e-2 * np.abs(v).max()
    # a zero value projection leaves the hidden state untouched whatever the gate
    wts3 = dict(wts2)
    wts3["wv"] = np.zeros((H, H), np.uint16)
    wts3["bv"] = np.zeros(H, np.uint16)
    p, _, _, _ = oracle.draft_head_step(h, e, wts3, 1)
    assert np.array_equal(p, h64)
    # ties among the top logits: lower index first
    wts4 = dict(wts)
    wts4["lm_head"] = np.zeros((V, H), np.uint16)
    _, ids, vals, _ = oracle.draft_head_step(h, e, wts4, 3)
    assert ids.tolist() == [[0, 1, 2], [0, 1, 2]] and (vals == 0).all()
