"""Why the attention tolerance is read per output row.

The stated tolerance of the verify step is "max-abs 2e-2 and max-rel 1e-2" for a bf16 output
computed with fp32 accumulation.  This file restates that arithmetic in numpy - scores and
exponentials in float32, the probabilities rounded to bf16 before the P.V product, float32
accumulation, one rounding of the normalised result to bf16 - and compares it with the CPU
checker's float64 result.  No kernel is involved: the numbers below are what ANY implementation
of the stated precision produces.

Two readings of "max-rel" are evaluated on the same data:
  row-normalised   max over output rows of  max|err| / max|ref|           (the one the tests use)
  element-wise     max over elements of |err| / max(|ref|, row max / 64)  (floored ratio)
Rounding a probability to bf16 perturbs every output element of the row by an amount proportional
to the row's scale, not to the element, so the element-wise ratio of the stated arithmetic itself
exceeds 1e-2 by an order of magnitude while the row-normalised one stays below it.
"""
import numpy as np
import pytest

from paper_2408_00264_b200 import workloads as W
from parity_util import ATTN_MAX_ABS, ATTN_MAX_REL, log_parity


def stated_arithmetic(w):
    """Tree attention in the stated precision; returns bf16 bit patterns [B, N, Hq, D]."""
    c = w.cfg
    B, N, Hq, Hkv, D = c.batch, c.n_nodes, c.n_q_heads, c.n_kv_heads, c.head_dim
    G = Hq // Hkv
    f32 = W.bf16_bits_to_f32
    out = np.zeros((B, N, Hq, D), dtype=np.uint16)
    scale_log2 = np.float32(w.scale * 1.4426950408889634)
    for b in range(B):
        L = int(w.ctx_len[b])
        anc = np.zeros((N, N), dtype=bool)          # row i: i and its ancestors
        for i in range(N):
            j = i
            while j >= 0:
                anc[i, j] = True
                j = int(w.parent[b, j])
        for g in range(Hkv):
            if w.block_table is None:
                kc, vc = f32(w.k_cache[b, :L, g]), f32(w.v_cache[b, :L, g])
            else:
                t = np.arange(L)
                pg = w.block_table[b, t // 64]
                kc, vc = f32(w.k_cache[pg, t % 64, g]), f32(w.v_cache[pg, t % 64, g])
            K = np.concatenate([kc, f32(w.k_tree[b, :, g])]).astype(np.float32)
            V = np.concatenate([vc, f32(w.v_tree[b, :, g])]).astype(np.float32)
            for hq in range(G):
                h = g * G + hq
                q = f32(w.q[b, :, h]).astype(np.float32)                 # [N, D]
                s = (q @ K.T).astype(np.float32) * scale_log2            # float32 scores, log2 domain
                allowed = np.concatenate([np.ones((N, L), bool), anc], axis=1)
                s = np.where(allowed, s, np.float32(-np.inf))
                m = s.max(axis=1, keepdims=True)
                p = np.exp2((s - m).astype(np.float32)).astype(np.float32)
                l = p.sum(axis=1, dtype=np.float32)                      # row sum of the float32 values
                p16 = f32(W.f32_to_bf16_bits(p)).astype(np.float32)      # P enters the product as bf16
                o = (p16 @ V).astype(np.float32) / l[:, None]
                out[b, :, h] = W.f32_to_bf16_bits(o.astype(np.float32))
    return out


def both_readings(got_bits, ref):
    got = W.bf16_bits_to_f64(got_bits)
    err = np.abs(got - ref)
    row_max = np.abs(ref).max(axis=-1, keepdims=True)
    row_rel = (err.max(axis=-1, keepdims=True) / row_max).max()
    floored = (err / np.maximum(np.abs(ref), row_max / 64.0)).max()
    return float(err.max()), float(row_rel), float(floored)


CASES = {
    "C1": lambda: W.CONFIGS["C1"],
    "small-gqa": lambda: W.small_config(batch=2, n_q_heads=8, n_kv_heads=2, ctx=(200, 900), n_nodes=40,
                                        vocab=64, seed=W.BASE_SEED + 501),
    "small-paged": lambda: W.small_config(batch=2, n_q_heads=4, n_kv_heads=4, ctx=(64, 2000), n_nodes=24,
                                          vocab=64, paged=True, seed=W.BASE_SEED + 502),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_stated_arithmetic_meets_the_row_normalised_reading_only(oracle, name):
    w = W.generate(CASES[name]())
    ref = oracle.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree, w.parent, w.ctx_len, w.scale,
                           block_table=w.block_table)[0]
    max_abs, row_rel, floored = both_readings(stated_arithmetic(w), ref)
    print("%s: stated arithmetic vs float64: max-abs %.3e, row-normalised max-rel %.3e, "
          "element-wise floored max-rel %.3e" % (name, max_abs, row_rel, floored))
    log_parity("stated-arithmetic:" + name, max_abs=max_abs, max_row_rel=row_rel, max_floored_rel=floored)
    assert max_abs <= ATTN_MAX_ABS
    assert row_rel <= ATTN_MAX_REL                  # the reading the parity tests apply
    assert row_rel >= 2.0 ** -10                    # and it is not vacuous: bf16 rounding shows
    if name == "C1":
        assert floored > 5 * ATTN_MAX_REL           # the element-wise reading rejects the arithmetic itself
