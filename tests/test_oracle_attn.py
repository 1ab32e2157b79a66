"""Pins for the CPU checker's tree attention (Sec. 2.1: attention whose causal mask is the token
tree's topology matrix).  Every comparison routine here is written separately from the checker:
numpy/torch library calls or explicit path linearisation, never the checker's own loops."""
import math

import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W


def f64(bits):
    return W.bf16_bits_to_f64(bits)


def small(**kw):
    return W.generate(W.small_config(**kw))


def run(orc, w, **kw):
    return orc.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree, w.parent, w.ctx_len,
                         w.scale, block_table=w.block_table, **kw)


def cache_rows(w, b, g):
    """K and V rows of the committed context of sequence b, kv head g, as float64 [L, D]."""
    L = int(w.ctx_len[b])
    if w.block_table is None:
        return f64(w.k_cache[b, :L, g]), f64(w.v_cache[b, :L, g])
    idx = np.arange(L)
    pg = w.block_table[b, idx // 64]
    return f64(w.k_cache[pg, idx % 64, g]), f64(w.v_cache[pg, idx % 64, g])


def decode_last(q, K, V, scale):
    """Textbook single-query softmax attention (numpy, float64)."""
    s = scale * (K @ q)
    p = np.exp(s - s.max())
    return (p / p.sum()) @ V, s.max() + math.log(p.sum())


def path_to(parent, i):
    out = []
    while i >= 0:
        out.append(i)
        i = parent[i]
    return out[::-1]


@pytest.mark.parametrize("paged", [False, True])
def test_path_linearisation(oracle, paged):
    # Node i must see exactly: context, then root ... i.  Its output is what an ordinary causal
    # decoder gives for the last token of that explicit sequence.
    w = small(batch=2, n_q_heads=4, n_kv_heads=2, ctx=(3, 150), n_nodes=13, paged=paged)
    out, out16, lse, st = run(oracle, w)
    assert (st == 0).all()
    G = w.cfg.group
    for b in range(w.cfg.batch):
        for i in range(w.cfg.n_nodes):
            pth = path_to(w.parent[b], i)
            for h in range(w.cfg.n_q_heads):
                g = h // G
                Kc, Vc = cache_rows(w, b, g)
                K = np.concatenate([Kc, f64(w.k_tree[b, pth, g])])
                V = np.concatenate([Vc, f64(w.v_tree[b, pth, g])])
                ref, ref_lse = decode_last(f64(w.q[b, i, h]), K, V, w.scale)
                np.testing.assert_allclose(out[b, i, h], ref, rtol=1e-11, atol=1e-13)
                assert abs(lse[b, i, h] - ref_lse) < 1e-11


def _with_parent(w, parent):
    w.parent[:] = parent
    return w


def test_chain_is_causal_prefill(oracle):
    w = _with_parent(small(batch=1, n_q_heads=2, n_kv_heads=1, ctx=40, n_nodes=9), W.tree_chain(9))
    out = run(oracle, w)[0]
    Kc, Vc = cache_rows(w, 0, 0)
    K = torch.from_numpy(np.concatenate([Kc, f64(w.k_tree[0, :, 0])]))
    V = torch.from_numpy(np.concatenate([Vc, f64(w.v_tree[0, :, 0])]))
    for h in range(2):
        Q = torch.from_numpy(f64(w.q[0, :, h]))
        # causal prefill of the 9 new tokens on top of 40 cached ones
        mask = torch.ones(9, 49, dtype=torch.bool).tril(diagonal=40)
        ref = torch.nn.functional.scaled_dot_product_attention(
            Q[None, None], K[None, None], V[None, None], attn_mask=mask, scale=w.scale)[0, 0]
        np.testing.assert_allclose(out[0, :, h], ref.numpy(), rtol=1e-11, atol=1e-13)


def test_star_and_forest_are_independent_decodes(oracle):
    n = 7
    w = _with_parent(small(batch=1, n_q_heads=2, n_kv_heads=2, ctx=33, n_nodes=n), W.tree_star(n))
    out = run(oracle, w)[0]
    for h in range(2):
        Kc, Vc = cache_rows(w, 0, h)
        for i in range(n):
            extra = [0] if i == 0 else [0, i]
            K = np.concatenate([Kc, f64(w.k_tree[0, extra, h])])
            V = np.concatenate([Vc, f64(w.v_tree[0, extra, h])])
            ref, _ = decode_last(f64(w.q[0, i, h]), K, V, w.scale)
            np.testing.assert_allclose(out[0, i, h], ref, rtol=1e-11, atol=1e-13)
    w = _with_parent(w, W.tree_forest(n))
    out, _, _, st = run(oracle, w)
    assert (st == 0).all()            # several roots are legal for attention
    for h in range(2):
        Kc, Vc = cache_rows(w, 0, h)
        for i in range(n):
            K = np.concatenate([Kc, f64(w.k_tree[0, [i], h])])
            V = np.concatenate([Vc, f64(w.v_tree[0, [i], h])])
            ref, _ = decode_last(f64(w.q[0, i, h]), K, V, w.scale)
            np.testing.assert_allclose(out[0, i, h], ref, rtol=1e-11, atol=1e-13)


def topology_matrix(parent):
    """N x N boolean matrix by transitive closure of the parent relation (matrix powers)."""
    n = len(parent)
    A = np.eye(n, dtype=np.int64)
    for i in range(n):
        if parent[i] >= 0:
            A[i, parent[i]] = 1
    M = A.copy()
    for _ in range(n):
        M = ((M @ A) > 0).astype(np.int64)
    return M.astype(bool)


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2), (6, 1)])
def test_library_attention_with_explicit_mask(oracle, hq, hkv):
    w = small(batch=2, n_q_heads=hq, n_kv_heads=hkv, ctx=(1, 70), n_nodes=17)
    out, out16, lse, _ = run(oracle, w)
    G = hq // hkv
    for b in range(2):
        L = int(w.ctx_len[b])
        N = w.cfg.n_nodes
        mask = np.concatenate([np.ones((N, L), bool), topology_matrix(w.parent[b])], axis=1)
        K = np.concatenate([f64(w.k_cache[b, :L]), f64(w.k_tree[b])]).transpose(1, 0, 2)
        V = np.concatenate([f64(w.v_cache[b, :L]), f64(w.v_tree[b])]).transpose(1, 0, 2)
        Q = f64(w.q[b]).transpose(1, 0, 2)
        Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)
        Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q)[None], Kt[None], Vt[None],
            attn_mask=torch.from_numpy(mask), scale=w.scale)[0]
        np.testing.assert_allclose(out[b].transpose(1, 0, 2), ref.numpy(), rtol=1e-11, atol=1e-13)
        # the bf16 output is the double result rounded once
        ref16 = ref.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        got16 = out16[b].transpose(1, 0, 2)
        diff = np.abs(f64(got16) - f64(ref16))
        assert (diff <= np.abs(f64(ref16)) * 2.0 ** -7 + 1e-30).all()   # at most one bf16 step
        assert (got16 == ref16).mean() > 0.999


def test_single_node_is_textbook_decode_and_empty_context(oracle):
    w = small(batch=1, n_q_heads=2, n_kv_heads=1, ctx=0, n_nodes=1)
    out, _, lse, _ = run(oracle, w)
    # one key (the node itself): the softmax weight is 1, the output is its V row
    for h in range(2):
        np.testing.assert_allclose(out[0, 0, h], f64(w.v_tree[0, 0, 0]), rtol=0, atol=0)
        s = w.scale * float(f64(w.q[0, 0, h]) @ f64(w.k_tree[0, 0, 0]))
        assert abs(lse[0, 0, h] - s) < 1e-12


def test_zero_query_gives_mean_of_visible_values(oracle):
    # q = 0 makes every visible score 0, so the output is the plain mean of the visible V rows
    w = small(batch=1, n_q_heads=1, n_kv_heads=1, ctx=5, n_nodes=6)
    w.q[:] = 0
    out, _, lse, _ = run(oracle, w)
    for i in range(6):
        pth = path_to(w.parent[0], i)
        V = np.concatenate([f64(w.v_cache[0, :5, 0]), f64(w.v_tree[0, pth, 0])])
        np.testing.assert_allclose(out[0, i, 0], V.mean(axis=0), rtol=1e-13, atol=1e-15)
        assert abs(lse[0, i, 0] - math.log(len(V))) < 1e-13


def test_convex_hull_and_lse(oracle):
    w = small(batch=1, n_q_heads=4, n_kv_heads=2, ctx=64, n_nodes=10)
    out, _, lse, _ = run(oracle, w)
    for h in range(4):
        g = h // 2
        for i in range(10):
            pth = path_to(w.parent[0], i)
            V = np.concatenate([f64(w.v_cache[0, :64, g]), f64(w.v_tree[0, pth, g])])
            K = np.concatenate([f64(w.k_cache[0, :64, g]), f64(w.k_tree[0, pth, g])])
            assert (out[0, i, h] <= V.max(axis=0) + 1e-12).all()
            assert (out[0, i, h] >= V.min(axis=0) - 1e-12).all()
            s = w.scale * (K @ f64(w.q[0, i, h]))
            two_pass = math.log(np.exp(s).sum())      # scores are small: no overflow
            assert abs(lse[0, i, h] - two_pass) < 1e-10


def test_mask_exactness_and_relabelling(oracle):
    w = small(batch=1, n_q_heads=2, n_kv_heads=1, ctx=20, n_nodes=12, seed=W.BASE_SEED + 5)
    out = run(oracle, w)[0]
    N = 12
    big = W.f32_to_bf16_bits(np.full(128, 3.0e4, np.float32))
    for i in range(N):
        anc = set(path_to(w.parent[0], i))
        k2, v2 = w.k_tree.copy(), w.v_tree.copy()
        for j in range(N):
            if j not in anc:
                k2[0, j, 0] = big
                v2[0, j, 0] = big
        o2 = oracle.tree_attn(w.q, w.k_cache, w.v_cache, k2, v2, w.parent, w.ctx_len, w.scale)[0]
        assert np.array_equal(o2[0, i], out[0, i])      # bit-identical
    # another topological order of the same tree: outputs are the same rows, permuted.
    # (A node's ancestors keep their relative order, so even the summation order is unchanged.)
    rng = np.random.default_rng(0)
    depth = W.tree_depths(w.parent[0])
    order = np.lexsort((rng.random(N), depth))          # new -> old; parents stay before children
    inv = np.empty(N, dtype=np.int64)
    inv[order] = np.arange(N)
    par2 = np.array([[-1 if w.parent[0][o] < 0 else inv[w.parent[0][o]] for o in order]], np.int32)
    o3 = oracle.tree_attn(w.q[:, order], w.k_cache, w.v_cache, w.k_tree[:, order],
                          w.v_tree[:, order], par2, w.ctx_len, w.scale)[0]
    np.testing.assert_allclose(o3[0], out[0, order], rtol=1e-13, atol=1e-15)


def test_paged_equals_contiguous_and_row_subset(oracle):
    w = small(batch=2, n_q_heads=4, n_kv_heads=2, ctx=(60, 200), n_nodes=9, paged=True)
    out_p = run(oracle, w)[0]
    cap = int(w.ctx_len.max()) + 9
    kc = np.zeros((2, cap, 2, 128), np.uint16)
    vc = np.zeros_like(kc)
    for b in range(2):
        idx = np.arange(int(w.ctx_len[b]))
        kc[b, idx] = w.k_cache[w.block_table[b, idx // 64], idx % 64]
        vc[b, idx] = w.v_cache[w.block_table[b, idx // 64], idx % 64]
    out_c = oracle.tree_attn(w.q, kc, vc, w.k_tree, w.v_tree, w.parent, w.ctx_len, w.scale)[0]
    assert np.array_equal(out_p, out_c)
    rows = np.array([[1, 8, 3], [0, 0, 0], [1, 2, 1]], np.int32)
    sub = run(oracle, w, rows=rows)[0]
    for r, (b, i, h) in enumerate(rows):
        assert np.array_equal(sub[r], out_p[b, i, h])


def test_malformed_tree_is_flagged(oracle):
    w = small(batch=2, n_q_heads=2, n_kv_heads=1, ctx=4, n_nodes=5)
    w.parent[1, 3] = 3                       # a node may not be its own parent
    st = run(oracle, w)[3]
    assert st[0] == 0 and st[1] != 0


def test_bf16_rounding_helper(oracle):
    # exact bf16 values map to themselves; midpoints go to the even neighbour; just above a
    # midpoint goes up.  Checked on every positive normal bf16 pattern of a few binades.
    for hi in list(range(0x3F00, 0x3F90)) + list(range(0x0080, 0x0100)) + [0x7F7E]:
        a = float(W.bf16_bits_to_f64(np.array([hi], np.uint16))[0])
        b = float(W.bf16_bits_to_f64(np.array([hi + 1], np.uint16))[0])
        assert oracle.f64_to_bf16_bits(a) == hi
        assert oracle.f64_to_bf16_bits(-a) == hi | 0x8000
        mid = (a + b) / 2
        assert oracle.f64_to_bf16_bits(mid) == (hi if hi % 2 == 0 else hi + 1)
        assert oracle.f64_to_bf16_bits(np.nextafter(mid, np.inf)) == hi + 1
        assert oracle.f64_to_bf16_bits(np.nextafter(mid, -np.inf)) == hi
    assert oracle.f64_to_bf16_bits(0.0) == 0 and oracle.f64_to_bf16_bits(-0.0) == 0x8000
