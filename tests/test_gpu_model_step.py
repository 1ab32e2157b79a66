"""GPU parity of the pieces of a whole-model verify step: the interval form of the tree mask, the
commit of all layers in one launch, and the composed step (attention per layer, LM head fused with
the greedy choice, walk, commit) against the CPU checker, also when replayed from one CUDA graph."""
import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W
from parity_util import attn_errors, ATTN_MAX_ABS, ATTN_MAX_REL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def clv():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2408_00264_b200 import binding
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def oracle():
    import oracle as o
    o.build()
    return o


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def test_interval_labels_both_ways(clv, oracle):
    rng = np.random.default_rng(5)
    for n in (1, 2, 7, 33, 64, 128):
        par = np.stack([W.tree_random(n, 6, rng) for _ in range(5)] + [W.tree_chain(n), W.tree_star(n), W.tree_forest(n)])
        par = par.astype(np.int32)
        if n >= 3:
            par[1, 2] = 2 if n == 3 else 5      # malformed: parent not before child
        B = len(par)
        tin = torch.full((B, n), -9, dtype=torch.int32, device="cuda")
        tout = torch.full((B, n), -9, dtype=torch.int32, device="cuda")
        st = torch.full((B,), -9, dtype=torch.int32, device="cuda")
        clv.clv_tree_to_intervals(dev(par), tin, tout, st)
        r_in, r_out, r_st = oracle.tree_to_intervals(par)
        assert np.array_equal(st.cpu().numpy(), r_st)
        assert np.array_equal(tin.cpu().numpy(), r_in) and np.array_equal(tout.cpu().numpy(), r_out)
        back = torch.full((B, n), -9, dtype=torch.int32, device="cuda")
        st2 = torch.full((B,), -9, dtype=torch.int32, device="cuda")
        good = r_st == 0
        clv.clv_tree_from_intervals(tin, tout, back, st2)
        torch.cuda.synchronize()
        r_back, r_st2 = oracle.tree_from_intervals(r_in, r_out)
        assert np.array_equal(back.cpu().numpy(), r_back) and np.array_equal(st2.cpu().numpy(), r_st2)
        assert np.array_equal(back.cpu().numpy()[good], par[good])
    # labels that nest but are not canonical, and labels that are no forest
    cases_in = np.array([[10, 20, 40, 25], [0, 1, 1, 5], [0, 1, 2, 3], [1, 0, 2, 3]], np.int32)
    cases_out = np.array([[100, 35, 50, 30], [9, 4, 3, 6], [2, 3, 4, 4], [2, 4, 3, 4]], np.int32)
    back = torch.full((4, 4), -9, dtype=torch.int32, device="cuda")
    st = torch.full((4,), -9, dtype=torch.int32, device="cuda")
    clv.clv_tree_from_intervals(dev(cases_in), dev(cases_out), back, st)
    torch.cuda.synchronize()
    r_back, r_st = oracle.tree_from_intervals(cases_in, cases_out)
    assert r_st.tolist() == [0, 7, 7, 7] and r_back[0].tolist() == [-1, 0, 0, 1]
    assert np.array_equal(back.cpu().numpy(), r_back) and np.array_equal(st.cpu().numpy(), r_st)


def planted_model_inputs(oracle, cfg, n_layers, hidden_dim, vocab):
    """A workload whose drafted tokens often are what the LM head will choose (so that paths are
    accepted), per-layer tensors, and the LM head's inputs."""
    w = W.generate(cfg)
    B, N = cfg.batch, cfg.n_nodes
    h, wt, win = W.make_lm_head(B * N, hidden_dim, vocab, seed=cfg.seed + 3)
    win = win.reshape(B, N)
    rng = np.random.default_rng(cfg.seed)
    for b in range(B):
        seen = set()
        for c in range(1, N):
            p = int(w.parent[b, c])
            if p not in seen and rng.random() < 0.7:      # the first child of a node carries the node's winner
                w.tokens[b, c] = win[b, p]
            seen.add(p)
    return w, W.layer_tensors(w, n_layers), h, wt


def check_model_step(oracle, clv, st, w, layers, h, wt, attn=True):
    from paper_2408_00264_b200.step import bits_of
    q, k_tree, v_tree, k_cache, v_cache = layers
    L = q.shape[0]
    assert st.status.cpu().numpy().max() == 0
    if attn:
        for l in range(L):
            ref = oracle.tree_attn(q[l], k_cache[l], v_cache[l], k_tree[l], v_tree[l], w.parent, w.ctx_len, w.scale,
                                   block_table=w.block_table)[0]
            max_abs, max_rel = attn_errors(bits_of(st.out[l]), ref)
            assert max_abs <= ATTN_MAX_ABS and max_rel <= ATTN_MAX_REL, (l, max_abs, max_rel)
    ids = oracle.lm_head_argmax(h, wt).reshape(w.parent.shape)
    assert np.array_equal(st.ids.cpu().numpy(), ids)
    alen, aidx, nxt, s1 = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    assert np.array_equal(st.accept_len.cpu().numpy(), alen) and np.array_equal(st.accept_idx.cpu().numpy(), aidx)
    assert np.array_equal(st.next_token.cpu().numpy(), nxt)
    for l in range(L):
        kc, vc, new_len, s2 = oracle.kv_commit(k_cache[l], v_cache[l], k_tree[l], v_tree[l], aidx, alen, w.ctx_len,
                                               block_table=w.block_table)
        assert np.array_equal(bits_of(st.k_cache[l]), kc) and np.array_equal(bits_of(st.v_cache[l]), vc), l
    assert np.array_equal(st.ctx_len_out.cpu().numpy(), new_len)
    return alen


@pytest.mark.parametrize("paged,n_nodes", [(False, 24), (True, 24), (False, 40)])
def test_whole_model_step(clv, oracle, paged, n_nodes):
    from paper_2408_00264_b200.step import ModelVerifyStep
    cfg = W.small_config(batch=3, n_q_heads=8, n_kv_heads=2, ctx=(30, 400), n_nodes=n_nodes, vocab=3000,
                         paged=paged, seed=W.BASE_SEED + 40 + n_nodes)
    w, layers, h, wt = planted_model_inputs(oracle, cfg, 3, 128, 3000)
    tin, tout, _ = oracle.tree_to_intervals(w.parent)
    st = ModelVerifyStep(w, layers, h, wt, intervals=(tin, tout))      # the tree arrives as interval labels
    st.run()
    torch.cuda.synchronize()
    assert np.array_equal(st.parent.cpu().numpy(), w.parent)
    alen = check_model_step(oracle, clv, st, w, layers, h, wt)
    assert alen.max() >= 2
    # the same step replayed from one CUDA graph on fresh buffers
    st2 = ModelVerifyStep(w, layers, h, wt, intervals=(tin, tout))
    st2.run()                                 # first calls outside capture (one-time set-up per device)
    torch.cuda.synchronize()
    st3 = ModelVerifyStep(w, layers, h, wt, intervals=(tin, tout))
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        st3.run()
    g.replay()
    torch.cuda.synchronize()
    check_model_step(oracle, clv, st3, w, layers, h, wt, attn=False)
    assert torch.equal(st3.out, st.out)


@pytest.mark.parametrize("paged", [False, True])
def test_commit_of_all_layers_with_a_failing_sequence(clv, oracle, paged):
    from paper_2408_00264_b200.step import ModelVerifyStep, bits_of
    cfg = W.small_config(batch=4, n_q_heads=4, n_kv_heads=2, ctx=(10, 150), n_nodes=12, vocab=64, paged=paged,
                         seed=W.BASE_SEED + 61)
    w = W.generate(cfg)
    L = 5
    layers = W.layer_tensors(w, L)
    if paged:
        w.block_table[2, :] = -1                 # sequence 2 has no page for its accepted rows
    else:
        w.ctx_len[2] = w.cap_tokens              # ... or no room left
    h, wt, _ = W.make_lm_head(4 * 12, 64, 64, seed=1)
    st = ModelVerifyStep(w, layers, h, wt)
    ids = oracle.argmax(w.logits, 64)
    alen, aidx, _, _ = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    st.accept_len.copy_(torch.from_numpy(alen)); st.accept_idx.copy_(torch.from_numpy(aidx))
    status = torch.full((4,), -9, dtype=torch.int32, device="cuda")
    clv.clv_kv_commit_layers(st.shape, st.caches[0], L, st.k_cache[0].numel(), st.k_tree, st.v_tree,
                             st.k_tree[0].numel(), st.accept_idx, st.accept_len, st.ctx_len, st.ctx_len_out, status)
    torch.cuda.synchronize()
    for l in range(L):
        kc, vc, new_len, s2 = oracle.kv_commit(layers[3][l], layers[4][l], layers[1][l], layers[2][l], aidx, alen,
                                               w.ctx_len, block_table=w.block_table)
        assert np.array_equal(bits_of(st.k_cache[l]), kc) and np.array_equal(bits_of(st.v_cache[l]), vc)
    assert np.array_equal(status.cpu().numpy(), s2) and s2[2] == 7
    assert np.array_equal(st.ctx_len_out.cpu().numpy(), new_len)
    # host-detectable mistakes: aliasing ctx_len_out with ctx_len, a stride shorter than a layer
    code = clv.clv_kv_commit_layers(st.shape, st.caches[0], L, st.k_cache[0].numel(), st.k_tree, st.v_tree,
                                    st.k_tree[0].numel(), st.accept_idx, st.accept_len, st.ctx_len, st.ctx_len,
                                    status, check=False)
    assert code == clv.CLV_ERR_UNSUPPORTED
    code = clv.clv_kv_commit_layers(st.shape, st.caches[0], L, 8, st.k_tree, st.v_tree, st.k_tree[0].numel(),
                                    st.accept_idx, st.accept_len, st.ctx_len, st.ctx_len_out, status, check=False)
    assert code == clv.CLV_ERR_SHAPE
