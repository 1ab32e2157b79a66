"""The calls composed on the device: speculated sequences -> token tree -> tree attention ->
LM head with greedy choice -> acceptance walk -> KV commit, every stage compared with the CPU
checker run over the same inputs."""
import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W
from parity_util import assert_attn_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("paged", [False, True])
def test_draft_to_commit(oracle, paged):
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2408_00264_b200 import binding as clv
    from paper_2408_00264_b200.step import VerifyStep, bits_of
    B, N, V, K = 3, 64, 3000, 128
    cfg = W.small_config(batch=B, n_q_heads=8, n_kv_heads=2, ctx=(50, 400), n_nodes=N, vocab=64,
                         paged=paged, seed=W.BASE_SEED + 404)
    w = W.generate(cfg)
    w.path_cap = 8      # room for the root and five drafted tokens
    root, cand, lens = W.make_candidates(B, 20, 5, V, seed=17, p_follow=0.8)
    st = VerifyStep(w, logits=False)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()  # noqa: E731
    n_nodes = torch.zeros(B, dtype=torch.int32, device="cuda")
    node_of = torch.zeros(B, 20, 5, dtype=torch.int32, device="cuda")
    tstat = torch.zeros(B, dtype=torch.int32, device="cuda")
    # 1. the tree, written straight into the step's parent/tokens arrays
    clv.clv_build_token_tree(dev(root), dev(cand), dev(lens), st.tokens, st.parent, n_nodes, node_of, tstat)
    tok, par, nn, nof, ts = oracle.build_token_tree(root, cand, lens, N)
    torch.cuda.synchronize()
    assert (ts == 0).all() and np.array_equal(tstat.cpu().numpy(), ts)
    assert np.array_equal(st.tokens.cpu().numpy(), tok) and np.array_equal(st.parent.cpu().numpy(), par)
    # 2. hidden states whose LM-head winner is, for every node with children, its first child's
    #    token (so that the walk accepts a path), else a token nobody drafted
    rng = np.random.default_rng(5)
    wt = W.f32_to_bf16_bits(rng.standard_normal((V, K), dtype=np.float32) / np.float32(np.sqrt(K)))
    winner = np.zeros((B, N), dtype=np.int64)
    for b in range(B):
        for i in range(N):
            kids = [j for j in range(1, int(nn[b])) if par[b, j] == i]
            winner[b, i] = tok[b, kids[0]] if kids and rng.random() < 0.8 else int(rng.integers(0, V))
    hid = rng.standard_normal((B * N, K), dtype=np.float32) + np.float32(12.0) * W.bf16_bits_to_f32(
        wt[winner.reshape(-1)])
    hb = W.f32_to_bf16_bits(hid)
    # 3. the device path
    lm_status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st.tree_attn()
    clv.clv_lm_head_argmax(W.as_torch_bf16(hb).cuda(), W.as_torch_bf16(wt).cuda(), st.ids.view(-1),
                           lm_status, st.workspace)
    st.accept_walk()
    st.kv_commit()
    torch.cuda.synchronize()
    # 4. the checker over the same inputs
    ref, _, lse, astat = oracle.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree, par, w.ctx_len,
                                          w.scale, block_table=w.block_table)
    assert np.array_equal(st.status[0].cpu().numpy(), astat) and (astat == 0).all()
    assert_attn_close(bits_of(st.out), ref, "pipeline")
    ids = oracle.lm_head_argmax(hb, wt).reshape(B, N)
    assert int(lm_status.item()) == 0
    assert np.array_equal(ids, winner) and np.array_equal(st.ids.cpu().numpy(), ids)
    alen, aidx, nxt, wstat = oracle.accept_walk(par, tok, ids, w.path_cap)
    assert (wstat == 0).all() and alen.max() > 1
    assert np.array_equal(st.accept_len.cpu().numpy(), alen)
    assert np.array_equal(st.accept_idx.cpu().numpy(), aidx)
    assert np.array_equal(st.next_token.cpu().numpy(), nxt)
    kc, vc, new_len, cstat = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen,
                                              w.ctx_len, block_table=w.block_table)
    assert np.array_equal(st.ctx_len_out.cpu().numpy(), new_len)
    assert np.array_equal(bits_of(st.k_cache), kc) and np.array_equal(bits_of(st.v_cache), vc)
