"""GPU parity: every C-ABI call against the CPU checker on the same seeded inputs.

Integer outputs (argmax ids, accepted path, next token, status, context lengths) and the committed
cache bytes must match exactly; the attention output must be within max-abs 2e-2 and max-rel 1e-2
of the checker's float64 result."""
import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W
from parity_util import assert_attn_close, attn_errors, log_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def clv():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2408_00264_b200 import binding
    binding.lib()          # raises if the library was not built: there is no fallback
    return binding


def make_step(w, **kw):
    from paper_2408_00264_b200.step import VerifyStep
    return VerifyStep(w, **kw)


def bits(t):
    from paper_2408_00264_b200.step import bits_of
    return bits_of(t)


def check_attention(oracle, w, st, rows=None):
    if rows is None:
        ref, _, lse, status = oracle.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree,
                                               w.parent, w.ctx_len, w.scale,
                                               block_table=w.block_table)
        got = bits(st.out)
        got_lse = st.lse.cpu().numpy().astype(np.float64)
    else:
        ref, _, lse, status = oracle.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree,
                                               w.parent, w.ctx_len, w.scale,
                                               block_table=w.block_table, rows=rows)
        g = bits(st.out)
        got = g[rows[:, 0], rows[:, 1], rows[:, 2]]
        got_lse = st.lse.cpu().numpy().astype(np.float64)[rows[:, 0], rows[:, 1], rows[:, 2]]
    assert np.array_equal(st.status[0].cpu().numpy(), status)
    assert_attn_close(got, ref, w.cfg.name)
    assert np.abs(got_lse - lse).max() < 2e-3
    if w.cfg.name in W.CONFIGS:
        a, r = attn_errors(got, ref)
        log_parity(w.cfg.name, rows=int(np.prod(got.shape[:-1])), max_abs=a, max_row_rel=r,
                   max_lse_abs=float(np.abs(got_lse - lse).max()))
    return ref


def check_accept_and_commit(oracle, w, st):
    ids = oracle.argmax(w.logits, w.cfg.vocab)
    assert np.array_equal(st.ids.cpu().numpy(), ids)
    alen, aidx, nxt, s1 = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    assert np.array_equal(st.accept_len.cpu().numpy(), alen)
    assert np.array_equal(st.accept_idx.cpu().numpy(), aidx)
    assert np.array_equal(st.next_token.cpu().numpy(), nxt)
    assert np.array_equal(st.status[1].cpu().numpy(), s1)
    kc, vc, new_len, s2 = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen,
                                           w.ctx_len, block_table=w.block_table)
    assert np.array_equal(st.ctx_len_out.cpu().numpy(), new_len)
    assert np.array_equal(st.status[2].cpu().numpy(), s2)
    assert np.array_equal(bits(st.k_cache), kc)      # whole buffers, byte for byte
    assert np.array_equal(bits(st.v_cache), vc)
    return alen


def full_step(clv, oracle, w, rows=None):
    st = make_step(w)
    st.run()
    torch.cuda.synchronize()
    check_attention(oracle, w, st, rows)
    alen = check_accept_and_commit(oracle, w, st)
    # a second step on fresh buffers gives bit-identical outputs (no stale workspace state)
    st2 = make_step(w)
    st2.workspace = st.workspace
    st2.run(fused_tail=False)   # the walk and the commit as two launches: same results as the fused one
    torch.cuda.synchronize()
    assert torch.equal(st2.ids, st.ids) and torch.equal(st2.accept_idx, st.accept_idx)
    assert torch.equal(st2.accept_len, st.accept_len) and torch.equal(st2.next_token, st.next_token)
    assert torch.equal(st2.ctx_len_out, st.ctx_len_out) and torch.equal(st2.status, st.status)
    assert torch.equal(st2.k_cache, st.k_cache) and torch.equal(st2.v_cache, st.v_cache)
    assert_attn_close(bits(st2.out), W.bf16_bits_to_f64(bits(st.out)), "repeat")
    return alen


# ------------------------------------------------------------------ the five stated workloads
@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4", "C5"])
def test_config_full_compare(clv, oracle, name):
    # every attention row, every id, the accepted paths and the whole committed cache, at the
    # stated sizes (the checker needs a few seconds for C4 and some tens of seconds for C5)
    w = W.generate(W.CONFIGS[name])
    alen = full_step(clv, oracle, w)
    assert (alen >= 1).all()


# ------------------------------------------------------------------ shapes around tile edges
@pytest.mark.parametrize("ctx", [0, 1, 63, 64, 65, 127, 129, 700])
@pytest.mark.parametrize("n_nodes,hq,hkv", [(1, 4, 4), (7, 4, 1), (33, 8, 2), (64, 4, 4),
                                            (128, 8, 2), (100, 6, 3)])
def test_attention_shapes(clv, oracle, ctx, n_nodes, hq, hkv):
    cfg = W.small_config(batch=2, n_q_heads=hq, n_kv_heads=hkv, ctx=ctx, n_nodes=n_nodes,
                         max_depth=6, vocab=64, seed=W.BASE_SEED + ctx * 131 + n_nodes)
    w = W.generate(cfg)
    st = make_step(w)
    st.tree_attn()
    torch.cuda.synchronize()
    check_attention(oracle, w, st)


@pytest.mark.parametrize("tree", ["chain", "star", "forest"])
@pytest.mark.parametrize("paged", [False, True])
def test_attention_special_trees_and_paging(clv, oracle, tree, paged):
    n = 40
    cfg = W.small_config(batch=3, n_q_heads=8, n_kv_heads=2, ctx=(1, 300), n_nodes=n, vocab=64,
                         paged=paged)
    w = W.generate(cfg)
    w.parent[:] = {"chain": W.tree_chain, "star": W.tree_star, "forest": W.tree_forest}[tree](n)
    st = make_step(w)
    st.tree_attn()
    torch.cuda.synchronize()
    check_attention(oracle, w, st)


@pytest.mark.parametrize("hq,hkv,n_nodes", [(6, 2, 37), (12, 2, 37), (5, 1, 37), (28, 4, 64), (24, 2, 128),
                                             (7, 1, 18), (7, 1, 19)])
def test_attention_group_sizes_that_do_not_divide_128(clv, oracle, hq, hkv, n_nodes):
    # a 128-row tile holds whole nodes only, so with such group sizes some of its rows stay idle
    cfg = W.small_config(batch=2, n_q_heads=hq, n_kv_heads=hkv, ctx=(30, 500), n_nodes=n_nodes, vocab=64,
                         seed=W.BASE_SEED + hq)
    w = W.generate(cfg)
    st = make_step(w)
    st.tree_attn()
    torch.cuda.synchronize()
    check_attention(oracle, w, st)


def test_attention_many_splits_and_ragged(clv, oracle):
    # few (sequence, head) units and a long context: the key axis is split many ways; one
    # sequence is much shorter than max_ctx_len so some splits of it are empty
    cfg = W.small_config(batch=2, n_q_heads=2, n_kv_heads=1, ctx=(40, 2500), n_nodes=20, vocab=64,
                         seed=W.BASE_SEED + 9)
    w = W.generate(cfg)
    w.ctx_len[0] = 40
    st = make_step(w)
    st.max_ctx_len = 2500
    st.workspace = clv.new_workspace(st.shape, st.cache, 2500)
    st.tree_attn()
    torch.cuda.synchronize()
    check_attention(oracle, w, st)


def _scale_bf16_by_pow2(bits_arr, k):
    """bf16 bit patterns times 2^k, exactly (normal numbers; zeros stay zeros)."""
    b = bits_arr.astype(np.int64)
    expo = (b >> 7) & 0xFF
    new = np.clip(expo + k, 1, 254)
    out = (b & ~(0xFF << 7)) | (new << 7)
    return np.where(expo == 0, b, out).astype(np.uint16)


@pytest.mark.parametrize("k_lo,k_hi", [(40, 40), (-40, -40), (30, -30), (-30, 30)])
def test_attention_value_magnitudes_across_splits(clv, oracle, k_lo, k_hi):
    # The split-KV partial sums travel between blocks in fp16, every row scaled by its own power of
    # two.  Values far outside the fp16 range, and key ranges whose values differ by 2^60, must
    # come out as the checker computes them (relative to each output row's scale: the absolute
    # tolerance presupposes values of order one and is not applied here).
    from parity_util import attn_errors, ATTN_MAX_REL
    cfg = W.small_config(batch=2, n_q_heads=8, n_kv_heads=2, ctx=(1500, 2300), n_nodes=48, vocab=64,
                         seed=W.BASE_SEED + 77)
    w = W.generate(cfg)
    half = w.v_cache.shape[1] // 2 if w.v_cache.ndim == 4 else None
    assert half is not None
    w.v_cache[:, :half] = _scale_bf16_by_pow2(w.v_cache[:, :half], k_lo)
    w.v_cache[:, half:] = _scale_bf16_by_pow2(w.v_cache[:, half:], k_hi)
    w.v_tree[:] = _scale_bf16_by_pow2(w.v_tree, k_hi)
    st = make_step(w)
    st.tree_attn()
    torch.cuda.synchronize()
    ref, _, lse, status = oracle.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree, w.parent,
                                           w.ctx_len, w.scale, block_table=w.block_table)
    got = bits(st.out)
    assert np.array_equal(st.status[0].cpu().numpy(), status)
    assert np.isfinite(W.bf16_bits_to_f64(got)).all()
    _, rel = attn_errors(got, ref)
    assert rel <= ATTN_MAX_REL, rel
    assert np.abs(st.lse.cpu().numpy().astype(np.float64) - lse).max() < 2e-3


def test_attention_mask_exactness_on_device(clv, oracle):
    # overwriting K/V of nodes that are not ancestors must not change a node's output at all
    cfg = W.small_config(batch=1, n_q_heads=4, n_kv_heads=2, ctx=100, n_nodes=24, vocab=64)
    w = W.generate(cfg)
    st = make_step(w)
    st.tree_attn()
    torch.cuda.synchronize()
    base = st.out.clone()
    i = 17
    anc = set()
    j = i
    while j >= 0:
        anc.add(j)
        j = int(w.parent[0, j])
    big = W.f32_to_bf16_bits(np.full(128, 3.0e4, np.float32))
    for j in range(24):
        if j not in anc:
            w.k_tree[0, j, :] = big
            w.v_tree[0, j, :] = big
    st2 = make_step(w)
    st2.tree_attn()
    torch.cuda.synchronize()
    assert torch.equal(st2.out[0, i], base[0, i])


def test_attention_flags_bad_sequences(clv, oracle):
    cfg = W.small_config(batch=3, n_q_heads=4, n_kv_heads=2, ctx=70, n_nodes=10, vocab=64)
    w = W.generate(cfg)
    w.parent[1, 4] = 6                      # parent after child
    st = make_step(w)
    st.ctx_len[2] = w.cap_tokens + 5        # context larger than the cache rows
    st.tree_attn()
    torch.cuda.synchronize()
    assert st.status[0].cpu().tolist() == [0, clv.CLV_ERR_TREE, clv.CLV_ERR_TREE]
    ref = oracle.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree, w.parent, w.ctx_len,
                           w.scale)[0]
    assert_attn_close(bits(st.out)[0], ref[0], "valid sequence beside bad ones")


@pytest.mark.parametrize("paged", [False, True])
def test_attention_units_of_many_row_tiles(clv, oracle, paged):
    # four row tiles per (sequence, kv head) (GQA 4 x 128 nodes = 512 rows): such units are worked
    # by blocks of two row tiles; ragged contexts, one of them shorter than a key tile, key splits
    cfg = W.small_config(batch=3, n_q_heads=8, n_kv_heads=2, ctx=(50, 1300), n_nodes=128, vocab=64,
                         paged=paged, seed=W.BASE_SEED + 512)
    w = W.generate(cfg)
    st = make_step(w)
    st.tree_attn()
    torch.cuda.synchronize()
    check_attention(oracle, w, st)


@pytest.mark.parametrize("n_nodes", [24, 128])   # one row tile per block / two row tiles per block
def test_attention_wait_that_runs_out_is_reported_and_leaves_the_library_usable(clv, oracle, n_nodes):
    # Every on-chip wait of the attention kernel is bounded.  With the bound cut to a few dozen SM
    # cycles the ordinary wait for the first tile (a load from device memory takes far longer)
    # runs out: the blocks must leave in order - copies and tensor-core work in flight waited for,
    # tensor memory released - the call itself succeeds, and status[] says CLV_ERR_TIMEOUT.
    # Nothing faults; the next call, on the same workspace, is an ordinary one.
    cfg = W.small_config(batch=2, n_q_heads=8, n_kv_heads=2, ctx=(300, 700), n_nodes=n_nodes, vocab=64,
                         seed=W.BASE_SEED + 404)
    w = W.generate(cfg)
    st = make_step(w)
    try:
        clv.clv_test_set_wait_limit(32)
        st.tree_attn()
        torch.cuda.synchronize()
    finally:
        clv.clv_test_set_wait_limit(0)
    assert st.status[0].cpu().tolist() == [clv.CLV_ERR_TIMEOUT] * 2
    st.status.zero_()
    st.tree_attn()
    torch.cuda.synchronize()
    check_attention(oracle, w, st)


# ------------------------------------------------------------------ argmax
@pytest.mark.parametrize("vocab,ld_pad", [(1, 0), (7, 0), (8, 8), (2047, 0), (2049, 16),
                                          (32000, 0), (50257, 8), (128256, 0)])
def test_argmax_sizes(clv, oracle, vocab, ld_pad):
    rows_b, rows_n = 2, 5
    ld = (vocab + 7) // 8 * 8 + ld_pad
    rng = np.random.default_rng(vocab)
    winner = rng.integers(0, vocab, size=rows_b * rows_n)
    lg = W.make_logits(rows_b * rows_n, vocab, ld, winner, 0.5, seed=vocab + 1)
    lg[:, vocab:] = 0x7F00                  # huge values in the padding must be ignored
    shape = clv.make_shape(rows_b, rows_n, 1, 1, vocab, 1)
    ws = clv.new_workspace(shape, None, 0)
    d = torch.from_numpy(lg.view(np.int16)).cuda()
    ids = torch.empty(rows_b, rows_n, dtype=torch.int32, device="cuda")
    clv.clv_accept_argmax(shape, d, ld, ids, ws)
    clv.clv_accept_argmax(shape, d, ld, ids, ws)     # the workspace is reusable as is
    torch.cuda.synchronize()
    ref = oracle.argmax(lg, vocab)
    assert np.array_equal(ids.cpu().numpy().reshape(-1), ref)
    if vocab > 1:
        assert np.array_equal(ref, winner)


def test_argmax_ties_zeros_and_infinities(clv, oracle):
    vocab = 40000                            # several chunks per row
    cfg = W.small_config(batch=1, n_nodes=8, vocab=vocab)
    w = W.generate(cfg)
    lg = w.logits[0]
    lg[:] = W.f32_to_bf16_bits(np.full(lg.shape, -1.0, np.float32))
    one = 0x3F80
    lg[0, [39999, 17, 20000]] = one          # equal maxima in different chunks: lowest index
    lg[1, vocab - 1] = one                   # maximum in the very last column
    lg[2, 0] = one
    lg[3, :] = 0x8000                        # all -0.0 with a +0.0 later: index 0
    lg[3, 30000] = 0x0000
    lg[4, :] = 0xFF80                        # all -inf
    lg[5, 25000] = 0x0000                    # +0.0 after -0.0, both above the -1 background
    lg[5, 123] = 0x8000
    lg[6, [5, 6, 7, 4]] = one                # ties inside one 16-byte vector
    lg[7, :] = 0xFF80
    lg[7, 33333] = 0xC2C8                    # -100 among -inf
    st = make_step(w)
    st.accept_argmax()
    torch.cuda.synchronize()
    ref = oracle.argmax(w.logits, vocab)
    assert ref[0].tolist() == [17, vocab - 1, 0, 0, 0, 123, 4, 33333]
    assert np.array_equal(st.ids.cpu().numpy(), ref)


@pytest.mark.parametrize("rows_b,rows_n,vocab", [(3, 7, 40008), (1, 1, 8), (2, 64, 9000), (5, 3, 2051), (1, 128, 33)])
def test_argmax_cuts_ties_and_ragged_rows(clv, oracle, rows_b, rows_n, vocab):
    # A row is scanned in pieces by several blocks, wherever the cuts fall: equal maxima planted far
    # apart (first index wins), maxima in the ragged last elements of a row (vocab not a multiple
    # of 8), and a second call on the same workspace.
    ld = (vocab + 7) // 8 * 8 + 8
    rng = np.random.default_rng(vocab * 31 + rows_n)
    rows = rows_b * rows_n
    lg = np.empty((rows, ld), np.uint16)
    lg[:] = W.f32_to_bf16_bits(rng.standard_normal((rows, ld)).astype(np.float32))
    big = int(W.f32_to_bf16_bits(np.array([9.0], np.float32))[0])
    for r in range(rows):
        k = r % 4
        if k == 0:
            pos = sorted(set(int(x) for x in rng.integers(0, vocab, size=5)))
            lg[r, pos] = big                      # ties far apart
        elif k == 1:
            lg[r, vocab - 1] = big                # the very last (possibly ragged) element
        elif k == 2:
            lg[r, max(0, vocab - 3)] = big
            lg[r, vocab // 2] = big               # tie between the middle and the ragged end
        # k == 3: plain random row
    lg[:, vocab:] = 0x7F00                        # huge values in the padding must be ignored
    shape = clv.make_shape(rows_b, rows_n, 1, 1, vocab, 1)
    ws = clv.new_workspace(shape, None, 0)
    d = torch.from_numpy(lg.view(np.int16)).cuda()
    ids = torch.full((rows_b, rows_n), -5, dtype=torch.int32, device="cuda")
    ref = oracle.argmax(lg, vocab)
    for _ in range(2):
        clv.clv_accept_argmax(shape, d, ld, ids, ws)
        torch.cuda.synchronize()
        assert np.array_equal(ids.cpu().numpy().reshape(-1), ref)
        ids.fill_(-5)


# ------------------------------------------------------------------ walk and commit
def test_walk_random_trees_and_errors(clv, oracle):
    rng = np.random.default_rng(5)
    B, N = 64, 48
    cfg = W.small_config(batch=B, n_nodes=N, vocab=16, n_q_heads=1, n_kv_heads=1, ctx=1)
    w = W.generate(cfg)
    tokens = np.stack([W._draw_tokens(w.parent[b], 64, rng) for b in range(B)])
    ids = np.stack([W._plant_winners(w.parent[b], tokens[b], 64, 0.7, rng) for b in range(B)])
    w.parent[3, 0] = 0                        # root is not a root
    w.parent[4, 9] = -1                       # second root
    w.parent[5, 7] = 7                        # self parent
    w.parent[6] = W.tree_chain(N)             # deep chain, every edge agreeing: overflows path_cap
    tokens[6] = np.arange(N)
    ids[6, :-1] = tokens[6, 1:]
    from paper_2408_00264_b200 import binding as b
    dev = "cuda"
    shape = b.make_shape(B, N, 1, 1, 16, 9)
    t = lambda a: torch.from_numpy(a).to(dev)
    alen = torch.empty(B, dtype=torch.int32, device=dev)
    aidx = torch.empty(B, 9, dtype=torch.int32, device=dev)
    nxt = torch.empty(B, dtype=torch.int32, device=dev)
    stt = torch.empty(B, dtype=torch.int32, device=dev)
    b.clv_accept_walk(shape, t(w.parent), t(tokens), t(ids), alen, aidx, nxt, stt)
    torch.cuda.synchronize()
    r_len, r_idx, r_nxt, r_st = oracle.accept_walk(w.parent, tokens, ids, 9)
    assert np.array_equal(alen.cpu().numpy(), r_len) and np.array_equal(aidx.cpu().numpy(), r_idx)
    assert np.array_equal(nxt.cpu().numpy(), r_nxt) and np.array_equal(stt.cpu().numpy(), r_st)
    assert r_st[[3, 4, 5, 6]].tolist() == [7, 7, 7, 7] and r_len.max() >= 2


@pytest.mark.parametrize("paged", [False, True])
def test_commit_edges_alias_and_capacity(clv, oracle, paged):
    cfg = W.small_config(batch=4, n_q_heads=8, n_kv_heads=2, ctx=(50, 140), n_nodes=12, vocab=64,
                         paged=paged, p_accept=0.9)
    w = W.generate(cfg)
    ids = oracle.argmax(w.logits, 64)
    alen, aidx, _, _ = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    alen = alen.copy()
    aidx = aidx.copy()
    ctx = w.ctx_len.copy()
    alen[1] = 0                                # nothing to commit
    if paged:
        ctx[2] = w.block_table.shape[1] * 64 - 1   # second accepted row has no page
    else:
        ctx[2] = w.cap_tokens - 1                  # second accepted row has no slot
    alen[2] = max(2, alen[2]); aidx[2, :2] = [0, 1]
    aidx[3, 0] = 12                            # node index outside the tree
    st = make_step(w)
    st.ctx_len.copy_(torch.from_numpy(ctx))
    st.accept_len.copy_(torch.from_numpy(alen))
    st.accept_idx.copy_(torch.from_numpy(aidx))
    st.kv_commit(ctx_len_out=st.ctx_len)       # in place: ctx_len_out aliases ctx_len
    torch.cuda.synchronize()
    kc, vc, new_len, s2 = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen,
                                           ctx, block_table=w.block_table)
    assert s2.tolist() == [0, 0, 7, 7]
    assert np.array_equal(st.ctx_len.cpu().numpy(), new_len)
    assert np.array_equal(st.status[2].cpu().numpy(), s2)
    assert np.array_equal(bits(st.k_cache), kc) and np.array_equal(bits(st.v_cache), vc)


@pytest.mark.parametrize("paged", [False, True])
def test_walk_commit_in_one_launch_with_errors(clv, oracle, paged):
    # malformed trees, a path longer than path_cap and a cache without room: the fused call gives
    # what the two calls give, sequence by sequence, and what the checker gives
    cfg = W.small_config(batch=6, n_q_heads=4, n_kv_heads=2, ctx=(10, 200), n_nodes=20, vocab=64,
                         paged=paged, seed=W.BASE_SEED + 31)
    w = W.generate(cfg)
    w.parent[1, 5] = 7            # parent after child
    w.parent[2, 0] = 0            # root is not a root
    w.parent[3, 4] = -1           # a second root: the walk refuses, attention would not
    if paged:
        w.block_table[4, :] = -1                 # sequence 4 has no page for its accepted rows
    else:
        w.ctx_len[4] = w.cap_tokens              # ... or no room left in its cache rows
    results = []
    for fused in (True, False):
        st = make_step(w)
        st.accept_argmax()
        if fused:
            st.accept_walk_commit()
        else:
            st.accept_walk()
            st.kv_commit()
        torch.cuda.synchronize()
        results.append(st)
    a, b = results
    for name in ("accept_len", "accept_idx", "next_token", "ctx_len_out", "k_cache", "v_cache"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    assert torch.equal(a.status[1:], b.status[1:])
    ids = oracle.argmax(w.logits, w.cfg.vocab)
    alen, aidx, nxt, s1 = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    kc, vc, new_len, s2 = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen, w.ctx_len,
                                           block_table=w.block_table)
    assert np.array_equal(a.accept_len.cpu().numpy(), alen) and np.array_equal(a.accept_idx.cpu().numpy(), aidx)
    assert np.array_equal(a.status[1].cpu().numpy(), s1) and np.array_equal(a.status[2].cpu().numpy(), s2)
    assert np.array_equal(a.ctx_len_out.cpu().numpy(), new_len)
    assert np.array_equal(bits(a.k_cache), kc) and np.array_equal(bits(a.v_cache), vc)
    assert s1.tolist()[1:4] == [7, 7, 7] and s2.tolist()[4] == 7 and s2.tolist()[0] == 0


def test_guard_bands_untouched(clv, oracle):
    # outputs live inside larger sentinel-filled buffers; nothing outside them may change
    cfg = W.small_config(batch=2, n_q_heads=8, n_kv_heads=2, ctx=(10, 333), n_nodes=19, vocab=4099)
    w = W.generate(cfg)
    st = make_step(w)
    pad = 4096

    def guarded(t):
        flat = torch.full((t.numel() + 2 * pad,), 0x5A5A if t.element_size() == 2 else 0x5A5A5A5A,
                          dtype=torch.int16 if t.element_size() == 2 else torch.int32,
                          device=t.device)
        inner = flat[pad: pad + t.numel()].view(t.dtype).view(t.shape)
        return flat, inner
    guards = {}
    for name in ["out", "lse", "ids", "accept_len", "accept_idx", "next_token", "ctx_len_out"]:
        g, inner = guarded(getattr(st, name))
        guards[name] = g
        setattr(st, name, inner)
    st.run()
    torch.cuda.synchronize()
    for name, g in guards.items():
        s = 0x5A5A if g.dtype == torch.int16 else 0x5A5A5A5A
        assert bool((g[:pad] == s).all()) and bool((g[-pad:] == s).all()), name
    check_attention(oracle, w, st)
    check_accept_and_commit(oracle, w, st)


def test_verify_step_from_host_buffers(clv, oracle):
    cfg = W.small_config(batch=3, n_q_heads=8, n_kv_heads=2, ctx=(20, 400), n_nodes=30, vocab=5000,
                         p_accept=0.8)
    w = W.generate(cfg)
    st = make_step(w, logits=False)
    c = w.cfg
    pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
    hq, hk, hv = pin(w.q), pin(w.k_tree), pin(w.v_tree)
    hp, ht, hl = pin(w.parent), pin(w.tokens), pin(w.logits)
    B, N = c.batch, c.n_nodes
    o_out = torch.empty(B, N, c.n_q_heads, 128, dtype=torch.int16).pin_memory()
    o_ids = torch.empty(B, N, dtype=torch.int32).pin_memory()
    o_len = torch.empty(B, dtype=torch.int32).pin_memory()
    o_idx = torch.empty(B, w.path_cap, dtype=torch.int32).pin_memory()
    o_nxt = torch.empty(B, dtype=torch.int32).pin_memory()
    o_st = torch.empty(3, B, dtype=torch.int32).pin_memory()
    hin = clv.ClvHostInputs(hq.data_ptr(), hk.data_ptr(), hv.data_ptr(), hp.data_ptr(),
                            ht.data_ptr(), hl.data_ptr(), w.logits.shape[-1])
    hout = clv.ClvHostOutputs(o_out.data_ptr(), o_ids.data_ptr(), o_len.data_ptr(),
                              o_idx.data_ptr(), o_nxt.data_ptr(), o_st.data_ptr())
    staging = torch.empty(clv.clv_staging_bytes(st.shape, w.logits.shape[-1]), dtype=torch.uint8,
                          device="cuda")
    clv.clv_verify_step_host(st.shape, st.cache, hin, hout, st.ctx_len, st.max_ctx_len, st.scale,
                             staging, st.workspace)
    torch.cuda.synchronize()
    ref = oracle.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree, w.parent, w.ctx_len,
                           w.scale)[0]
    assert_attn_close(o_out.numpy().view(np.uint16), ref, "host step")
    ids = oracle.argmax(w.logits, c.vocab)
    alen, aidx, nxt, _ = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    assert np.array_equal(o_ids.numpy(), ids) and np.array_equal(o_len.numpy(), alen)
    assert np.array_equal(o_idx.numpy(), aidx) and np.array_equal(o_nxt.numpy(), nxt)
    assert (o_st.numpy() == 0).all()
    kc, vc, new_len, _ = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen,
                                          w.ctx_len)
    assert np.array_equal(st.ctx_len.cpu().numpy(), new_len)
    assert np.array_equal(bits(st.k_cache), kc) and np.array_equal(bits(st.v_cache), vc)


def test_host_step_with_a_bad_argument_leaves_the_stream_empty(clv, oracle):
    # a stride the argmax refuses: the call must fail before its first copy, so neither the
    # staging area nor the device-side context lengths change
    cfg = W.small_config(batch=2, n_q_heads=4, n_kv_heads=2, ctx=(20, 100), n_nodes=10, vocab=1000)
    w = W.generate(cfg, ld_pad=4)                       # ld = 1004, not a multiple of 8
    st = make_step(w, logits=False)
    pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
    host = [pin(x) for x in (w.q, w.k_tree, w.v_tree, w.parent, w.tokens, w.logits)]
    hin = clv.ClvHostInputs(*[t.data_ptr() for t in host], w.logits.shape[-1])
    outs = [torch.zeros(4096, dtype=torch.int32).pin_memory() for _ in range(6)]
    hout = clv.ClvHostOutputs(*[t.data_ptr() for t in outs])
    staging = torch.full((clv.clv_staging_bytes(st.shape, w.logits.shape[-1]),), 0x5A, dtype=torch.uint8,
                         device="cuda")
    ctx_before = st.ctx_len.clone()
    code = clv.clv_verify_step_host(st.shape, st.cache, hin, hout, st.ctx_len, st.max_ctx_len, st.scale,
                                    staging, st.workspace, check=False)
    torch.cuda.synchronize()
    assert code == clv.CLV_ERR_ALIGN
    assert bool((staging == 0x5A).all()) and torch.equal(st.ctx_len, ctx_before)
    assert all(int(t.abs().sum()) == 0 for t in outs)
