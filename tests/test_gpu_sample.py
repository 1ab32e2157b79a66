"""GPU parity of clv_accept_sample (stochastic acceptance, temperature > 0) against the CPU checker.

The outputs are integers decided by comparing a caller-supplied uniform with a probability.  The
checker works in float64, the kernels in float32 with hardware exp2, so a comparison whose two
sides lie within rounding distance may fall either way: the checker reports, per sequence, the
smallest distance between a uniform and its threshold.  Accepted paths must be identical wherever
no accept test was that close (which must hold for nearly all sequences).  The drawn token must be
identical where the draw had that margin too; otherwise it must be a valid inverse of the running
sum within MARGIN of the mass left (with 128256 tokens of about 1e-5 each, float32 running sums
cannot always name the same token as float64 ones).
"""
import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W

pytestmark = pytest.mark.gpu
MARGIN = 2e-4   # float32 sums of up to 128256 terms with 2-ulp exponentials: relative error ~1e-5


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


def run_gpu(clv, logits_bits, vocab, parent, tokens, uniforms, temperature, path_cap):
    B, N = parent.shape
    ld = logits_bits.shape[-1]
    shape = clv.make_shape(B, N, 1, 1, vocab, path_cap)
    ws = clv.new_workspace(shape, None, 0)
    i32 = dict(dtype=torch.int32, device="cuda")
    out = [torch.full((B,), -9, **i32), torch.full((B, path_cap), -9, **i32), torch.full((B,), -9, **i32),
           torch.full((B,), -9, **i32)]
    d_lg = torch.from_numpy(np.ascontiguousarray(logits_bits).view(np.int16)).cuda()
    dev = lambda a, t: torch.from_numpy(np.ascontiguousarray(a, dtype=t)).cuda()  # noqa: E731
    args = (shape, d_lg, ld, dev(parent, np.int32), dev(tokens, np.int32), dev(uniforms, np.float32), temperature)
    clv.clv_accept_sample(*args, *out, ws)
    clv.clv_accept_sample(*args, *out, ws)     # the workspace is reusable as is
    torch.cuda.synchronize()
    return [t.cpu().numpy() for t in out]


def draw_is_valid(lg_row, vocab, struck, temperature, u_last, v, tol):
    """Is v the inverse of the running sum at u_last, give or take tol of the mass left?  (float64,
    numpy: the running sums of what is left of the row's softmax, in vocabulary order)"""
    x = W.bf16_bits_to_f64(lg_row[:vocab]) / temperature
    e = np.exp(x - x.max())
    e[list(struck)] = 0.0
    if not (0 <= v < vocab) or e[v] <= 0.0:
        return False
    run = np.cumsum(e)
    left = run[-1]
    target = float(u_last) * left
    return run[v] - e[v] - tol * left <= target <= run[v] + tol * left


def compare(oracle, got, lg, vocab, parent, tokens, u, temperature, path_cap, min_robust=0.9):
    alen, aidx, nxt, st, margin = oracle.accept_sample(lg, vocab, parent, tokens, u, temperature, path_cap)
    robust = margin[:, 0] > MARGIN
    assert robust.mean() >= min_robust, "too few sequences whose accept tests rounding cannot change"
    assert np.array_equal(got[3], st)
    for name, a, b in (("accept_len", got[0], alen), ("accept_idx", got[1], aidx)):
        assert np.array_equal(a[robust], b[robust]), name
    N = parent.shape[1]
    for b in range(parent.shape[0]):
        if st[b] != 0:
            assert got[0][b] == 0 and got[2][b] == -1
            continue
        n = int(got[0][b])
        path = got[1][b, :n]
        # always well formed: a root-to-node path of the tree
        assert n >= 1 and path[0] == 0 and all(parent[b, path[j]] == path[j - 1] for j in range(1, n))
        if robust[b] and margin[b, 1] > MARGIN:
            assert got[2][b] == nxt[b]
        else:
            last = int(path[-1])
            struck = {int(tokens[b, c]) for c in range(N) if parent[b, c] == last and 0 <= tokens[b, c] < vocab}
            assert draw_is_valid(lg[b, last], vocab, struck, temperature, u[b, N], int(got[2][b]), MARGIN)
    return alen


@pytest.mark.parametrize("temperature", [1.0, 0.6, 1.7])
@pytest.mark.parametrize("vocab,n_nodes", [(64, 9), (1000, 20), (4099, 33), (8192, 10), (32000, 64), (32771, 12),
                                           (128256, 64)])   # around the edges of the 4096-logit slices and 32768-logit pieces
def test_sample_random_trees(clv, oracle, vocab, n_nodes, temperature):
    B = 6 if vocab > 100000 else 24
    cfg = W.small_config(batch=B, n_nodes=n_nodes, vocab=vocab, seed=W.BASE_SEED + vocab + n_nodes)
    w = W.generate(cfg, ld_pad=8)
    # the generator's winners lead by 0.5 only: lift them so that drafted tokens are likely to be
    # accepted at these temperatures and the walk goes several levels deep
    ids = oracle.argmax(w.logits, vocab)
    bi, ni = np.meshgrid(np.arange(B), np.arange(n_nodes), indexing="ij")
    lift = np.log(vocab) + 1.0
    w.logits[bi, ni, ids] = W.f32_to_bf16_bits((W.bf16_bits_to_f64(w.logits[bi, ni, ids]) + lift).astype(np.float32))
    w.logits[:, :, vocab:] = 0x7F00          # huge values in the padding must be ignored
    u = W.make_uniforms(B, n_nodes, seed=vocab * 7 + int(temperature * 10))
    got = run_gpu(clv, w.logits, vocab, w.parent, w.tokens, u, temperature, w.path_cap)
    alen = compare(oracle, got, w.logits, vocab, w.parent, w.tokens, u, temperature, w.path_cap)
    assert alen.max() >= 2                    # some drafts were accepted


def test_sample_low_temperature_is_the_greedy_walk(clv, oracle):
    cfg = W.small_config(batch=8, n_nodes=30, vocab=5000, seed=W.BASE_SEED + 77)
    w = W.generate(cfg)
    u = W.make_uniforms(8, 30, seed=5)
    got = run_gpu(clv, w.logits, 5000, w.parent, w.tokens, u, 1e-2, w.path_cap)
    ids = oracle.argmax(w.logits, 5000)
    alen, aidx, nxt, st = oracle.accept_walk(w.parent, w.tokens, ids, w.path_cap)
    assert np.array_equal(got[0], alen) and np.array_equal(got[1], aidx) and np.array_equal(got[2], nxt)
    assert np.array_equal(got[3], st)


def test_sample_special_values_and_bad_trees(clv, oracle):
    vocab, N, ld = 50, 4, 56
    lg = np.zeros((4, N, ld), np.uint16)
    lg[:] = W.f32_to_bf16_bits(np.random.default_rng(3).normal(0, 1, size=(4, N, ld)).astype(np.float32))
    lg[0, 0, 7] = 0xFF80                     # a logit of -inf carries no probability
    lg[0, 0, 9] = 0xFF80
    lg[1, 0, :] = 0xFF80                     # a row that is -inf except one entry: that entry is certain
    lg[1, 0, 33] = 0x3F80
    lg[:, :, vocab:] = 0x7F00
    parent = np.array([[-1, 0, 0, 1], [-1, 0, 0, 0], [-1, 2, 0, 1], [-1, 0, 1, 2]], np.int32)   # third: malformed
    tokens = np.array([[0, 7, 9, 3], [0, 5, 33, 6], [0, 1, 2, 3], [0, 4, 4, 4]], np.int32)
    u = W.make_uniforms(4, N, seed=11)
    u[0, 1] = 0.0                            # even u = 0 does not accept a token of probability zero
    u[0, 2] = 0.0
    got = run_gpu(clv, lg, vocab, parent, tokens, u, 1.0, N)
    alen, aidx, nxt, st, margin = oracle.accept_sample(lg, vocab, parent, tokens, u, 1.0, N)
    assert st.tolist() == [0, 0, 7, 0] and np.array_equal(got[3], st)
    ok = margin.min(axis=1) > MARGIN
    ok[0] = margin[0, 1] > MARGIN            # its accept tests have margin 0 but are exact: 0 < 0 is false
    assert np.array_equal(got[0][ok], alen[ok]) and np.array_equal(got[1][ok], aidx[ok])
    assert np.array_equal(got[2][ok], nxt[ok])
    assert got[0][0] == 1 and got[2][0] not in (7, 9)
    assert got[0][1] >= 2 and got[1][1, 1] == 2        # the certain token's child is accepted whatever u
    assert got[0][2] == 0 and got[2][2] == -1 and (got[1][2] == -1).all()


def test_sample_emitted_tokens_follow_the_target(clv):
    # many sequences with the same small tree and logits, each with its own uniforms: the first
    # emitted token (accepted child's token, or the drawn one) is distributed as the root's softmax
    B, N, vocab, ld = 20000, 5, 12, 16
    rng = np.random.default_rng(42)
    lg1 = np.zeros((N, ld), np.uint16)
    lg1[:, :vocab] = W.f32_to_bf16_bits(rng.normal(0, 1.3, size=(N, vocab)).astype(np.float32))
    lg1[:, vocab:] = 0xFF80
    parent1 = np.array([-1, 0, 0, 0, 1], np.int32)
    tokens1 = np.array([0, 3, 8, 1, 5], np.int32)
    lg = np.broadcast_to(lg1, (B, N, ld))
    parent = np.broadcast_to(parent1, (B, N))
    tokens = np.broadcast_to(tokens1, (B, N))
    u = W.make_uniforms(B, N, seed=99)
    got = run_gpu(clv, lg, vocab, parent, tokens, u, 1.0, N)
    alen, aidx, nxt = got[0], got[1], got[2]
    first = np.where(alen > 1, tokens1[aidx[:, 1].clip(0)], nxt)
    x = W.bf16_bits_to_f64(lg1[0, :vocab])
    p0 = np.exp(x - x.max())
    p0 /= p0.sum()
    freq = np.bincount(first, minlength=vocab)[:vocab] / B
    assert np.abs(freq - p0).max() < 5.0 * np.sqrt(0.25 / B)


def test_sample_then_commit(clv, oracle):
    # the accepted path of the stochastic walk drives clv_kv_commit like the greedy one does
    from paper_2408_00264_b200.step import VerifyStep, bits_of
    cfg = W.small_config(batch=4, n_q_heads=4, n_kv_heads=2, ctx=(20, 200), n_nodes=24, vocab=777,
                         seed=W.BASE_SEED + 5)
    w = W.generate(cfg)
    st = VerifyStep(w, device="cuda")
    u = W.make_uniforms(4, 24, seed=8)
    clv.clv_accept_sample(st.shape, st.logits, st.ld, st.parent, st.tokens, torch.from_numpy(u).cuda(), 1.0,
                          st.accept_len, st.accept_idx, st.next_token, st.status[1], st.workspace)
    st.kv_commit()
    torch.cuda.synchronize()
    alen, aidx, nxt, s1, margin = oracle.accept_sample(w.logits, 777, w.parent, w.tokens, u, 1.0, w.path_cap)
    assert (margin[:, 0] > MARGIN).all()      # no accept test near its threshold: the paths are unique
    kc, vc, new_len, s2 = oracle.kv_commit(w.k_cache, w.v_cache, w.k_tree, w.v_tree, aidx, alen, w.ctx_len)
    assert np.array_equal(st.accept_len.cpu().numpy(), alen) and np.array_equal(st.accept_idx.cpu().numpy(), aidx)
    sure = margin[:, 1] > MARGIN
    assert np.array_equal(st.next_token.cpu().numpy()[sure], nxt[sure])
    assert np.array_equal(st.ctx_len_out.cpu().numpy(), new_len)
    assert np.array_equal(bits_of(st.k_cache), kc) and np.array_equal(bits_of(st.v_cache), vc)
