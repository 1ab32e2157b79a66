"""GPU parity of clv_lm_head_argmax (LM head fused with the greedy choice) against the CPU checker."""
import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def clv():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2408_00264_b200 import binding
    binding.lib()
    return binding


def run_gpu(clv, h_bits, w_bits, ld_pad=0):
    rows, K = h_bits.shape
    V = w_bits.shape[0]
    hid = torch.zeros(rows, K + ld_pad, dtype=torch.bfloat16, device="cuda")
    hid[:, :K] = W.as_torch_bf16(h_bits).cuda()
    wgt = torch.zeros(V, K + ld_pad, dtype=torch.bfloat16, device="cuda")
    wgt[:, :K] = W.as_torch_bf16(w_bits).cuda()
    ids = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    status = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    shape = clv.make_shape(1, 1, 1, 1, vocab=8)
    ws = clv.new_workspace(shape, None, 0)
    for _ in range(2):   # twice: the second call finds the workspace as the first left it
        clv.clv_lm_head_argmax(hid[:, :K], wgt[:, :K], ids, status, ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return ids.cpu().numpy()


def check_rows(oracle, h_bits, w_bits, got, rows=None):
    """Exact where the checker's best logit leads by more than two bf16 steps; elsewhere the GPU's
    choice must be a logit that rounds to the maximum (fp32 accumulation can move a logit across a
    rounding boundary, nothing more) and, among equally rounded ones within reach, any is valid."""
    sel = np.arange(h_bits.shape[0]) if rows is None else np.asarray(rows)
    ids, z = oracle.lm_head_argmax(h_bits, w_bits, rows=sel.astype(np.int32), want_logits=True)
    n_exact = 0
    for i, r in enumerate(sel):
        zr = z[i]
        top = zr.max()
        step = 2.0 ** (np.floor(np.log2(max(abs(top), 1e-30))) - 7)   # bf16 spacing at the maximum
        near = np.flatnonzero(zr >= top - 2 * step)
        if len(near) == 1:
            assert got[r] == ids[i] == near[0], (r, got[r], ids[i])
            n_exact += 1
        else:
            assert got[r] in near, (r, got[r], near)
    return n_exact


@pytest.mark.parametrize("rows,K,V", [(1, 64, 10), (5, 128, 255), (128, 64, 256), (129, 192, 257),
                                       (300, 256, 1000), (64, 4096, 1500), (700, 128, 5000)])
def test_planted_winners_exact(clv, oracle, rows, K, V):
    h, w, win = W.make_lm_head(rows, K, V, seed=100 + rows + V)
    got = run_gpu(clv, h, w, ld_pad=8 if rows % 2 else 0)
    assert np.array_equal(got, win)
    assert np.array_equal(oracle.lm_head_argmax(h, w), win)


def test_unplanted_rows_are_valid_choices(clv, oracle):
    h, w, _ = W.make_lm_head(200, 512, 4000, seed=77, planted=0.0)
    got = run_gpu(clv, h, w)
    assert check_rows(oracle, h, w, got) > 100


def test_ties_and_special_values(clv, oracle):
    K, V = 64, 600
    rng = np.random.default_rng(9)
    hid = np.zeros((4, K), dtype=np.float32)
    hid[:, 0] = 1.0
    w = np.zeros((V, K), dtype=np.float32)
    w[:, 0] = rng.integers(-3, 3, size=V).astype(np.float32)   # many exact ties at the maximum 2
    w[[17, 300, 599], 0] = 5.0                                   # equal logits in different tiles
    hb, wb = W.f32_to_bf16_bits(hid), W.f32_to_bf16_bits(w)
    got = run_gpu(clv, hb, wb)
    assert np.array_equal(got, oracle.lm_head_argmax(hb, wb))
    assert (got == 17).all()
    # a row of zeros (every logit +0) takes index 0; -0 and +0 are equal
    hid[1] = 0.0
    w[0, 0] = -1.0
    hb, wb = W.f32_to_bf16_bits(hid), W.f32_to_bf16_bits(w)
    got = run_gpu(clv, hb, wb)
    assert np.array_equal(got, oracle.lm_head_argmax(hb, wb))
    assert got[1] == 0


def test_best_two_logits_one_bf16_step_apart(clv, oracle):
    # Built, not drawn: every product and sum below is exact in fp32, so the GPU must pick the
    # checker's index although the two best logits are neighbouring bf16 numbers (1.75 and
    # 1.75 + 2^-7): this is the near-tie branch of check_rows, entered on purpose, in both orders
    # of the two candidates and with the candidates in different 256-entry tiles.
    K, V = 64, 700
    hid = np.zeros((4, K), dtype=np.float32)
    hid[:, :3] = 1.0
    w = np.zeros((V, K), dtype=np.float32)
    w[:, 0] = 1.0                                    # every other logit is 1.0
    lo = np.array([1.0, 0.5, 0.25], dtype=np.float32)            # sums to 1.75
    hi = np.array([1.0, 0.5, 0.25 + 2.0 ** -7], dtype=np.float32)  # one bf16 step above
    cases = [(100, 300), (300, 100), (5, 6), (699, 0)]           # (index of hi, index of lo)
    got_all, ref_all = [], []
    for i_hi, i_lo in cases:
        wc = w.copy()
        wc[i_hi, :3] = hi
        wc[i_lo, :3] = lo
        hb, wb = W.f32_to_bf16_bits(hid), W.f32_to_bf16_bits(wc)
        got = run_gpu(clv, hb, wb)
        ref, z = oracle.lm_head_argmax(hb, wb, want_logits=True)
        assert z[0, i_hi] - z[0, i_lo] == 2.0 ** -7
        assert check_rows(oracle, hb, wb, got) == 0      # no row has a clear winner ...
        assert np.array_equal(got, ref) and (got == i_hi).all()   # ... and yet the choice is exact
        got_all.append(got)
        ref_all.append(ref)


def test_unplanted_rows_agree_with_the_checker_almost_everywhere(clv, oracle):
    # drawn logits, no planted winner: the exact index wherever the lead is clear, a logit within
    # reach of the maximum elsewhere, and the two sides may differ only on such near ties
    h, w, _ = W.make_lm_head(300, 256, 6000, seed=78, planted=0.0)
    got = run_gpu(clv, h, w)
    n_exact = check_rows(oracle, h, w, got)
    ref = oracle.lm_head_argmax(h, w)
    assert n_exact >= 150
    assert (got == ref).mean() >= 0.9


def test_wait_that_runs_out_is_reported_and_leaves_the_library_usable(clv, oracle):
    # the kernel's waits are bounded; with the bound cut to a few dozen SM cycles the wait for the
    # first weight tile runs out: the call succeeds, status says CLV_ERR_TIMEOUT, nothing faults,
    # and the same workspace serves an ordinary call right afterwards
    h, w, win = W.make_lm_head(40, 128, 3000, seed=41)
    hid, wgt = W.as_torch_bf16(h).cuda(), W.as_torch_bf16(w).cuda()
    ids = torch.full((40,), -7, dtype=torch.int32, device="cuda")
    status = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    ws = clv.new_workspace(clv.make_shape(1, 1, 1, 1, vocab=8), None, 0)
    try:
        clv.clv_test_set_wait_limit(32)
        clv.clv_lm_head_argmax(hid, wgt, ids, status, ws)
        torch.cuda.synchronize()
    finally:
        clv.clv_test_set_wait_limit(0)
    assert int(status.item()) == clv.CLV_ERR_TIMEOUT
    clv.clv_lm_head_argmax(hid, wgt, ids, status, ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(ids.cpu().numpy(), win)
    assert np.array_equal(ids.cpu().numpy(), oracle.lm_head_argmax(h, w))


def test_full_size_sampled_rows(clv, oracle):
    # the shape the bench times: 256 tree nodes, hidden 4096, vocabulary 128256
    h, w, win = W.make_lm_head(256, 4096, 128256, seed=W.BASE_SEED + 3000)
    got = run_gpu(clv, h, w)
    assert np.array_equal(got, win)
    sel = np.array([0, 127, 128, 255], dtype=np.int32)
    assert np.array_equal(oracle.lm_head_argmax(h, w, rows=sel), win[sel])


def test_argument_errors(clv):
    hid = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    wgt = torch.zeros(10, 64, dtype=torch.bfloat16, device="cuda")
    ids = torch.zeros(4, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = clv.new_workspace(clv.make_shape(1, 1, 1, 1, vocab=8), None, 0)
    assert clv.clv_lm_head_argmax(hid, wgt, ids, status, None, check=False) != 0
    bad = torch.zeros(4, 72, dtype=torch.bfloat16, device="cuda")[:, :40]   # hidden size not a multiple of 64
    badw = torch.zeros(10, 72, dtype=torch.bfloat16, device="cuda")[:, :40]
    assert clv.clv_lm_head_argmax(bad, badw, ids, status, ws, check=False) != 0
    assert clv.clv_lm_head_argmax(hid, wgt, ids, status, ws, check=False) == 0
    torch.cuda.synchronize()
