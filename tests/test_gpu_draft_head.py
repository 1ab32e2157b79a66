"""GPU parity of clv_draft_head_step (one step of a Clover-2 draft head) against the CPU checker.

The checker works in float64 throughout; the kernels round the operands of each product to bf16
once (like the activations of a bf16 model) and accumulate in fp32.  So the hidden state is
compared within the attention's tolerance (row-normalised 1e-2), the logits of the proposals within
TOL of the row's largest magnitude, and the proposals themselves must be the checker's wherever its
logits are further apart than that; elsewhere every proposed token must be one the checker ranks
within TOL of its k-th best."""
import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W

pytestmark = pytest.mark.gpu
TOL = 1e-2


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


def run_gpu(clv, h, e, wts, k_top):
    R, H = h.shape
    V = wts["lm_head"].shape[0]
    dw = {n: (v if n == "n_heads" else W.as_torch_bf16(v).cuda()) for n, v in wts.items()}
    head = clv.make_draft_head(dw)
    ws = clv.new_draft_head_workspace(R, H, V)
    hid = torch.empty(R, H, dtype=torch.bfloat16, device="cuda")
    ids = torch.full((R, k_top), -9, dtype=torch.int32, device="cuda")
    vals = torch.zeros(R, k_top, dtype=torch.float32, device="cuda")
    st = torch.full((5,), -9, dtype=torch.int32, device="cuda")
    dh, de = W.as_torch_bf16(h).cuda(), W.as_torch_bf16(e).cuda()
    for _ in range(2):                      # the workspace is reusable as is
        clv.clv_draft_head_step(head, dh, de, k_top, hid, ids, vals, st, ws)
    torch.cuda.synchronize()
    assert st.cpu().tolist() == [0] * 5
    return hid.float().cpu().numpy().astype(np.float64), ids.cpu().numpy(), vals.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("R,H,nh,V,k", [(3, 64, 4, 500, 5), (16, 256, 8, 3000, 8), (5, 128, 2, 777, 1),
                                         (130, 128, 4, 1000, 4), (8, 4096, 32, 128256, 8),
                                         (4, 64, 4, 9000, 32),      # the widest one-pass selection, two levels
                                         (2, 64, 2, 3000, 40),      # beyond it: one pass per proposal
                                         (70, 192, 48, 2049, 2),    # head size 4; one entry in the second slice
                                         (1, 64, 1, 100, 3), (256, 64, 2, 300, 3)])   # fewest and most rows
def test_draft_head_step(clv, oracle, R, H, nh, V, k):
    h, e, wts = W.make_draft_head(R, H, nh, V, seed=R + H + V)
    p, ids, vals, logits = oracle.draft_head_step(h, e, wts, k)
    hid, g_ids, g_vals = run_gpu(clv, h, e, wts, k)
    row_rel = np.abs(hid - p).max(axis=1) / np.abs(p).max(axis=1)
    assert row_rel.max() <= 1e-2, row_rel.max()
    for r in range(R):
        scale = np.abs(logits[r]).max()
        tol = TOL * scale
        assert len(set(g_ids[r].tolist())) == k and g_ids[r].min() >= 0 and g_ids[r].max() < V
        assert np.abs(g_vals[r] - logits[r, g_ids[r]]).max() <= tol           # the logits it reports
        assert (np.diff(g_vals[r]) <= 0).all()                               # highest first
        order = np.sort(logits[r])[::-1]
        gaps = order[:k] - order[1:k + 1]                                    # k-th against (k+1)-th included
        if gaps.min() > 2 * tol:
            assert np.array_equal(g_ids[r], ids[r])
        else:
            assert (logits[r, g_ids[r]] >= vals[r, k - 1] - 2 * tol).all()  # every proposal is a near-top token


def test_draft_head_step_planted_proposals_and_errors(clv, oracle):
    # rows whose best tokens lead clearly: the proposals must be exactly the checker's
    R, H, nh, V, k = 6, 128, 4, 2000, 3
    h, e, wts = W.make_draft_head(R, H, nh, V, seed=77)
    _, _, _, logits = oracle.draft_head_step(h, e, wts, k)
    # make three vocabulary rows multiples of the first rows' normalised state: huge logits there
    p, _, _, _ = oracle.draft_head_step(h, e, wts, k)
    y = p / np.sqrt((p * p).mean(-1, keepdims=True) + 1e-5) * W.bf16_bits_to_f64(wts["norm2"])
    lm = W.bf16_bits_to_f64(wts["lm_head"]).copy()
    for j, t in enumerate((5, 1500, 1999)):
        lm[t] = y[0] * (3.0 - j) / np.sqrt(H)
    wts["lm_head"] = W.f32_to_bf16_bits(lm.astype(np.float32))
    _, ids, vals, logits = oracle.draft_head_step(h, e, wts, k)
    assert ids[0].tolist() == [5, 1500, 1999]
    hid, g_ids, g_vals = run_gpu(clv, h, e, wts, k)
    assert g_ids[0].tolist() == [5, 1500, 1999]
    # host-detectable mistakes
    dw = {n: (v if n == "n_heads" else W.as_torch_bf16(v).cuda()) for n, v in wts.items()}
    head = clv.make_draft_head(dw)
    ws = clv.new_draft_head_workspace(R, H, V)
    t = lambda *s, dt=torch.bfloat16: torch.zeros(*s, dtype=dt, device="cuda")  # noqa: E731
    args = (t(R, H), t(R, H), k, t(R, H), t(R, k, dt=torch.int32), t(R, k, dt=torch.float32), t(5, dt=torch.int32))
    assert clv.clv_draft_head_step(head, *args, ws[:1024], check=False) == clv.CLV_ERR_WORKSPACE
    bad = clv.make_draft_head(dw)
    bad.n_heads = 3                                          # does not divide the hidden size
    assert clv.clv_draft_head_step(bad, *args, ws, check=False) == clv.CLV_ERR_UNSUPPORTED
    assert clv.clv_draft_head_step(head, t(R, H), t(R, H), 65, t(R, H), t(R, 65, dt=torch.int32),
                                   t(R, 65, dt=torch.float32), t(5, dt=torch.int32), ws, check=False) == clv.CLV_ERR_UNSUPPORTED


def test_draft_head_step_equal_logits_rank_by_index(clv, oracle):
    # vocabulary rows that are copies of one another give equal logits on both sides (the same
    # products in the same order): the proposals must list them lower index first
    R, H, nh, V, k = 4, 128, 4, 4500, 6
    h, e, wts = W.make_draft_head(R, H, nh, V, seed=311)
    p, _, _, _ = oracle.draft_head_step(h, e, wts, k)
    y = p / np.sqrt((p * p).mean(-1, keepdims=True) + 1e-5) * W.bf16_bits_to_f64(wts["norm2"])
    lm = W.bf16_bits_to_f64(wts["lm_head"]).copy()
    copies = (4100, 17, 2047, 2048, 3333)                    # in different slices and next to a slice edge
    for t in copies:
        lm[t] = y[1] * 2.5 / np.sqrt(H)
    wts["lm_head"] = W.f32_to_bf16_bits(lm.astype(np.float32))
    _, ids, vals, logits = oracle.draft_head_step(h, e, wts, k)
    assert ids[1, :5].tolist() == sorted(copies)
    hid, g_ids, g_vals = run_gpu(clv, h, e, wts, k)
    assert g_ids[1, :5].tolist() == sorted(copies) and (g_vals[1, :5] == g_vals[1, 0]).all()
    for r in range(R):
        same = np.diff(g_vals[r]) == 0
        assert (np.diff(g_ids[r])[same] > 0).all()
