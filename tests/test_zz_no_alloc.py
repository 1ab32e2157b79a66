"""The argmax entry point for callers that cannot allocate device memory.

Some users of the library run where device allocation is off the table at call time: inside an
engine that gave the whole GPU to its own memory pool at start-up, as a plug-in that only ever
receives input and output tensors, or on a latency path that must not hit cudaMalloc's implicit
synchronisation.  `clv_accept_argmax_noalloc` keeps its counters and partial results in a fixed
array inside the library instead of a workspace.  This file checks, through the C ABI, that it
returns exactly what `clv_accept_argmax` returns, twice in a row (the array keeps the previous
call's contents), that it refuses problems beyond its fixed capacity, that a call leaves the free
device memory unchanged and that a call can be recorded in a CUDA graph and replayed.

The file name sorts last on purpose, so a run that stops at the first failure has already
executed every other test.
"""
import numpy as np
import pytest
import torch

from paper_2408_00264_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def clv():
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    from paper_2408_00264_b200 import binding
    binding.lib()
    return binding


def _logits(rows, vocab, seed):
    rng = np.random.default_rng(seed)
    winner = rng.integers(0, vocab, size=rows)
    ld = (vocab + 7) // 8 * 8
    return W.make_logits(rows, vocab, ld, winner, 0.5, seed=seed + 1), ld


@pytest.mark.parametrize("batch,nodes,vocab", [(2, 5, 2049), (4, 64, 128256), (1, 16, 32000)])
def test_noalloc_matches_workspace_entry_point_twice(clv, oracle, batch, nodes, vocab):
    shape = clv.make_shape(batch, nodes, 1, 1, vocab, 1)
    ws = clv.new_workspace(shape, None, 0)
    ids_ref = torch.empty(batch, nodes, dtype=torch.int32, device="cuda")
    ids_new = torch.full((batch, nodes), -7, dtype=torch.int32, device="cuda")
    for call in range(2):                       # second call: different data, same built-in array
        lg, ld = _logits(batch * nodes, vocab, seed=100 * call + vocab)
        if call == 1:
            lg[0, :] = 0x3F80                   # a row of equal values: the lowest index must win
        d = torch.from_numpy(lg.view(np.int16)).cuda()
        clv.clv_accept_argmax(shape, d, ld, ids_ref, ws)
        ids_new.fill_(-7)
        clv.clv_accept_argmax_noalloc(shape, d, ld, ids_new)
        torch.cuda.synchronize()
        assert torch.equal(ids_new, ids_ref)    # integer output: exact
        assert int(ids_new.min()) >= 0 and int(ids_new.max()) < vocab
        # and both are what the CPU checker finds, so this file stands on its own
        assert np.array_equal(ids_new.cpu().numpy().reshape(-1), oracle.argmax(lg, vocab))


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch(clv):
    d = torch.zeros(16, dtype=torch.int16, device="cuda")
    ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    too_many_rows = clv.make_shape(64, 128, 1, 1, 32000, 1)          # 8192 rows > 4096
    code = clv.clv_accept_argmax_noalloc(too_many_rows, d, 32000, ids, check=False)
    assert code == clv.CLV_ERR_TOO_LARGE
    assert "scratch" in clv.clv_status_string(code)
    with pytest.raises(clv.ClvError):
        clv.clv_accept_argmax_noalloc(too_many_rows, d, 32000, ids)
    # as many rows as allowed, but a vocabulary so wide that rows x (thread blocks per row)
    # exceeds the array: 4096 rows x 33 pieces of 32768 logits
    too_many_pieces = clv.make_shape(32, 128, 1, 1, 33 * 32768, 1)
    code = clv.clv_accept_argmax_noalloc(too_many_pieces, d, 33 * 32768, ids, check=False)
    assert code == clv.CLV_ERR_TOO_LARGE


def test_noalloc_allocates_nothing(clv):
    # the point of the entry point: the free device memory is the same before and after a call
    # (the first call on the device has already been made by the tests above or is made here)
    vocab, rows = 32000, 16
    lg, ld = _logits(rows, vocab, seed=5)
    d = torch.from_numpy(lg.view(np.int16)).cuda()
    shape = clv.make_shape(1, rows, 1, 1, vocab, 1)
    ids = torch.empty(1, rows, dtype=torch.int32, device="cuda")
    clv.clv_accept_argmax_noalloc(shape, d, ld, ids)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    clv.clv_accept_argmax_noalloc(shape, d, ld, ids)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_noalloc_call_can_be_captured_in_a_graph(clv, oracle):
    # after the first call on the device (which looks up the array's address) a call is a clearing
    # of the counters and a launch on the caller's stream: both can be recorded and replayed
    vocab, rows = 5000, 24
    lg, ld = _logits(rows, vocab, seed=9)
    d = torch.from_numpy(lg.view(np.int16)).cuda()
    shape = clv.make_shape(1, rows, 1, 1, vocab, 1)
    ids = torch.full((1, rows), -7, dtype=torch.int32, device="cuda")
    clv.clv_accept_argmax_noalloc(shape, d, ld, ids)      # warm-up, outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        clv.clv_accept_argmax_noalloc(shape, d, ld, ids)
    for seed in (10, 11):                                  # new data in the same buffer, replayed twice
        lg2, _ = _logits(rows, vocab, seed=seed)
        d.copy_(torch.from_numpy(lg2.view(np.int16)))
        ids.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(ids.cpu().numpy().reshape(-1), oracle.argmax(lg2, vocab))
