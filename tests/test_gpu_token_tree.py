"""GPU parity of clv_build_token_tree against the CPU checker (bit-exact: integer work)."""
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


def run_gpu(clv, root, cand, lens, cap):
    B, C, D = cand.shape
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()  # noqa: E731
    out = [torch.full(s, -9, dtype=torch.int32, device="cuda")
           for s in ((B, cap), (B, cap), (B,), (B, C, D), (B,))]
    clv.clv_build_token_tree(dev(root), dev(cand), dev(lens), *out)
    torch.cuda.synchronize()
    return [t.cpu().numpy() for t in out]


def same(a, b):
    return all(np.array_equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("B,C,D,vocab,cap", [(1, 1, 1, 3, 2), (3, 7, 4, 3, 32), (4, 32, 6, 4, 128),
                                              (2, 64, 8, 2, 128), (5, 128, 16, 2, 128),
                                              (2, 33, 5, 1000, 128), (3, 100, 3, 6, 128)])
def test_matches_the_checker(clv, oracle, B, C, D, vocab, cap):
    root, cand, lens = W.make_candidates(B, C, D, vocab, seed=B * 1000 + C)
    want = oracle.build_token_tree(root, cand, lens, cap)
    got = run_gpu(clv, root, cand, lens, cap)
    assert same(got, want)
    assert set(want[4].tolist()) <= {0, 7}


def test_overflow_bad_lengths_and_duplicates(clv, oracle):
    root, cand, lens = W.make_candidates(4, 40, 6, 50, seed=5)      # few shared prefixes: many nodes
    for cap in (1, 5, 128):
        assert same(run_gpu(clv, root, cand, lens, cap), oracle.build_token_tree(root, cand, lens, cap))
    bad = lens.copy()
    bad[2, 3] = 7
    bad[0, 0] = -1
    got = run_gpu(clv, root, cand, bad, 128)
    assert same(got, oracle.build_token_tree(root, cand, bad, 128))
    assert got[4].tolist()[0] == 7 and got[4].tolist()[2] == 7
    cand[:, 1:] = cand[:, :1]                                       # all candidates equal: a chain
    lens[:, 1:] = lens[:, :1]
    got = run_gpu(clv, root, cand, lens, 64)
    assert same(got, oracle.build_token_tree(root, cand, lens, 64))
    assert (got[2] == lens[:, 0] + 1).all()


def test_built_tree_goes_through_the_verify_calls(clv, oracle):
    # tokens/parent with their padding are accepted as they are by the walk on the device
    root, cand, lens = W.make_candidates(3, 16, 5, 5, seed=13)
    cap = 64
    tok, par, n, node_of, st = run_gpu(clv, root, cand, lens, cap)
    ids = np.full((3, cap), 10 ** 6, dtype=np.int32)
    chains = []
    for b in range(3):
        c = int(np.argmax(lens[b]))
        L = int(lens[b, c])
        chain = [0] + [int(x) for x in node_of[b, c, :L]]
        for j in range(L):
            ids[b, chain[j]] = cand[b, c, j]
        chains.append(chain)
    shape = clv.make_shape(3, cap, 1, 1, vocab=8, path_cap=8)
    dev = lambda a: torch.from_numpy(a).cuda()  # noqa: E731
    alen = torch.zeros(3, dtype=torch.int32, device="cuda")
    aidx = torch.zeros(3, 8, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(3, dtype=torch.int32, device="cuda")
    wst = torch.zeros(3, dtype=torch.int32, device="cuda")
    clv.clv_accept_walk(shape, dev(par), dev(tok), dev(ids), alen, aidx, nxt, wst)
    torch.cuda.synchronize()
    assert wst.cpu().tolist() == [0, 0, 0]
    for b in range(3):
        assert alen[b].item() == len(chains[b])
        assert aidx[b, :len(chains[b])].cpu().tolist() == chains[b]
    ref = oracle.accept_walk(par, tok, ids, 8)
    assert np.array_equal(alen.cpu().numpy(), ref[0]) and np.array_equal(aidx.cpu().numpy(), ref[1])


def test_argument_errors(clv):
    z = lambda *s: torch.zeros(*s, dtype=torch.int32, device="cuda")  # noqa: E731
    args = (z(1), z(1, 200, 4), z(1, 200), z(1, 16), z(1, 16), z(1), z(1, 200, 4), z(1))
    assert clv.clv_build_token_tree(*args, check=False) != 0          # too many candidates
    args = (z(1), z(1, 4, 17), z(1, 4), z(1, 16), z(1, 16), z(1), z(1, 4, 17), z(1))
    assert clv.clv_build_token_tree(*args, check=False) != 0          # sequences too long
    args = (z(1), z(1, 4, 4), z(1, 4), z(1, 200), z(1, 200), z(1), z(1, 4, 4), z(1))
    assert clv.clv_build_token_tree(*args, check=False) != 0          # more than 128 nodes asked for
