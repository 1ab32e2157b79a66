"""Host logic of the multi-GPU run on CPU: two gloo ranks shard a batch without overlap and the
benchmark's whole-job figures are max-of-times and sum-of-bytes.  (Sequences are independent, so
the data path has no collective; only the timing reduction uses one.)"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2408_00264_b200 import workloads as W
    mine = list(W.shard_sequences(7, rank, world))
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    step, e2e, nbytes = bench.reduce_over_ranks(dist, "cpu", 10.0 + rank, 100.0 - rank, 1000.0 * (rank + 1))
    if rank == 0:
        out.put((gathered, step, e2e, nbytes))
    dist.destroy_process_group()


def test_two_ranks_shard_and_reduce():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    gathered, step, e2e, nbytes = out.get()
    assert sorted(gathered[0] + gathered[1]) == list(range(7)) and not set(gathered[0]) & set(gathered[1])
    assert step == 11.0 and e2e == 100.0 and nbytes == 3000.0


def test_gpus_flag_without_a_launcher_starts_its_own_ranks(monkeypatch):
    """`bench.py --gpus N` with no WORLD_SIZE in the environment must start N ranks itself (one per
    GPU, rendezvous on 127.0.0.1); under a launcher (WORLD_SIZE set) it must not."""
    import bench
    calls = []
    monkeypatch.setattr(bench, "launch_ranks", lambda world, argv: calls.append((world, list(argv))))
    monkeypatch.setattr(bench, "run_clv", lambda args: calls.append(("run", args.gpus)))
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    bench.main(["--gpus", "4", "--steps", "7"])
    assert calls == [(4, ["--gpus", "4", "--steps", "7"])]
    calls.clear()
    monkeypatch.setenv("WORLD_SIZE", "4")
    bench.main(["--gpus", "4", "--steps", "7"])
    assert calls == [("run", 4)]
    calls.clear()
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    bench.main(["--gpus", "1"])
    assert calls == [("run", 1)]
    env = bench.rank_env(2, 4, 29511)
    assert env == {"RANK": "2", "LOCAL_RANK": "2", "WORLD_SIZE": "4", "MASTER_ADDR": "127.0.0.1",
                   "MASTER_PORT": "29511"}
    assert 1024 < bench.free_port() < 65536
