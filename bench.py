#!/usr/bin/env python
"""Benchmark of the tree-verification step (tree attention -> argmax -> walk -> KV commit).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl clv|reference]

One "step" is one pass of all four calls over one batch of seeded synthetic input (LLaMA3-8B
shape by default: batch 4, GQA 32/8, context 4096, 64 tree nodes, vocabulary 128256).  Rank 0
prints one JSON line.  `value` is the achieved HBM throughput of the whole job: algorithmic bytes
of the step (each cached K/V byte, tree K/V, Q, O and every logit once) divided by step time, with
the inputs resident on the device; `e2e` is the same through the host-buffer entry point with the
copies inside the timed region.  Sequences are independent, so with N > 1 every rank runs its own
batch (weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "verify-step achieved HBM GB/s (algorithmic bytes / step time)"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
ROTATE = 4   # distinct input sets cycled between steps: 4 x 138 MB > 2 x L2 (126 MB)
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in
# profiles/verify_step_C3.md; valid for the kernels as they were when that capture was taken
NCU_TRAFFIC = {("C3", "tree_attn"): 71.7e6, ("C3", "accept_argmax"): 65.9e6}


def time_token_tree(batch, node_cap, dev):
    """clv_build_token_tree for `batch` sequences, 32 speculated sequences of up to 6 tokens each
    (latency bound: one small block per sequence): microseconds per launch, replayed from a graph."""
    import torch
    from paper_2408_00264_b200 import binding as clv
    from paper_2408_00264_b200 import workloads as W
    root, cand, lens = W.make_candidates(batch, 32, 6, 6, seed=W.BASE_SEED + 9)
    t = lambda a: torch.from_numpy(a).to(dev)  # noqa: E731
    ins = (t(root), t(cand), t(lens))
    outs = [torch.zeros(s, dtype=torch.int32, device=dev)
            for s in ((batch, node_cap), (batch, node_cap), (batch,), (batch, 32, 6), (batch,))]
    for _ in range(3):
        clv.clv_build_token_tree(*ins, *outs)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(8):
            clv.clv_build_token_tree(*ins, *outs)
    g.replay()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    torch.cuda.synchronize()
    a.record(cur)
    for _ in range(20):
        g.replay()
    b.record(cur)
    torch.cuda.synchronize()
    return {"batch": batch, "n_cand": 32, "max_len": 6, "node_cap": node_cap,
            "us": a.elapsed_time(b) / 160 * 1e3, "nodes": outs[2].cpu().tolist()[:4]}


def time_lm_head(rows, hidden, vocab, dev, args):
    """clv_lm_head_argmax on `rows` tree nodes: microseconds per launch (CUDA events, launches
    replayed from a CUDA graph over two copies of the weight matrix, 2 x 1.05 GB at vocabulary
    128256, so that no launch finds its weights in L2), with the rates against both roofs."""
    import torch
    from paper_2408_00264_b200 import binding as clv
    from paper_2408_00264_b200 import workloads as W
    h, w, win = W.make_lm_head(rows, hidden, vocab, seed=W.BASE_SEED + 77)
    hid = W.as_torch_bf16(h).to(dev)
    wgt = [W.as_torch_bf16(w).to(dev)]
    wgt.append(wgt[0].clone())
    ids = torch.zeros(rows, dtype=torch.int32, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = clv.new_workspace(clv.make_shape(1, 1, 1, 1, vocab=8), None, 0, dev)
    for i in range(4):
        clv.clv_lm_head_argmax(hid, wgt[i % 2], ids, st, ws)
    torch.cuda.synchronize()
    ok = bool((ids.cpu().numpy() == win).all()) and int(st.item()) == 0
    if args.no_graph:
        run = lambda: [clv.clv_lm_head_argmax(hid, wgt[i], ids, st, ws) for i in range(2)]  # noqa: E731
    else:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(2):
                clv.clv_lm_head_argmax(hid, wgt[i], ids, st, ws)
        run = g.replay
    run()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    torch.cuda.synchronize()
    reps = 10
    a.record(cur)
    for _ in range(reps):
        run()
    b.record(cur)
    torch.cuda.synchronize()
    us = a.elapsed_time(b) / (2 * reps) * 1e3
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except (OSError, ValueError):
        pass
    tf_peak, tf_kind = (peaks["bf16_tflops"], "measured") if "bf16_tflops" in peaks else (1590.0, "fallback")
    bw_peak, bw_kind = measured_peaks()
    tflops = 2.0 * rows * hidden * vocab / us / 1e6
    gbs = (vocab + rows) * hidden * 2 / us / 1e3
    return {"rows": rows, "hidden": hidden, "vocab": vocab, "us": us, "ids_match_planted_winners": ok,
            "tflops": tflops, "frac_of_bf16_peak": {"of_%s_%.0f_TFLOPs" % (tf_kind, tf_peak): tflops / tf_peak},
            "algorithmic_bytes": (vocab + rows) * hidden * 2 + rows * 4, "gbs": gbs,
            "frac_of_hbm_peak": {"of_%s_%.0f_GBps" % (bw_kind, bw_peak): gbs / bw_peak},
            "launches_timed": 2 * reps}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None
        self.period = period_s

    def _loop(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake": 0x80, "sw_power_cap": 0x4}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self):
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------- reference arm
def oracle_sample_step(orc, w, n_attn_rows: int, n_logit_rows: int, seq: int = 0):
    """One bounded sample of the step on the CPU checker: some attention rows and logits rows of
    one sequence, then that sequence's walk and commit.  Returns algorithmic bytes covered."""
    c = w.cfg
    rows = np.array([(seq, (r // c.n_q_heads) % c.n_nodes, r % c.n_q_heads)
                     for r in range(n_attn_rows)], dtype=np.int32)
    orc.tree_attn(w.q, w.k_cache, w.v_cache, w.k_tree, w.v_tree, w.parent, w.ctx_len, w.scale,
                  block_table=w.block_table, rows=rows)
    ids = orc.argmax(w.logits[seq, :n_logit_rows], c.vocab)
    full = np.zeros((1, c.n_nodes), np.int32)
    full[0, :n_logit_rows] = ids
    orc.accept_walk(w.parent[seq:seq + 1], w.tokens[seq:seq + 1], full, w.path_cap)
    total = w.algorithmic_bytes()
    frac_attn = n_attn_rows / float(c.batch * c.n_nodes * c.n_q_heads)
    frac_lg = n_logit_rows / float(c.batch * c.n_nodes)
    return total["attn"] * frac_attn + total["logits"] * frac_lg


def time_oracle(orc, w, steps: int, warmup: int, budget_s: float):
    """Times `steps` sample-steps of the checker, the sample sized so the run fits the budget."""
    c = w.cfg
    t0 = time.perf_counter()
    oracle_sample_step(orc, w, 32, 1)
    t_unit = max(time.perf_counter() - t0, 1e-4)          # 32 attention rows + 1 logits row
    per_step = budget_s / max(1, steps + warmup)
    k = max(1.0 / 32.0, per_step / t_unit)
    n_attn = int(min(c.n_nodes * c.n_q_heads, max(1, round(32 * k))))
    n_lg = int(min(c.n_nodes, max(1, round(k))))
    for _ in range(warmup):
        oracle_sample_step(orc, w, n_attn, n_lg)
    nbytes = 0.0
    t0 = time.perf_counter()
    for _ in range(steps):
        nbytes += oracle_sample_step(orc, w, n_attn, n_lg)
    dt = time.perf_counter() - t0
    sample = ("%d attention rows (b,node,head) + %d logits rows of sequence 0 per step, plus its "
              "walk; bytes scaled by the covered fraction" % (n_attn, n_lg))
    return nbytes / dt / 1e9, dt / steps * 1e3, sample


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as orc
    from paper_2408_00264_b200 import workloads as W
    orc.build()
    w = W.generate(W.CONFIGS[args.workload])
    gbs, ms, sample = time_oracle(orc, w, args.steps, args.warmup, budget_s=90.0)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": orc.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w):
    c = w.cfg
    return {"workload": "%s: LLaMA3-8B-shaped verify step" % c.name if c.name == "C3" else c.name,
            "batch": c.batch, "n_q_heads": c.n_q_heads, "n_kv_heads": c.n_kv_heads,
            "head_dim": c.head_dim, "ctx_len": (int(w.ctx_len.min()), int(w.ctx_len.max())),
            "tree_nodes": c.n_nodes, "vocab": c.vocab, "paged": bool(c.paged),
            "cache_policy": "inputs rotate over %d distinct buffer sets (> 2x L2) between steps"
                            % ROTATE}


def reduce_over_ranks(dist, device, step_ms, e2e_ms, local_bytes):
    """Whole-job figures from per-rank ones: the slowest rank sets the time (max), the bytes of all
    ranks add up (every rank runs its own batch; there is no other exchange)."""
    if dist is None:
        return step_ms, e2e_ms, local_bytes
    import torch
    t = torch.tensor([step_ms, e2e_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    tot = torch.tensor([local_bytes], device=device, dtype=torch.float64)
    dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), float(tot[0])


# ----------------------------------------------------------------------------- device arm
def run_clv(args):
    import torch
    from paper_2408_00264_b200 import binding as clv
    from paper_2408_00264_b200 import workloads as W
    from paper_2408_00264_b200.step import VerifyStep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    clv.lib()

    import dataclasses
    cfg = dataclasses.replace(W.CONFIGS[args.workload], seed=W.CONFIGS[args.workload].seed + rank)
    w = W.generate(cfg)
    sets = [VerifyStep(w, device=dev, with_lse=False) for _ in range(ROTATE)]
    nbytes = w.algorithmic_bytes()
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- whole step, inputs resident -------------------------------------------------------
    for i in range(max(args.warmup, 3)):
        sets[i % ROTATE].run()
    torch.cuda.synchronize()
    graphs = None
    if not args.no_graph:
        graphs = []
        for s in sets:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                s.run()
            graphs.append(g)
        for i in range(max(args.warmup, 3)):
            graphs[i % ROTATE].replay()
        stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with ClockSampler(local) as clocks:
        e0.record(stream)
        if graphs is not None:
            for i in range(args.steps):
                graphs[i % ROTATE].replay()
        else:
            for i in range(args.steps):
                sets[i % ROTATE].run()
        e1.record(stream)
        barrier()
    step_ms = e0.elapsed_time(e1) / args.steps

    # ---- each call alone, back to back over the rotating sets (same stream) -----------------
    def time_call(name, n):
        """Microseconds per launch of one call, back to back over the rotating input sets.  The
        launches are replayed from a CUDA graph (one launch per input set) so that host launch
        overhead does not set the pace of the short kernels."""
        for i in range(3):
            getattr(sets[i % ROTATE], name)()
        torch.cuda.synchronize()
        if args.no_graph:
            run, per = (lambda: [getattr(sets[i], name)() for i in range(ROTATE)]), ROTATE
        else:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(ROTATE):
                    getattr(sets[i], name)()
            run, per = g.replay, ROTATE
        run()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cur = torch.cuda.current_stream()
        torch.cuda.synchronize()
        a.record(cur)
        reps = max(1, n // per)
        for _ in range(reps):
            run()
        b.record(cur)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * per) * 1e3
    n_k = max(20, min(args.steps, 400))
    call_us = {k: time_call(k, n_k) for k in ("tree_attn", "accept_argmax", "accept_walk", "kv_commit")}

    # ---- end to end from pinned host buffers ------------------------------------------------
    c = w.cfg
    B, N = c.batch, c.n_nodes
    pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()  # noqa: E731
    host = [pin(x) for x in (w.q, w.k_tree, w.v_tree, w.parent, w.tokens, w.logits)]
    o_out = torch.empty(B, N, c.n_q_heads, 128, dtype=torch.int16).pin_memory()
    o_ids = torch.empty(B, N, dtype=torch.int32).pin_memory()
    o_len = torch.empty(B, dtype=torch.int32).pin_memory()
    o_idx = torch.empty(B, w.path_cap, dtype=torch.int32).pin_memory()
    o_nxt = torch.empty(B, dtype=torch.int32).pin_memory()
    o_st = torch.empty(3, B, dtype=torch.int32).pin_memory()
    hin = clv.ClvHostInputs(*[t.data_ptr() for t in host], w.logits.shape[-1])
    hout = clv.ClvHostOutputs(o_out.data_ptr(), o_ids.data_ptr(), o_len.data_ptr(), o_idx.data_ptr(),
                              o_nxt.data_ptr(), o_st.data_ptr())
    s0 = sets[0]
    staging = torch.empty(clv.clv_staging_bytes(s0.shape, w.logits.shape[-1]), dtype=torch.uint8,
                          device=dev)
    ctx0 = s0.ctx_len.clone()
    h2d = sum(t.numel() * t.element_size() for t in host)
    d2h = sum(t.numel() * t.element_size() for t in (o_out, o_ids, o_len, o_idx, o_nxt, o_st))
    n_e2e = 0 if args.no_e2e else max(3, min(args.steps, 50))

    def host_step():
        s0.ctx_len.copy_(ctx0, non_blocking=True)   # keep the context length fixed across steps
        clv.clv_verify_step_host(s0.shape, s0.cache, hin, hout, s0.ctx_len, s0.max_ctx_len, s0.scale,
                                 staging, s0.workspace)
    e2e_ms = float("nan")
    if n_e2e:
        for _ in range(3):
            host_step()
        barrier()
        e0.record(stream)
        for _ in range(n_e2e):
            host_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / n_e2e

    # ---- the step before the argmax: LM head fused with the greedy choice (rank 0 only) ---------
    lm_head = None
    tree_us = None
    if rank == 0 and not args.no_lm_head:
        lm_head = time_lm_head(B * N, 4096, c.vocab, dev, args)
        tree_us = time_token_tree(B, 128, dev)

    # ---- max over ranks ------------------------------------------------------------------------
    step_ms, e2e_ms, job_bytes = reduce_over_ranks(dist, dev, step_ms, e2e_ms, float(nbytes["total"]))
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    value = job_bytes / (step_ms * 1e-3) / 1e9
    dom = "tree_attn" if call_us["tree_attn"] >= call_us["accept_argmax"] else "accept_argmax"
    dom_bytes = nbytes["attn"] if dom == "tree_attn" else nbytes["logits"]
    achieved = dom_bytes / (call_us[dom] * 1e-6) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w),
        "step_us": step_ms * 1e3,
        "tree_tokens_per_s": world * B * N / (step_ms * 1e-3),
        "frac_of_hbm_peak": {"of_%s_%.0f_GBps" % (peak_kind, peak): value / world / peak,
                             "of_nominal_8000_GBps": value / world / NOMINAL_HBM_GBS},
        "call_us": call_us, "launch_mode": "per-call" if graphs is None else "cuda-graph replay",
        "step_schedule": "clv_tree_attn, clv_accept_argmax, clv_accept_walk_commit (walk and commit in one launch) on one stream",
        "algorithmic_bytes": nbytes,
        "roofline": {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": peak,
                     "peak_source": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": NCU_TRAFFIC.get((args.workload, dom))},
        "e2e": {"value": job_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                "steps": n_e2e},
        "next_rows": {"lm_head_argmax": lm_head, "build_token_tree": tree_us},
        "gpu_launches": 3 * args.steps,   # attention, argmax, walk + commit in one launch
        "clocks": clocks.summary(),
    }
    if not args.no_cpu_baseline and world == 1:
        import oracle as orc
        orc.build()
        gbs, ms, sample = time_oracle(orc, w, steps=3, warmup=1, budget_s=16.0)
        line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": orc.threads(),
                                "kind": "oracle", "sample": sample}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="C3", choices=["C1", "C2", "C3", "C4", "C5"])
    ap.add_argument("--impl", default="clv", choices=["clv", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch the four calls per step directly")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lm-head", action="store_true",
                    help="skip the timing of clv_lm_head_argmax (hidden 4096, the workload's rows and vocabulary)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer timing (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_clv(args)


if __name__ == "__main__":
    main()
