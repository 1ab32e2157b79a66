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
ROTATE = 32  # at most this many distinct input sets are cycled between steps
L2_BYTES = 126e6

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


def time_accept_sample(w, dev):
    """clv_accept_sample (temperature 1) on the workload's logits and trees: microseconds per call
    (two launches: the statistics pass streams every logit once, then one block per sequence walks),
    replayed from a CUDA graph over two copies of the logits."""
    import torch
    from paper_2408_00264_b200 import binding as clv
    from paper_2408_00264_b200 import workloads as W
    c = w.cfg
    B, N = c.batch, c.n_nodes
    shape = clv.make_shape(B, N, c.n_q_heads, c.n_kv_heads, c.vocab, w.path_cap)
    ws = clv.new_workspace(shape, None, 0, dev)
    lg = [torch.from_numpy(w.logits.view(np.int16)).to(dev)]
    lg.append(lg[0].clone())
    t = lambda a: torch.from_numpy(a).to(dev)  # noqa: E731
    parent, tokens, u = t(w.parent), t(w.tokens), t(W.make_uniforms(B, N, seed=W.BASE_SEED + 3))
    i32 = dict(dtype=torch.int32, device=dev)
    outs = [torch.zeros(B, **i32), torch.zeros(B, w.path_cap, **i32), torch.zeros(B, **i32), torch.zeros(B, **i32)]
    call = lambda i: clv.clv_accept_sample(shape, lg[i], w.logits.shape[-1], parent, tokens, u, 1.0, *outs, ws)  # noqa: E731
    for i in range(4):
        call(i % 2)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(2):
            call(i)
    g.replay()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    torch.cuda.synchronize()
    a.record(cur)
    for _ in range(20):
        g.replay()
    b.record(cur)
    torch.cuda.synchronize()
    us = a.elapsed_time(b) / 40 * 1e3
    nbytes = B * N * c.vocab * 2
    return {"batch": B, "n_nodes": N, "vocab": c.vocab, "temperature": 1.0, "us": us, "launches_per_call": 2,
            "accept_len": outs[0].cpu().tolist()[:8], "logits_bytes": nbytes, "gbs_of_logits_stream": nbytes / us / 1e3}


def time_model_step(w, n_layers, dev):
    """Whole-model verify step on the workload's shape: clv_tree_attn per layer (each layer its own
    Q, tree K/V and cache), clv_lm_head_argmax (hidden 4096), walk, one commit for all layers; one
    CUDA graph, replayed.  With 32 layers of C3 the caches alone are 2.1 GB, so every launch is cold."""
    import torch
    from paper_2408_00264_b200 import workloads as W
    from paper_2408_00264_b200.step import ModelVerifyStep
    c = w.cfg
    layers = W.layer_tensors(w, n_layers)
    h, wt, _ = W.make_lm_head(c.batch * c.n_nodes, 4096, c.vocab, seed=W.BASE_SEED + 78)
    st = ModelVerifyStep(w, layers, h, wt, device=dev)
    for _ in range(2):
        st.run()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        st.run()
    g.replay()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    torch.cuda.synchronize()
    reps = 10
    a.record(cur)
    for _ in range(reps):
        g.replay()
    b.record(cur)
    torch.cuda.synchronize()
    us = a.elapsed_time(b) / reps * 1e3
    nb = w.algorithmic_bytes()
    total = n_layers * nb["attn"] + (c.vocab + c.batch * c.n_nodes) * 4096 * 2
    return {"layers": n_layers, "us": us, "launches": n_layers + 3, "status_max": int(st.status.max().item()),
            "accept_len": st.accept_len.cpu().tolist()[:8], "algorithmic_bytes": total,
            "gbs": total / us / 1e3}


def time_draft_head(rows, hidden, n_heads, vocab, dev):
    """clv_draft_head_step (Attention Decoder, output projector, norm + LM head, top-8) on `rows`
    rows with random weights: microseconds per step (8 launches, replayed from a CUDA graph) and the
    rate at which the step streams its weights (1.22 GB at hidden 4096 and vocabulary 128256: far
    larger than the L2, so every step reads them from HBM)."""
    import torch
    from paper_2408_00264_b200 import binding as clv
    from paper_2408_00264_b200 import workloads as W
    h, e, wts = W.make_draft_head(rows, hidden, n_heads, vocab, seed=W.BASE_SEED + 31)
    dw = {n: (v if n == "n_heads" else W.as_torch_bf16(v).to(dev)) for n, v in wts.items()}
    head = clv.make_draft_head(dw)
    ws = clv.new_draft_head_workspace(rows, hidden, vocab, dev)
    k = 8
    hid = torch.empty(rows, hidden, dtype=torch.bfloat16, device=dev)
    ids = torch.zeros(rows, k, dtype=torch.int32, device=dev)
    vals = torch.zeros(rows, k, dtype=torch.float32, device=dev)
    st = torch.zeros(5, dtype=torch.int32, device=dev)
    dh, de = W.as_torch_bf16(h).to(dev), W.as_torch_bf16(e).to(dev)
    call = lambda: clv.clv_draft_head_step(head, dh, de, k, hid, ids, vals, st, ws)  # noqa: E731
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        call()
    g.replay()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    torch.cuda.synchronize()
    reps = 20
    a.record(cur)
    for _ in range(reps):
        g.replay()
    b.record(cur)
    torch.cuda.synchronize()
    us = a.elapsed_time(b) / reps * 1e3
    wbytes = (3 * hidden * hidden + 2 * hidden * hidden + vocab * hidden) * 2
    bw_peak, bw_kind = measured_peaks()
    return {"rows": rows, "hidden": hidden, "n_heads": n_heads, "vocab": vocab, "k_top": k, "us": us,
            "launches": 8, "status": st.cpu().tolist(), "weight_bytes": wbytes, "gbs": wbytes / us / 1e3,
            "frac_of_hbm_peak": {"of_%s_%.0f_GBps" % (bw_kind, bw_peak): wbytes / us / 1e3 / bw_peak}}


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


def workload_config(w, input_sets=None):
    c = w.cfg
    policy = "not applicable"
    if input_sets is not None:
        policy = ("one step's inputs are larger than twice the L2" if input_sets == 1 else
                  "inputs rotate over %d distinct buffer sets (> 2x L2 in total) between steps" % input_sets)
    return {"workload": "%s: LLaMA3-8B-shaped verify step" % c.name if c.name == "C3" else c.name,
            "batch": c.batch, "n_q_heads": c.n_q_heads, "n_kv_heads": c.n_kv_heads,
            "head_dim": c.head_dim, "ctx_len": (int(w.ctx_len.min()), int(w.ctx_len.max())),
            "tree_nodes": c.n_nodes, "vocab": c.vocab, "paged": bool(c.paged),
            "cache_policy": policy}


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
# Which roof binds the attention of each workload (arithmetic intensity against the machine's
# ridge): few query rows per kv head leave it to the memory system, 256 rows (C3) sit on the ridge,
# 512 rows (C5) make it a dense contraction.  The argmax is a pure stream everywhere.
ATTN_BOUND = {"C1": "hbm", "C2": "hbm", "C3": "hbm", "C4": "hbm", "C5": "tensor"}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from ncu captures of the library whose
# clv_version() is the first element; a different library version reports null instead
NCU_TRAFFIC = {
    (111, "C1", "tree_attn"): 8.88e6, (111, "C2", "tree_attn"): 35.2e6, (111, "C3", "tree_attn"): 72.7e6,
    (111, "C4", "tree_attn"): 521.0e6, (111, "C5", "tree_attn"): 1089.0e6,
    (111, "C1", "accept_argmax"): 1.04e6, (111, "C2", "accept_argmax"): 4.11e6, (111, "C3", "accept_argmax"): 65.7e6,
    (111, "C4", "accept_argmax"): 263.0e6, (111, "C5", "accept_argmax"): 263.0e6,
}
MIN_TIMED_MS = 200.0   # the --steps loop is repeated until this much has been timed


def all_peaks():
    """(HBM GB/s, bf16 burst TFLOP/s, bf16 sustained TFLOP/s, 'measured' | 'fallback')."""
    try:
        d = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, 1590.0, 1400.0, "fallback"


def attention_flops(w):
    """4 B Hq N (L + N) D: Q K^T and P V over the context and the whole tree tile."""
    c = w.cfg
    return float(sum(4.0 * c.n_q_heads * c.n_nodes * (int(L) + c.n_nodes) * c.head_dim for L in w.ctx_len))


def measure_workload(name, args, dev, rank, dist, clocks_index, lib_version):
    """Step time and per-call times of one workload on this rank's GPU (inputs resident, CUDA-graph
    replay over rotating input sets, CUDA events on the launching stream)."""
    import dataclasses
    import torch
    from paper_2408_00264_b200 import workloads as W
    from paper_2408_00264_b200.step import VerifyStep

    cfg = dataclasses.replace(W.CONFIGS[name], seed=W.CONFIGS[name].seed + rank)
    w = W.generate(cfg)
    nbytes = w.algorithmic_bytes()
    # enough distinct input sets that their bytes exceed twice the L2, so that every step is cold
    # (C3: 4 x 138 MB; a workload larger than the L2 needs no second set)
    rotate = 1 if nbytes["total"] > 2 * L2_BYTES else max(1, min(ROTATE, int(4 * L2_BYTES // nbytes["total"]) + 1))
    sets = [VerifyStep(w, device=dev, with_lse=False) for _ in range(rotate)]
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    warm = max(args.warmup, 3)
    for i in range(warm):
        sets[i % rotate].run()
    torch.cuda.synchronize()
    graphs = None
    if not args.no_graph:
        graphs = []
        for st in sets:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                st.run()
            graphs.append(g)
        for i in range(warm):
            graphs[i % rotate].replay()
        stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps_ms = []
    barrier()
    with ClockSampler(clocks_index) as clocks:
        total = 0.0
        while True:   # exactly --steps steps per repeat; repeats until enough has been timed
            barrier()
            e0.record(stream)
            for i in range(args.steps):
                if graphs is not None:
                    graphs[i % rotate].replay()
                else:
                    sets[i % rotate].run()
            e1.record(stream)
            barrier()
            ms = e0.elapsed_time(e1)
            reps_ms.append(ms / args.steps)
            total += ms
            # every rank must take the same number of repeats: the slowest clock decides
            go = total < MIN_TIMED_MS and len(reps_ms) < 200
            if dist is not None:
                t = torch.tensor([1.0 if go else 0.0], device=dev)
                dist.all_reduce(t, op=dist.ReduceOp.MAX)
                go = bool(t.item() > 0)
            if not go:
                break
    step_ms = statistics.median(reps_ms)

    def time_call(call, n):
        """Microseconds per launch of one call, back to back over the rotating input sets, replayed
        from a CUDA graph so that host launch overhead does not set the pace of short kernels."""
        for i in range(3):
            getattr(sets[i % rotate], call)()
        torch.cuda.synchronize()
        if args.no_graph:
            run, per = (lambda: [getattr(sets[i], call)() for i in range(rotate)]), rotate
        else:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(rotate):
                    getattr(sets[i], call)()
            run, per = g.replay, rotate
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
    call_us = {k: time_call(k, n_k) for k in ("tree_attn", "accept_argmax", "accept_walk", "kv_commit",
                                              "accept_walk_commit")}

    hbm, tf_burst, tf_sust, kind = all_peaks()
    flops = attention_flops(w)
    attn_gbs = nbytes["attn"] / call_us["tree_attn"] / 1e3
    attn_tf = flops / call_us["tree_attn"] / 1e6
    arg_gbs = nbytes["logits"] / call_us["accept_argmax"] / 1e3
    dom = "tree_attn" if call_us["tree_attn"] >= call_us["accept_argmax"] else "accept_argmax"
    bound = ATTN_BOUND[name] if dom == "tree_attn" else "hbm"
    traffic = NCU_TRAFFIC.get((lib_version, name, dom))
    if bound == "tensor":
        # a kernel of most of a millisecond at the power cap: the sustained rate is its roof
        roof = {"kernel": dom, "bound": "tensor", "achieved": attn_tf, "peak": tf_sust,
                "peak_source": kind + " (sustained)", "unit": "TFLOP/s", "frac": attn_tf / tf_sust,
                "traffic": traffic}
    else:
        ach = attn_gbs if dom == "tree_attn" else arg_gbs
        roof = {"kernel": dom, "bound": "hbm", "achieved": ach, "peak": hbm, "peak_source": kind,
                "unit": "GB/s", "frac": ach / hbm, "traffic": traffic}
    res = {
        "workload": name, "step_us": step_ms * 1e3, "step_us_min": min(reps_ms) * 1e3,
        "repeats": len(reps_ms), "timed_ms": sum(reps_ms) * args.steps, "input_sets": rotate,
        "call_us": call_us, "algorithmic_bytes": nbytes, "attention_flops": flops,
        "step_gbs": nbytes["total"] / (step_ms * 1e-3) / 1e9,
        "roofline": roof,
        "attention": {"gbs": attn_gbs, "frac_of_hbm_%s" % kind: attn_gbs / hbm, "tflops": attn_tf,
                      "frac_of_bf16_burst_%s" % kind: attn_tf / tf_burst,
                      "frac_of_bf16_sustained_%s" % kind: attn_tf / tf_sust},
        "argmax": {"gbs": arg_gbs, "frac_of_hbm_%s" % kind: arg_gbs / hbm},
        "clocks": clocks.summary(),
    }
    return w, sets, res, reps_ms, graphs is not None


def run_clv(args):
    import torch
    from paper_2408_00264_b200 import binding as clv

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if local >= torch.cuda.device_count():
        raise SystemExit("bench.py: rank %d has no GPU (%d visible)" % (rank, torch.cuda.device_count()))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    L = clv.lib()
    version = int(L.clv_version())

    w, sets, main_res, reps_ms, graphed = measure_workload(args.workload, args, dev, rank, dist, local, version)
    nbytes = main_res["algorithmic_bytes"]
    step_ms = main_res["step_us"] * 1e-3
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

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
    sample_us = None
    model_us = None
    head_us = None
    if rank == 0 and not args.no_lm_head:
        lm_head = time_lm_head(B * N, 4096, c.vocab, dev, args)
        tree_us = time_token_tree(B, 128, dev)
        sample_us = time_accept_sample(w, dev)
        model_us = time_model_step(w, 32, dev) if args.workload in ("C1", "C2", "C3") else None
        head_us = time_draft_head(B, 4096, 32, c.vocab, dev)

    # ---- the other stated workloads, one after the other on rank 0's GPU (single-GPU runs) ------
    others = {}
    if world == 1 and args.all_workloads:
        del sets, s0, staging, host
        torch.cuda.empty_cache()
        for name in ("C1", "C2", "C3", "C4", "C5"):
            if name == args.workload:
                continue
            o_w, o_sets, o_res, _, _ = measure_workload(name, args, dev, rank, None, local, version)
            o_res["config"] = workload_config(o_w, o_res["input_sets"])
            others[name] = o_res
            del o_w, o_sets
            torch.cuda.empty_cache()

    # ---- max over ranks ------------------------------------------------------------------------
    step_ms, e2e_ms, job_bytes = reduce_over_ranks(dist, dev, step_ms, e2e_ms, float(nbytes["total"]))
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    hbm, tf_burst, tf_sust, peak_kind = all_peaks()
    value = job_bytes / (step_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, main_res["input_sets"]),
        "step_us": step_ms * 1e3, "step_us_min": main_res["step_us_min"], "repeats": main_res["repeats"],
        "timed_ms": main_res["timed_ms"],
        "timing": "--steps steps per repeat, repeats until %.0f ms are timed; ms_per_step is the median repeat "
                  "(max over ranks)" % MIN_TIMED_MS,
        "tree_tokens_per_s": world * B * N / (step_ms * 1e-3),
        "frac_of_hbm_peak": {"of_%s_%.0f_GBps" % (peak_kind, hbm): value / world / hbm,
                             "of_nominal_8000_GBps": value / world / NOMINAL_HBM_GBS},
        "call_us": main_res["call_us"], "launch_mode": "cuda-graph replay" if graphed else "per-call",
        "step_schedule": "clv_tree_attn, clv_accept_argmax, clv_accept_walk_commit (walk and commit in one launch) on one stream",
        "algorithmic_bytes": nbytes, "attention_flops": main_res["attention_flops"],
        "roofline": main_res["roofline"],
        "attention": main_res["attention"], "argmax": main_res["argmax"],
        "library_version": version,
        "e2e": {"value": job_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                "steps": n_e2e},
        "next_rows": {"lm_head_argmax": lm_head, "build_token_tree": tree_us, "accept_sample": sample_us, "model_step": model_us, "draft_head_step": head_us},
        "other_workloads": others,
        "gpu_launches": 3 * args.steps * main_res["repeats"],   # attention, argmax, walk + commit in one launch
        "clocks": main_res["clocks"],
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


# ----------------------------------------------------------------------------- ranks
def rank_env(rank, world, port):
    """The environment a launcher would give rank `rank` of `world` on this node."""
    return {"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
            "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)}


def _rank_entry(rank, world, port, argv):
    """One spawned rank: the launcher's environment, then the ordinary main."""
    os.environ.update(rank_env(rank, world, port))
    main(argv)


def free_port():
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def launch_ranks(world, argv, entry=_rank_entry):
    """`--gpus N` without a launcher: start N processes on this node, one per GPU."""
    import torch.multiprocessing as mp
    mp.spawn(entry, args=(world, free_port(), argv), nprocs=world, join=True)


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="C3", choices=["C1", "C2", "C3", "C4", "C5"])
    ap.add_argument("--impl", default="clv", choices=["clv", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch the calls of a step directly")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lm-head", action="store_true",
                    help="skip the timing of clv_lm_head_argmax (hidden 4096, the workload's rows and vocabulary)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer timing (profiling runs)")
    ap.add_argument("--no-other-workloads", dest="all_workloads", action="store_false",
                    help="time only --workload (by default a single-GPU run also times the other four)")
    ap.add_argument("--only", default=None, choices=["draft_head_step", "accept_sample"],
                    help="profiling aid: time just this call (C3's batch, hidden size and vocabulary), print its "
                         "figures and exit")
    args = ap.parse_args(argv)
    if args.only == "draft_head_step":
        import torch
        print(json.dumps({"draft_head_step": time_draft_head(4, 4096, 32, 128256, torch.device("cuda:0"))}))
        return
    if args.only == "accept_sample":
        import torch
        from paper_2408_00264_b200 import workloads as W
        w = W.generate(W.CONFIGS["C3"])
        print(json.dumps({"accept_sample": time_accept_sample(w, torch.device("cuda:0"))}))
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        if args.impl == "reference":   # the CPU arm runs on rank 0 alone
            run_reference(args)
            return
        launch_ranks(args.gpus, list(sys.argv[1:] if argv is None else argv))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_clv(args)


if __name__ == "__main__":
    main()
