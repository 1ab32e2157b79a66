"""Python access to the CPU checker (``clv_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the CPU-baseline
timing of the benchmark.  The GPU library never imports this package and this package never
imports the GPU library.

Every wrapper takes and returns numpy arrays; bf16 tensors are ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "clv_oracle.c")
_LIB = os.path.join(_HERE, "libclv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with gcc (plain -O2, OpenMP for the independent outer loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_f64_to_bf16.restype = ctypes.c_uint16
        _lib.orc_f64_to_bf16.argtypes = [ctypes.c_double]
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def threads() -> int:
    """Number of threads the OpenMP loops use."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


def f64_to_bf16_bits(x: float) -> int:
    return int(_load().orc_f64_to_bf16(float(x)))


def tree_attn(q, k_cache, v_cache, k_tree, v_tree, parent, ctx_len, scale, *,
              block_table=None, page_size=64, rows=None
              ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Tree attention by the definition (Sec. 2.1).

    q [B,N,Hq,D], k_tree/v_tree [B,N,Hkv,D], cache contiguous [B,cap,Hkv,D] or paged
    [P,page,Hkv,D] with block_table [B,max_pages].  ``rows``: optional int32 [R,3] of (b,i,h)
    to evaluate; default all.  Returns (out_f64 [R,D], out_bf16_bits [R,D], lse [R], status [B]);
    with rows=None the first three are reshaped to [B,N,Hq,...].
    """
    lib = _load()
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    k_tree = _c(k_tree, np.uint16); v_tree = _c(v_tree, np.uint16)
    parent = _c(parent, np.int32); ctx_len = _c(ctx_len, np.int32)
    B, N, Hq, D = q.shape
    Hkv = k_tree.shape[2]
    paged = block_table is not None
    if paged:
        block_table = _c(block_table, np.int32)
        cap, max_pages = 0, block_table.shape[1]
        page_size = k_cache.shape[1]
    else:
        cap, max_pages = k_cache.shape[1], 0
    if rows is None:
        R = B * N * Hq
        rows_arr = None
    else:
        rows_arr = _c(rows, np.int32).reshape(-1, 3)
        R = rows_arr.shape[0]
    out = np.empty((R, D), dtype=np.float64)
    out16 = np.empty((R, D), dtype=np.uint16)
    lse = np.empty(R, dtype=np.float64)
    status = np.zeros(B, dtype=np.int32)
    lib.orc_tree_attn(ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(Hq), ctypes.c_int(Hkv),
                      ctypes.c_int(D), _p(q), _p(k_cache), _p(v_cache), ctypes.c_int(int(paged)),
                      ctypes.c_int(cap), ctypes.c_int(page_size), ctypes.c_int(max_pages),
                      _p(block_table), _p(k_tree), _p(v_tree), _p(parent), _p(ctx_len),
                      ctypes.c_double(float(scale)), ctypes.c_int64(R), _p(rows_arr), _p(out),
                      _p(out16), _p(lse), _p(status))
    if rows is None:
        return (out.reshape(B, N, Hq, D), out16.reshape(B, N, Hq, D), lse.reshape(B, N, Hq),
                status)
    return out, out16, lse, status


def argmax(logits: np.ndarray, vocab: int) -> np.ndarray:
    """First strict maximum of each row; logits [..., ld] bf16 bits, the first ``vocab`` columns
    of a row are scanned (Sec. 4.2: temperature 0 = greedy target decoding)."""
    lib = _load()
    lg = _c(logits, np.uint16)
    ld = lg.shape[-1]
    lead = lg.shape[:-1]
    R = int(np.prod(lead)) if lead else 1
    ids = np.empty(R, dtype=np.int32)
    lib.orc_argmax(ctypes.c_int64(R), ctypes.c_int(vocab), ctypes.c_int64(ld), _p(lg), _p(ids))
    return ids.reshape(lead)


def lm_head_argmax(hidden: np.ndarray, weight: np.ndarray, rows=None, want_logits: bool = False):
    """Greedy choice from the LM head (Sec. 3.1 + Sec. 4.2): hidden [M, K] and weight [V, K] bf16
    bits; logits in float64, rounded to bf16, first strict maximum.  Returns ids [n] (and the
    unrounded float64 logits [n, V] if asked) for the selected rows (all if ``rows`` is None)."""
    lib = _load()
    h = _c(hidden, np.uint16)
    w = _c(weight, np.uint16)
    M, K = h.shape
    V = w.shape[0]
    assert w.shape[1] == K
    sel = None if rows is None else _c(np.asarray(rows), np.int32)
    n = M if sel is None else len(sel)
    ids = np.empty(n, dtype=np.int32)
    z = np.empty((n, V), dtype=np.float64) if want_logits else None
    rc = lib.orc_lm_head_argmax(ctypes.c_int(n), _p(sel), ctypes.c_int(K), ctypes.c_int(V),
                                ctypes.c_int64(K), ctypes.c_int64(K), _p(h), _p(w), _p(z), _p(ids))
    assert rc == 0
    return (ids, z) if want_logits else ids


def build_token_tree(root_token, cand, cand_len, node_cap: int):
    """Token tree by prefix matching (Sec. 2.1, caption of Fig. 2), written as the definition: the
    nodes are the distinct non-empty prefixes of the candidate sequences, node 0 is the root; they
    are numbered by depth and then by the first candidate that contains the prefix.  Plain Python
    over a dictionary of prefixes (the sizes are tiny).  Returns tokens, parent [B, node_cap],
    n_nodes [B], node_of [B, C, D], status [B]; padding slots are children of the root with token
    -1; a tree that does not fit, or a length outside [0, D], gives status 7 and the bare root."""
    cand = np.asarray(cand)
    B, C, D = cand.shape
    tokens = np.full((B, node_cap), -1, dtype=np.int32)
    parent = np.zeros((B, node_cap), dtype=np.int32)
    n_nodes = np.ones(B, dtype=np.int32)
    node_of = np.full((B, C, D), -1, dtype=np.int32)
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        tokens[b, 0] = root_token[b]
        parent[b, 0] = -1
        lens = [int(x) for x in cand_len[b]]
        if any(l < 0 or l > D for l in lens):
            status[b] = 7
            continue
        first = {}                      # prefix (tuple of tokens) -> first candidate holding it
        for c in range(C):
            for d in range(lens[c]):
                first.setdefault(tuple(int(t) for t in cand[b, c, :d + 1]), c)
        order = sorted(first, key=lambda pre: (len(pre), first[pre]))
        if 1 + len(order) > node_cap:
            status[b] = 7
            continue
        index = {pre: 1 + i for i, pre in enumerate(order)}
        for pre, i in index.items():
            tokens[b, i] = pre[-1]
            parent[b, i] = index[pre[:-1]] if len(pre) > 1 else 0
        n_nodes[b] = 1 + len(order)
        for c in range(C):
            for d in range(lens[c]):
                node_of[b, c, d] = index[tuple(int(t) for t in cand[b, c, :d + 1])]
    return tokens, parent, n_nodes, node_of, status


def tree_to_intervals(parent):
    """Compressed (linear) form of the tree mask (App. A.1: "a numerical comparison" instead of an
    N x N matrix; the figure is missing, the encoding taken is depth-first entry/exit labels): tin
    = position of the node in a depth-first walk that visits children in increasing node index
    (several roots: one after the other), tout = tin + size of the node's subtree.  Then j is an
    ancestor of i, or i itself, exactly if tin[j] <= tin[i] < tout[j].  Written as a recursive
    walk.  Returns tin, tout [B, N], status [B] (7 for a malformed parent[], labels -1)."""
    parent = np.asarray(parent, dtype=np.int32)
    B, N = parent.shape
    tin = np.full((B, N), -1, np.int32)
    tout = np.full((B, N), -1, np.int32)
    status = np.zeros(B, np.int32)
    for b in range(B):
        par = parent[b]
        if any(par[i] < -1 or par[i] >= i for i in range(N)):
            status[b] = 7
            continue
        kids = [[] for _ in range(N)]
        roots = []
        for i in range(N):
            (roots if par[i] < 0 else kids[par[i]]).append(i)
        clock = [0]

        def visit(v):
            tin[b, v] = clock[0]
            clock[0] += 1
            for c in kids[v]:
                visit(c)
            tout[b, v] = clock[0]
        for r in roots:
            visit(r)
    return tin, tout, status


def tree_from_intervals(tin, tout):
    """parent[] from depth-first labels: the parent of i is the node j != i whose interval
    [tin[j], tout[j]) contains tin[i] and is the narrowest such interval; -1 if there is none.
    Status 7 (parent all -1) if the labels are not those of a forest in topological node order:
    an empty interval, two nodes with the same tin, intervals that overlap without nesting, or a
    parent that does not come before its child."""
    tin = np.asarray(tin, dtype=np.int64)
    tout = np.asarray(tout, dtype=np.int64)
    B, N = tin.shape
    parent = np.full((B, N), -1, np.int32)
    status = np.zeros(B, np.int32)
    for b in range(B):
        ok = all(tout[b, i] > tin[b, i] for i in range(N)) and len(set(tin[b].tolist())) == N
        for i in range(N):
            for j in range(N):
                if not ok or i == j:
                    continue
                a0, a1, b0, b1 = tin[b, i], tout[b, i], tin[b, j], tout[b, j]
                if a0 < b0 < a1 < b1:          # overlap without nesting
                    ok = False
        if ok:
            for i in range(N):
                best = -1
                for j in range(N):
                    if j != i and tin[b, j] <= tin[b, i] < tout[b, j]:
                        if best < 0 or tout[b, j] - tin[b, j] < tout[b, best] - tin[b, best]:
                            best = j
                if best >= i:
                    ok = False
                parent[b, i] = best
        if not ok:
            parent[b] = -1
            status[b] = 7
    return parent, status


def draft_head_step(h, e, wts, k_top: int, eps: float = 1e-5):
    """One step of a Clover-2 draft head for every row (Sec. 3.1; App. A.3 prints the Attention
    Decoder), in float64 numpy, written as the definition.  h: [R, H] hidden states (of the target,
    or of the previous head), e: [R, H] embeddings of the previously emitted tokens; both uint16
    bf16 bits, like every weight in ``wts`` (a dict):
      norm1 [H], wq, wk, wv [H, H], bq, bk, bv [H], n_heads (int), wfc [H, 2H], bfc [H], norm2 [H],
      lm_head [V, H].
    Attention Decoder:  x = RMSNorm(h; norm1);  q = x wq^T + bq;  k = e wk^T + bk;  v = e wv^T + bv;
    per head j (H / n_heads consecutive features): gate_j = <q_j, k_j> / max(|q_j| |k_j|, 1e-8);
    a = h + v * gate (the gate broadcast over its head's features; no activation).
    Output projector: p = [a, e] wfc^T + bfc (a fully connected layer over the decoder's output and
    the token embedding).  Logits = RMSNorm(p; norm2) lm_head^T; the head's proposals are the k_top
    largest logits of each row, highest first, lower index first among equals.
    Returns (p float64 [R, H], top ids int32 [R, k_top], top logits float64 [R, k_top], logits [R, V])."""
    f = lambda a: _bits_to_f64(np.asarray(a))  # noqa: E731
    h64, e64 = f(h), f(e)
    R, H = h64.shape
    nh = int(wts["n_heads"])
    hd = H // nh

    def rms(x, g):
        return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * f(g)
    x = rms(h64, wts["norm1"])
    q = x @ f(wts["wq"]).T + f(wts["bq"])
    k = e64 @ f(wts["wk"]).T + f(wts["bk"])
    v = e64 @ f(wts["wv"]).T + f(wts["bv"])
    a = np.empty_like(h64)
    for r in range(R):
        for j in range(nh):
            sl = slice(j * hd, (j + 1) * hd)
            den = max(np.sqrt((q[r, sl] ** 2).sum()) * np.sqrt((k[r, sl] ** 2).sum()), 1e-8)
            gate = float(q[r, sl] @ k[r, sl]) / den
            a[r, sl] = h64[r, sl] + v[r, sl] * gate
    p = np.concatenate([a, e64], axis=1) @ f(wts["wfc"]).T + f(wts["bfc"])
    logits = rms(p, wts["norm2"]) @ f(wts["lm_head"]).T
    V = logits.shape[1]
    ids = np.empty((R, k_top), np.int32)
    vals = np.empty((R, k_top), np.float64)
    for r in range(R):
        order = sorted(range(V), key=lambda t: (-logits[r, t], t))[:k_top]
        ids[r] = order
        vals[r] = logits[r, order]
    return p, ids, vals, logits


def _bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def accept_walk(parent, tokens, ids, path_cap: int):
    """Greedy acceptance walk; returns (accept_len [B], accept_idx [B,path_cap], next_token [B],
    status [B])."""
    lib = _load()
    parent = _c(parent, np.int32); tokens = _c(tokens, np.int32); ids = _c(ids, np.int32)
    B, N = parent.shape
    alen = np.empty(B, dtype=np.int32)
    aidx = np.empty((B, path_cap), dtype=np.int32)
    nxt = np.empty(B, dtype=np.int32)
    status = np.empty(B, dtype=np.int32)
    lib.orc_accept_walk(ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(path_cap), _p(parent),
                        _p(tokens), _p(ids), _p(alen), _p(aidx), _p(nxt), _p(status))
    return alen, aidx, nxt, status


def accept_sample(logits, vocab: int, parent, tokens, uniforms, temperature: float, path_cap: int):
    """Stochastic acceptance (temperature > 0).  logits: uint16 bf16 bits [B, N, ld]; uniforms:
    float32 [B, N + 1].  Returns (accept_len [B], accept_idx [B,path_cap], next_token [B],
    status [B], margin [B, 2]): margin[:, 0] is the smallest distance between a uniform and the
    probability it was compared with over the accept tests of the sequence, margin[:, 1] the distance
    of the final draw's target to the nearer running sum around it (as a fraction of the mass left)."""
    lib = _load()
    lg = _c(logits, np.uint16)
    parent = _c(parent, np.int32); tokens = _c(tokens, np.int32)
    uniforms = _c(uniforms, np.float32)
    B, N = parent.shape
    assert lg.shape[0] == B and lg.shape[1] == N and uniforms.shape == (B, N + 1)
    ld = lg.shape[-1]
    alen = np.empty(B, dtype=np.int32)
    aidx = np.empty((B, path_cap), dtype=np.int32)
    nxt = np.empty(B, dtype=np.int32)
    status = np.empty(B, dtype=np.int32)
    margin = np.empty((B, 2), dtype=np.float64)
    rc = lib.orc_accept_sample(ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(vocab), ctypes.c_int64(ld),
                               ctypes.c_int(path_cap), _p(lg), _p(parent), _p(tokens), _p(uniforms),
                               ctypes.c_double(float(temperature)), _p(alen), _p(aidx), _p(nxt), _p(status),
                               _p(margin))
    assert rc == 0
    return alen, aidx, nxt, status, margin


def kv_commit(k_cache, v_cache, k_tree, v_tree, accept_idx, accept_len, ctx_len, *,
              block_table=None):
    """Returns (k_cache', v_cache', ctx_len_out, status); the inputs are not modified."""
    lib = _load()
    kc = np.array(k_cache, dtype=np.uint16, order="C", copy=True)
    vc = np.array(v_cache, dtype=np.uint16, order="C", copy=True)
    k_tree = _c(k_tree, np.uint16); v_tree = _c(v_tree, np.uint16)
    accept_idx = _c(accept_idx, np.int32); accept_len = _c(accept_len, np.int32)
    ctx_len = _c(ctx_len, np.int32)
    B, N, Hkv, D = k_tree.shape
    path_cap = accept_idx.shape[1]
    paged = block_table is not None
    if paged:
        block_table = _c(block_table, np.int32)
        cap, max_pages, n_pages, page = 0, block_table.shape[1], kc.shape[0], kc.shape[1]
    else:
        cap, max_pages, n_pages, page = kc.shape[1], 0, 0, 64
    out_len = np.empty(B, dtype=np.int32)
    status = np.empty(B, dtype=np.int32)
    lib.orc_kv_commit(ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(Hkv), ctypes.c_int(D),
                      ctypes.c_int(path_cap), _p(kc), _p(vc), ctypes.c_int(int(paged)),
                      ctypes.c_int(cap), ctypes.c_int(page), ctypes.c_int(n_pages),
                      ctypes.c_int(max_pages), _p(block_table), _p(k_tree), _p(v_tree),
                      _p(accept_idx), _p(accept_len), _p(ctx_len), _p(out_len), _p(status))
    return kc, vc, out_len, status
