"""Seeded synthetic inputs for the tree-verification step.

This module only *creates inputs*: draft trees, draft tokens, bf16 Q/K/V, target logits with
a planted winner, context lengths and KV-cache layouts.  It contains none of the verification
arithmetic (no attention, no argmax over the vocabulary as an output, no acceptance walk, no cache
update) and imports neither the CUDA binding nor the CPU checker, so both sides of a parity test
can be fed from it.

All tensors that are bf16 on the device are held here as ``numpy.uint16`` bit patterns; use
:func:`bf16_bits_to_f64` for an exact widening and :func:`as_torch_bf16` for a zero-copy torch
view.

The stand-in workloads follow the model shapes the paper evaluates (Vicuna-7B v1.5: 32 MHA heads;
LLaMA3-Instruct-8B: 32 query / 8 KV heads; Sec. 4.1 "Models and baselines"), with draft trees of
the kind Sec. 2.1 describes (speculations merged by prefix into a token tree).  The paper's
evaluation prompts and trained draft heads are not used: tokens and logits are random, and the
probability that the target agrees with a drafted child is a parameter.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple, Union

import numpy as np
import torch

BASE_SEED = 240800264
PAGE_SIZE = 64
HEAD_DIM = 128


# --------------------------------------------------------------------------------------
# bf16 helpers (bit-level; no arithmetic of the method)
# --------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even) and return the uint16 bit patterns."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return bf16_bits_to_f32(bits).astype(np.float64)


def as_torch_bf16(bits: np.ndarray) -> torch.Tensor:
    """Zero-copy torch.bfloat16 view of a uint16 bit-pattern array (CPU)."""
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)


def _bf16_round_up_bits(x: np.ndarray) -> np.ndarray:
    """Smallest bf16 >= x for finite positive float32 x, as uint16 bits."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    hi = b >> np.uint32(16)
    hi = hi + ((b & np.uint32(0xFFFF)) != 0).astype(np.uint32)
    return hi.astype(np.uint16)


def _normal_bf16(shape: Sequence[int], seed: int) -> np.ndarray:
    """N(0,1) float32 samples rounded to bf16 bits, generated in bounded-size pieces."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) % (2**63 - 1))
    n = int(np.prod(shape)) if len(shape) else 1
    out = torch.empty(n, dtype=torch.bfloat16)
    step = 1 << 26
    for s in range(0, n, step):
        e = min(n, s + step)
        out[s:e] = torch.randn(e - s, generator=g, dtype=torch.float32).to(torch.bfloat16)
    return out.view(torch.int16).numpy().view(np.uint16).reshape(tuple(shape))


# --------------------------------------------------------------------------------------
# Draft trees (parent-index arrays, topological order: parent[i] < i, parent[0] = -1)
# --------------------------------------------------------------------------------------
def tree_depths(parent: np.ndarray) -> np.ndarray:
    d = np.zeros(len(parent), dtype=np.int64)
    for i in range(len(parent)):
        d[i] = 0 if parent[i] < 0 else d[parent[i]] + 1
    return d


def tree_chain(n: int) -> np.ndarray:
    return np.arange(-1, n - 1, dtype=np.int32)


def tree_star(n: int) -> np.ndarray:
    p = np.zeros(n, dtype=np.int32)
    p[0] = -1
    return p


def tree_forest(n: int) -> np.ndarray:
    return np.full(n, -1, dtype=np.int32)


def tree_random(n: int, max_depth: int, rng: np.random.Generator) -> np.ndarray:
    """parent[i] uniform over the earlier nodes whose depth is below ``max_depth``."""
    parent = np.full(n, -1, dtype=np.int32)
    depth = np.zeros(n, dtype=np.int64)
    for i in range(1, n):
        cand = np.flatnonzero(depth[:i] < max_depth)
        p = int(cand[rng.integers(0, len(cand))])
        parent[i] = p
        depth[i] = depth[p] + 1
    return parent


def tree_topn(branching: Sequence[int], n: int, order: str = "score") -> np.ndarray:
    """Static draft tree: the root plus the n-1 best nodes of the full tree whose depth-d nodes
    have ``branching[d-1]`` ranked children.

    A node's score is the product over its root path of 1/(rank+1) (rank 0 = the draft head's
    top-1 guess), which imitates choosing the n nodes with the highest expected acceptance.
    Ties are broken by smaller depth, then by breadth-first position in the full tree.
    ``order='bfs'`` keeps the first n nodes in breadth-first order instead.
    The kept nodes are renumbered breadth-first.
    """
    # enumerate the full tree level by level; node = (den, depth, bfs_index, parent_full, path)
    nodes: List[Tuple[int, int, int, int]] = [(1, 0, 0, -1)]
    level = [0]
    for d, br in enumerate(branching, start=1):
        nxt = []
        for pidx in level:
            pden = nodes[pidx][0]
            for r in range(br):
                nodes.append((pden * (r + 1), d, len(nodes), pidx))
                nxt.append(len(nodes) - 1)
        level = nxt
    if n > len(nodes):
        raise ValueError("tree_topn: n exceeds the full tree")
    if order == "bfs":
        keep = list(range(n))
    else:
        rest = sorted(nodes[1:], key=lambda t: (t[0], t[1], t[2]))[: n - 1]
        keep = sorted([0] + [t[2] for t in rest])  # bfs index order == (depth, rank path)
    new_id = {full: i for i, full in enumerate(keep)}
    parent = np.full(n, -1, dtype=np.int32)
    for full, i in new_id.items():
        pf = nodes[full][3]
        parent[i] = -1 if pf < 0 else new_id[pf]
    return parent


# --------------------------------------------------------------------------------------
# Workload description
# --------------------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class VerifyConfig:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    ctx: Union[int, Tuple[int, int]]          # fixed L, or (lo, hi) inclusive for ragged
    n_nodes: int
    max_depth: int
    vocab: int
    branching: Optional[Tuple[int, ...]] = None   # None -> random parent[] per sequence
    paged: bool = False
    p_accept: Union[float, Tuple[float, float]] = 0.6
    seed: int = BASE_SEED
    head_dim: int = HEAD_DIM
    margin: float = 0.5

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


CONFIGS: Dict[str, VerifyConfig] = {
    "C1": VerifyConfig("C1", 1, 32, 32, 512, 16, 4, 32000, (4, 2, 1, 1), seed=BASE_SEED + 1000),
    "C2": VerifyConfig("C2", 1, 32, 32, 2048, 64, 6, 32000, (8, 4, 2, 2, 1, 1), seed=BASE_SEED + 2000),
    "C3": VerifyConfig("C3", 4, 32, 8, 4096, 64, 6, 128256, None, seed=BASE_SEED + 3000),
    "C4": VerifyConfig("C4", 32, 32, 8, (512, 8192), 32, 5, 128256, None, paged=True,
                       p_accept=(0.3, 0.8), seed=BASE_SEED + 4000),
    "C5": VerifyConfig("C5", 8, 32, 8, 32768, 128, 8, 128256, (10, 4, 2, 2, 1, 1, 1, 1),
                       seed=BASE_SEED + 5000),
}


@dataclasses.dataclass
class Workload:
    cfg: VerifyConfig
    scale: float
    ctx_len: np.ndarray            # int32 [B]
    parent: np.ndarray             # int32 [B,N]
    tokens: np.ndarray             # int32 [B,N]
    winner: np.ndarray             # int32 [B,N]  planted argmax (generator bookkeeping)
    q: np.ndarray                  # bf16 bits [B,N,Hq,D]
    k_tree: np.ndarray             # bf16 bits [B,N,Hkv,D]
    v_tree: np.ndarray
    k_cache: np.ndarray            # contiguous [B,cap,Hkv,D] or paged [P,64,Hkv,D]
    v_cache: np.ndarray
    logits: np.ndarray             # bf16 bits [B,N,ld]  (ld >= vocab)
    cap_tokens: int                # contiguous row capacity per sequence (0 if paged)
    block_table: Optional[np.ndarray]   # int32 [B,max_pages] or None
    n_pages: int
    max_pages_per_seq: int
    path_cap: int

    def algorithmic_bytes(self) -> Dict[str, int]:
        """Bytes the step must move at least once (each cached K/V row once per step, tree K/V,
        Q, O, logits once, ids and path arrays, accepted rows read and written by the commit)."""
        c = self.cfg
        row = c.n_kv_heads * c.head_dim * 2
        kv = int(self.ctx_len.astype(np.int64).sum()) * row * 2
        tree = c.batch * c.n_nodes * row * 2
        qo = c.batch * c.n_nodes * c.n_q_heads * c.head_dim * 2 * 2
        lg = c.batch * c.n_nodes * c.vocab * 2
        return {"kv": kv, "tree_kv": tree, "q_o": qo, "logits": lg,
                "attn": kv + tree + qo, "total": kv + tree + qo + lg}

    def attn_flops(self) -> int:
        c = self.cfg
        tot = 0
        for b in range(c.batch):
            tot += 4 * c.n_q_heads * c.n_nodes * (int(self.ctx_len[b]) + c.n_nodes) * c.head_dim
        return tot


def _draw_tokens(parent: np.ndarray, vocab: int, rng: np.random.Generator) -> np.ndarray:
    """Uniform draft tokens; the children of one node carry distinct tokens (prefix merging
    makes equal siblings impossible, Sec. 2.1 / Fig. 2 caption)."""
    n = len(parent)
    tok = rng.integers(0, vocab, size=n, dtype=np.int64)
    for p in range(-1, n):
        kids = np.flatnonzero(parent == p)
        if len(kids) > vocab:
            raise ValueError("a node has more children than there are distinct tokens")
        seen = set()
        for c in kids:
            while int(tok[c]) in seen:
                tok[c] = rng.integers(0, vocab)
            seen.add(int(tok[c]))
    return tok.astype(np.int32)


def _plant_winners(parent: np.ndarray, tokens: np.ndarray, vocab: int, p: float,
                   rng: np.random.Generator) -> np.ndarray:
    n = len(parent)
    win = np.zeros(n, dtype=np.int32)
    for i in range(n):
        kids = np.flatnonzero(parent == i)
        if len(kids) and rng.random() < p:
            win[i] = tokens[kids[rng.integers(0, len(kids))]]
        else:
            kid_tok = set(int(t) for t in tokens[kids])
            if len(kid_tok) >= vocab:
                raise ValueError("no token left that is not a child's token")
            w = int(rng.integers(0, vocab))
            while w in kid_tok:
                w = int(rng.integers(0, vocab))
            win[i] = w
    return win


def make_logits(rows: int, vocab: int, ld: int, winner: np.ndarray, margin: float,
                seed: int) -> np.ndarray:
    """N(0,1) float32 logits rounded to bf16, then per row the entry at ``winner`` raised to the
    smallest bf16 that is at least ``margin`` above every other entry of the row."""
    lg = _normal_bf16((rows, ld), seed)
    vals = bf16_bits_to_f32(lg[:, :vocab])
    r = np.arange(rows)
    vals[r, winner] = -np.inf
    top = vals.max(axis=1)
    del vals
    lg[r, winner] = _bf16_round_up_bits(top + np.float32(margin))
    return lg


def make_candidates(batch: int, n_cand: int, max_len: int, vocab: int, seed: int, p_follow: float = 0.6):
    """Speculated sequences with shared prefixes, as a draft model's top-k expansion produces them:
    every candidate copies a random earlier candidate of the same sequence up to a random depth
    (with probability ``p_follow``) and continues with uniform tokens below ``vocab``; lengths are
    uniform in [0, max_len].  Returns root_token [B], cand [B, n_cand, max_len] (unused positions
    hold -1) and cand_len [B, n_cand], all int32."""
    rng = np.random.default_rng(np.random.SeedSequence(seed))
    cand = np.full((batch, n_cand, max_len), -1, dtype=np.int32)
    lens = rng.integers(0, max_len + 1, size=(batch, n_cand)).astype(np.int32)
    for b in range(batch):
        for c in range(n_cand):
            n = int(lens[b, c])
            seq = rng.integers(0, vocab, size=n)
            if c > 0 and rng.random() < p_follow:
                o = int(rng.integers(0, c))
                k = int(rng.integers(0, min(n, int(lens[b, o])) + 1))
                seq[:k] = cand[b, o, :k]
            cand[b, c, :n] = seq
    root = rng.integers(0, vocab, size=batch).astype(np.int32)
    return root, cand, lens


def make_uniforms(batch: int, n_nodes: int, seed: int) -> np.ndarray:
    """Uniform numbers in [0, 1) for the stochastic acceptance: float32 [batch, n_nodes + 1] (entry
    c decides drafted node c, the last one draws the next token).  Multiples of 2^-24, so that the
    float32 value is exactly what a float64 reader sees."""
    rng = np.random.default_rng(seed)
    return (rng.integers(0, 1 << 24, size=(batch, n_nodes + 1)).astype(np.float64) / float(1 << 24)).astype(np.float32)


def make_lm_head(rows: int, hidden_dim: int, vocab: int, seed: int, planted: float = 12.0):
    """Inputs of the LM head for ``rows`` tree nodes: hidden states N(0,1) and a weight matrix
    N(0, 1/hidden_dim) (so that logits are about N(0,1)), both rounded to bf16 and returned as bit
    patterns [rows, hidden_dim] and [vocab, hidden_dim].  With ``planted`` > 0 every hidden row
    gets ``planted`` times the weight row of a drawn vocabulary entry added before rounding, which
    lifts that entry's logit about ``planted`` above the rest: ``winner`` [rows] holds the entries
    (a clear argmax); with ``planted`` = 0 the argmax is whatever the draw gives and ``winner`` is
    None.  Generated in slabs so that a 128256 x 4096 matrix needs no float64 copy."""
    ss = np.random.SeedSequence(seed).spawn(3)
    rng_w = np.random.default_rng(ss[0])
    weight = np.empty((vocab, hidden_dim), dtype=np.uint16)
    inv = np.float32(1.0 / np.sqrt(hidden_dim))
    slab = max(1, (1 << 24) // hidden_dim)
    for v0 in range(0, vocab, slab):
        v1 = min(vocab, v0 + slab)
        weight[v0:v1] = f32_to_bf16_bits(rng_w.standard_normal((v1 - v0, hidden_dim), dtype=np.float32) * inv)
    hid = np.random.default_rng(ss[1]).standard_normal((rows, hidden_dim), dtype=np.float32)
    winner = None
    if planted > 0:
        winner = np.random.default_rng(ss[2]).integers(0, vocab, size=rows).astype(np.int32)
        hid += np.float32(planted) * bf16_bits_to_f32(weight[winner])
    return f32_to_bf16_bits(hid), weight, winner


def generate(cfg: VerifyConfig, ld_pad: int = 0, extra_cap: int = 0,
             tree_order: str = "score") -> Workload:
    """Create every input of one verify step for ``cfg`` (deterministic in ``cfg.seed``).

    ``ld_pad`` adds unused columns to each logits row (row stride ld = vocab rounded up to 8,
    plus ld_pad); ``extra_cap`` adds spare rows to a contiguous cache.
    """
    B, N, Hq, Hkv, D = cfg.batch, cfg.n_nodes, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    if Hq % Hkv:
        raise ValueError("n_q_heads must be a multiple of n_kv_heads")
    root = np.random.SeedSequence(cfg.seed)
    ss = root.spawn(4 + B)
    rng_len = np.random.default_rng(ss[0])
    rng_tab = np.random.default_rng(ss[1])
    rng_p = np.random.default_rng(ss[2])

    if isinstance(cfg.ctx, tuple):
        ctx_len = rng_len.integers(cfg.ctx[0], cfg.ctx[1] + 1, size=B).astype(np.int32)
    else:
        ctx_len = np.full(B, cfg.ctx, dtype=np.int32)

    parent = np.zeros((B, N), dtype=np.int32)
    tokens = np.zeros((B, N), dtype=np.int32)
    winner = np.zeros((B, N), dtype=np.int32)
    for b in range(B):
        rng_b = np.random.default_rng(ss[4 + b])
        if cfg.branching is not None:
            parent[b] = tree_topn(cfg.branching, N, order=tree_order)
        else:
            parent[b] = tree_random(N, cfg.max_depth, rng_b)
        tokens[b] = _draw_tokens(parent[b], cfg.vocab, rng_b)
        if isinstance(cfg.p_accept, tuple):
            p = float(rng_p.uniform(cfg.p_accept[0], cfg.p_accept[1]))
        else:
            p = float(cfg.p_accept)
        winner[b] = _plant_winners(parent[b], tokens[b], cfg.vocab, p, rng_b)
    path_cap = int(max(tree_depths(parent[b]).max() for b in range(B))) + 1

    s0 = cfg.seed * 7919
    q = _normal_bf16((B, N, Hq, D), s0 + 1)
    k_tree = _normal_bf16((B, N, Hkv, D), s0 + 2)
    v_tree = _normal_bf16((B, N, Hkv, D), s0 + 3)

    if cfg.paged:
        pages_per_seq = [(int(ctx_len[b]) + N + PAGE_SIZE - 1) // PAGE_SIZE for b in range(B)]
        used = sum(pages_per_seq)
        n_pages = used + (used + 7) // 8
        max_pages = max(pages_per_seq)
        perm = rng_tab.permutation(n_pages).astype(np.int32)
        block_table = np.full((B, max_pages), -1, dtype=np.int32)
        o = 0
        for b in range(B):
            block_table[b, : pages_per_seq[b]] = perm[o: o + pages_per_seq[b]]
            o += pages_per_seq[b]
        k_cache = _normal_bf16((n_pages, PAGE_SIZE, Hkv, D), s0 + 4)
        v_cache = _normal_bf16((n_pages, PAGE_SIZE, Hkv, D), s0 + 5)
        cap = 0
    else:
        cap = int(ctx_len.max()) + N + extra_cap
        k_cache = _normal_bf16((B, cap, Hkv, D), s0 + 4)
        v_cache = _normal_bf16((B, cap, Hkv, D), s0 + 5)
        block_table, n_pages, max_pages = None, 0, 0

    ld = (cfg.vocab + 7) // 8 * 8 + ld_pad
    logits = make_logits(B * N, cfg.vocab, ld, winner.reshape(-1), cfg.margin, s0 + 6)
    logits = logits.reshape(B, N, ld)

    return Workload(cfg=cfg, scale=1.0 / math.sqrt(D), ctx_len=ctx_len, parent=parent,
                    tokens=tokens, winner=winner, q=q, k_tree=k_tree, v_tree=v_tree,
                    k_cache=k_cache, v_cache=v_cache, logits=logits, cap_tokens=cap,
                    block_table=block_table, n_pages=n_pages, max_pages_per_seq=max_pages,
                    path_cap=path_cap)


def layer_tensors(w: Workload, n_layers: int):
    """Per-layer Q, tree K/V and cache K/V for a whole-model verify step on the trees, contexts and
    (paged) block table of ``w``: layer 0 is ``w`` itself, every further layer draws fresh N(0,1)
    tensors of the same shapes.  Returns uint16 arrays with a leading layer axis."""
    s0 = w.cfg.seed * 7919
    out = []
    for name, off in (("q", 1), ("k_tree", 2), ("v_tree", 3), ("k_cache", 4), ("v_cache", 5)):
        base = getattr(w, name)
        layers = [base] + [_normal_bf16(base.shape, s0 + 1000 * l + off) for l in range(1, n_layers)]
        out.append(np.stack(layers))
    return tuple(out)


def make_draft_head(rows: int, hidden_dim: int, n_heads: int, vocab: int, seed: int):
    """Random inputs and weights of one Clover-2 draft-head step (trained heads are not available):
    hidden states and token embeddings N(0,1), projection weights N(0, 1/fan_in), small biases,
    norm gains around 1, all rounded to bf16.  Returns (h, e, weights dict) as uint16 bit patterns."""
    s = seed * 7919
    H = hidden_dim

    def scaled(shape, k, factor):
        x = bf16_bits_to_f32(_normal_bf16(shape, s + k)) * np.float32(factor)
        return f32_to_bf16_bits(x)
    inv = 1.0 / math.sqrt(H)
    wts = {"n_heads": n_heads,
           "norm1": f32_to_bf16_bits(1.0 + 0.1 * bf16_bits_to_f32(_normal_bf16((H,), s + 10))),
           "norm2": f32_to_bf16_bits(1.0 + 0.1 * bf16_bits_to_f32(_normal_bf16((H,), s + 11))),
           "wq": scaled((H, H), 12, inv), "wk": scaled((H, H), 13, inv), "wv": scaled((H, H), 14, inv),
           "bq": scaled((H,), 15, 0.1), "bk": scaled((H,), 16, 0.1), "bv": scaled((H,), 17, 0.1),
           "wfc": scaled((H, 2 * H), 18, 1.0 / math.sqrt(2 * H)), "bfc": scaled((H,), 19, 0.1),
           "lm_head": scaled((vocab, H), 20, inv)}
    return _normal_bf16((rows, H), s + 1), _normal_bf16((rows, H), s + 2), wts


def small_config(name: str = "small", **kw) -> VerifyConfig:
    """A reduced configuration for tests; keyword arguments override the defaults."""
    base = dict(name=name, batch=2, n_q_heads=8, n_kv_heads=2, ctx=200, n_nodes=24, max_depth=5,
                vocab=1000, branching=None, paged=False, p_accept=0.6, seed=BASE_SEED + 77)
    base.update(kw)
    return VerifyConfig(**base)


def shard_sequences(batch: int, rank: int, world: int) -> range:
    """Contiguous block of sequence indices owned by ``rank`` when a batch is split over
    ``world`` processes (sequences are independent, so no exchange is needed)."""
    per, rem = divmod(batch, world)
    lo = rank * per + min(rank, rem)
    return range(lo, lo + per + (1 if rank < rem else 0))
