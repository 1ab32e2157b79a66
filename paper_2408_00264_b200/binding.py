"""ctypes binding of libclv.so: argument marshalling only.

Every function has the name of the C entry point it forwards to (see ``include/clv.h``) and takes
torch CUDA tensors; all arithmetic of the verify step runs in the library's kernels.  There is no
CPU fallback: if the shared library has not been built, :func:`lib` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libclv.so")

CLV_OK = 0
CLV_ERR_NULL, CLV_ERR_SHAPE, CLV_ERR_UNSUPPORTED, CLV_ERR_ALIGN = 1, 2, 3, 4
CLV_ERR_WORKSPACE, CLV_ERR_CUDA, CLV_ERR_TREE, CLV_ERR_TIMEOUT = 5, 6, 7, 8
CLV_ERR_TOO_LARGE = 9

EXPORTS = (
    "clv_workspace_bytes", "clv_workspace_init", "clv_tree_attn", "clv_accept_argmax",
    "clv_accept_walk", "clv_kv_commit", "clv_staging_bytes", "clv_verify_step_host",
    "clv_status_string", "clv_last_cuda_error", "clv_version", "clv_accept_argmax_noalloc",
    "clv_lm_head_argmax", "clv_build_token_tree", "clv_accept_walk_commit", "clv_accept_sample",
    "clv_tree_to_intervals", "clv_tree_from_intervals", "clv_kv_commit_layers",
    "clv_draft_head_step", "clv_draft_head_workspace_bytes",
    "clv_test_set_wait_limit",
)


class ClvShape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_nodes", ctypes.c_int32),
                ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("vocab", ctypes.c_int32),
                ("path_cap", ctypes.c_int32)]


class ClvKvCache(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("paged", ctypes.c_int32),
                ("cap_tokens", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("n_pages", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
                ("block_table", ctypes.c_void_p)]


class ClvHostInputs(ctypes.Structure):
    _fields_ = [("q", ctypes.c_void_p), ("k_tree", ctypes.c_void_p), ("v_tree", ctypes.c_void_p),
                ("parent", ctypes.c_void_p), ("tokens", ctypes.c_void_p),
                ("logits", ctypes.c_void_p), ("ld", ctypes.c_int64)]


class ClvHostOutputs(ctypes.Structure):
    _fields_ = [("out", ctypes.c_void_p), ("argmax_ids", ctypes.c_void_p),
                ("accept_len", ctypes.c_void_p), ("accept_idx", ctypes.c_void_p),
                ("next_token", ctypes.c_void_p), ("status", ctypes.c_void_p)]


class ClvDraftHead(ctypes.Structure):
    _fields_ = [("hidden_dim", ctypes.c_int32), ("n_heads", ctypes.c_int32), ("vocab", ctypes.c_int32),
                ("rms_eps", ctypes.c_float)] + [(n, ctypes.c_void_p) for n in (
                    "norm1", "norm2", "wq", "wk", "wv", "bq", "bk", "bv", "wfc", "bfc", "lm_head")]


class ClvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().clv_status_string(code).decode()
        if code == CLV_ERR_CUDA:
            msg += " (cudaError %d)" % lib().clv_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libclv.so is missing at %s: build it with `python -m paper_2408_00264_b200.build`"
                % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz, f32 = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t,
                                 ctypes.c_float)
        L.clv_workspace_bytes.restype = sz
        L.clv_workspace_bytes.argtypes = [vp, vp, i32]
        L.clv_workspace_init.restype = i32
        L.clv_workspace_init.argtypes = [vp, sz, vp]
        L.clv_tree_attn.restype = i32
        L.clv_tree_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp, sz, vp]
        L.clv_accept_argmax.restype = i32
        L.clv_accept_argmax.argtypes = [vp, vp, i64, vp, vp, sz, vp]
        L.clv_accept_argmax_noalloc.restype = i32
        L.clv_accept_argmax_noalloc.argtypes = [vp, vp, i64, vp, vp]
        L.clv_lm_head_argmax.restype = i32
        L.clv_lm_head_argmax.argtypes = [vp, i64, vp, i64, i32, i32, i32, vp, vp, vp, sz, vp]
        L.clv_accept_walk_commit.restype = i32
        L.clv_accept_walk_commit.argtypes = [vp] * 15
        L.clv_tree_to_intervals.restype = i32
        L.clv_tree_to_intervals.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        L.clv_tree_from_intervals.restype = i32
        L.clv_tree_from_intervals.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        L.clv_kv_commit_layers.restype = i32
        L.clv_kv_commit_layers.argtypes = [vp, vp, i32, i64, vp, vp, i64, vp, vp, vp, vp, vp, vp]
        L.clv_draft_head_workspace_bytes.restype = sz
        L.clv_draft_head_workspace_bytes.argtypes = [i32, i32, i32]
        L.clv_draft_head_step.restype = i32
        L.clv_draft_head_step.argtypes = [vp, i32, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
        L.clv_accept_sample.restype = i32
        L.clv_accept_sample.argtypes = [vp, vp, i64, vp, vp, vp, f32, vp, vp, vp, vp, vp, sz, vp]
        L.clv_build_token_tree.restype = i32
        L.clv_build_token_tree.argtypes = [i32, i32, i32, i32] + [vp] * 9
        L.clv_accept_walk.restype = i32
        L.clv_accept_walk.argtypes = [vp] * 9
        L.clv_kv_commit.restype = i32
        L.clv_kv_commit.argtypes = [vp] * 10
        L.clv_staging_bytes.restype = sz
        L.clv_staging_bytes.argtypes = [vp, i64]
        L.clv_verify_step_host.restype = i32
        L.clv_verify_step_host.argtypes = [vp, vp, vp, vp, vp, i32, f32, vp, sz, vp, sz, vp]
        L.clv_status_string.restype = ctypes.c_char_p
        L.clv_status_string.argtypes = [i32]
        L.clv_last_cuda_error.restype = ctypes.c_int
        L.clv_version.restype = ctypes.c_int
        L.clv_test_set_wait_limit.restype = None
        L.clv_test_set_wait_limit.argtypes = [i64]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ref(s):
    return ctypes.cast(ctypes.byref(s), ctypes.c_void_p)


def make_shape(batch, n_nodes, n_q_heads, n_kv_heads, vocab=0, path_cap=1, head_dim=128) -> ClvShape:
    return ClvShape(batch, n_nodes, n_q_heads, n_kv_heads, head_dim, vocab, path_cap)


def make_cache(k: torch.Tensor, v: torch.Tensor, block_table: Optional[torch.Tensor] = None
               ) -> ClvKvCache:
    """Contiguous cache [B, cap, Hkv, 128] or, with a block table, a paged pool [P, 64, Hkv, 128]."""
    if block_table is None:
        return ClvKvCache(k.data_ptr(), v.data_ptr(), 0, k.shape[1], 64, 0, 0, None)
    return ClvKvCache(k.data_ptr(), v.data_ptr(), 1, 0, k.shape[1], k.shape[0],
                      block_table.shape[1], block_table.data_ptr())


def _check(code: int, where: str) -> None:
    if code != CLV_OK:
        raise ClvError(code, where)


def clv_workspace_bytes(shape: ClvShape, cache: Optional[ClvKvCache], max_ctx_len: int) -> int:
    return int(lib().clv_workspace_bytes(_ref(shape), None if cache is None else _ref(cache),
                                         int(max_ctx_len)))


def clv_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check(lib().clv_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                    _stream(stream)), "clv_workspace_init")


def new_workspace(shape: ClvShape, cache: Optional[ClvKvCache], max_ctx_len: int,
                  device="cuda") -> torch.Tensor:
    """Allocate (through torch) and initialise a workspace of the required size."""
    n = clv_workspace_bytes(shape, cache, max_ctx_len)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    clv_workspace_init(ws)
    return ws


def clv_tree_attn(shape, cache, q, k_tree, v_tree, parent, ctx_len, max_ctx_len, softmax_scale,
                  out, lse, status, workspace, stream=None, check=True) -> int:
    code = lib().clv_tree_attn(_ref(shape), _ref(cache), _ptr(q), _ptr(k_tree), _ptr(v_tree),
                               _ptr(parent), _ptr(ctx_len), int(max_ctx_len), float(softmax_scale),
                               _ptr(out), _ptr(lse), _ptr(status), _ptr(workspace),
                               0 if workspace is None else workspace.numel() * workspace.element_size(),
                               _stream(stream))
    if check:
        _check(code, "clv_tree_attn")
    return code


def clv_accept_argmax(shape, logits, ld, argmax_ids, workspace, stream=None, check=True) -> int:
    code = lib().clv_accept_argmax(_ref(shape), _ptr(logits), int(ld), _ptr(argmax_ids),
                                   _ptr(workspace),
                                   0 if workspace is None else workspace.numel() * workspace.element_size(),
                                   _stream(stream))
    if check:
        _check(code, "clv_accept_argmax")
    return code


def clv_accept_argmax_noalloc(shape, logits, ld, argmax_ids, stream=None, check=True) -> int:
    """clv_accept_argmax for callers that may not allocate device memory: no workspace argument,
    the scratch is a fixed array inside the library (limits and sharing rules in clv.h)."""
    code = lib().clv_accept_argmax_noalloc(_ref(shape), _ptr(logits), int(ld), _ptr(argmax_ids),
                                           _stream(stream))
    if check:
        _check(code, "clv_accept_argmax_noalloc")
    return code


def clv_accept_walk_commit(shape, cache, parent, tokens, argmax_ids, k_tree, v_tree, ctx_len, accept_len,
                           accept_idx, next_token, ctx_len_out, walk_status, commit_status, stream=None,
                           check=True) -> int:
    code = lib().clv_accept_walk_commit(_ref(shape), _ref(cache), _ptr(parent), _ptr(tokens),
                                        _ptr(argmax_ids), _ptr(k_tree), _ptr(v_tree), _ptr(ctx_len),
                                        _ptr(accept_len), _ptr(accept_idx), _ptr(next_token),
                                        _ptr(ctx_len_out), _ptr(walk_status), _ptr(commit_status),
                                        _stream(stream))
    if check:
        _check(code, "clv_accept_walk_commit")
    return code


def clv_accept_sample(shape, logits, ld, parent, tokens, uniforms, temperature, accept_len, accept_idx,
                      next_token, status, workspace, stream=None, check=True) -> int:
    """uniforms: float32 [B, N + 1] in [0, 1); temperature: python float > 0."""
    code = lib().clv_accept_sample(_ref(shape), _ptr(logits), int(ld), _ptr(parent), _ptr(tokens),
                                   _ptr(uniforms), float(temperature), _ptr(accept_len), _ptr(accept_idx),
                                   _ptr(next_token), _ptr(status), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream(stream))
    if check:
        _check(code, "clv_accept_sample")
    return code


def clv_tree_to_intervals(parent, tin, tout, status, stream=None, check=True) -> int:
    """parent, tin, tout: int32 [B, N]; status int32 [B]."""
    B, N = parent.shape
    code = lib().clv_tree_to_intervals(int(B), int(N), _ptr(parent), _ptr(tin), _ptr(tout), _ptr(status),
                                       _stream(stream))
    if check:
        _check(code, "clv_tree_to_intervals")
    return code


def clv_tree_from_intervals(tin, tout, parent, status, stream=None, check=True) -> int:
    B, N = tin.shape
    code = lib().clv_tree_from_intervals(int(B), int(N), _ptr(tin), _ptr(tout), _ptr(parent), _ptr(status),
                                         _stream(stream))
    if check:
        _check(code, "clv_tree_from_intervals")
    return code


def clv_kv_commit_layers(shape, cache, n_layers, cache_layer_stride, k_tree, v_tree, tree_layer_stride,
                         accept_idx, accept_len, ctx_len, ctx_len_out, status, stream=None, check=True) -> int:
    """cache: descriptor of layer 0; the strides are in bf16 elements between consecutive layers."""
    code = lib().clv_kv_commit_layers(_ref(shape), _ref(cache), int(n_layers), int(cache_layer_stride),
                                      _ptr(k_tree), _ptr(v_tree), int(tree_layer_stride), _ptr(accept_idx),
                                      _ptr(accept_len), _ptr(ctx_len), _ptr(ctx_len_out), _ptr(status),
                                      _stream(stream))
    if check:
        _check(code, "clv_kv_commit_layers")
    return code


def make_draft_head(weights: dict, rms_eps: float = 1e-5) -> ClvDraftHead:
    """weights: torch bf16 CUDA tensors under the names of ClvDraftHead's pointer fields, plus
    ``n_heads``; the tensors must stay alive while the descriptor is used."""
    H = weights["wq"].shape[0]
    d = ClvDraftHead(int(H), int(weights["n_heads"]), int(weights["lm_head"].shape[0]), float(rms_eps))
    for n in ("norm1", "norm2", "wq", "wk", "wv", "bq", "bk", "bv", "wfc", "bfc", "lm_head"):
        setattr(d, n, weights[n].data_ptr())
    return d


def clv_draft_head_step(head, h, e, k_top, hidden_out, top_ids, top_logits, status, workspace, stream=None,
                        check=True) -> int:
    """h, e, hidden_out: bf16 [rows, hidden]; top_ids int32 / top_logits float32 [rows, k_top]; status int32 [5]."""
    code = lib().clv_draft_head_step(_ref(head), int(h.shape[0]), _ptr(h), _ptr(e), int(k_top), _ptr(hidden_out),
                                     _ptr(top_ids), _ptr(top_logits), _ptr(status), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream))
    if check:
        _check(code, "clv_draft_head_step")
    return code


def new_draft_head_workspace(rows: int, hidden_dim: int, vocab: int, device="cuda") -> torch.Tensor:
    n = int(lib().clv_draft_head_workspace_bytes(int(rows), int(hidden_dim), int(vocab)))
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    clv_workspace_init(ws)
    return ws


def clv_build_token_tree(root_token, cand, cand_len, tokens, parent, n_nodes, node_of, status,
                         stream=None, check=True) -> int:
    """cand int32 [B, n_cand, max_len], cand_len [B, n_cand], root_token [B]; outputs tokens and
    parent [B, node_cap], n_nodes [B], node_of [B, n_cand, max_len], status [B] (all int32)."""
    B, C, D = cand.shape
    code = lib().clv_build_token_tree(int(B), int(C), int(D), int(tokens.shape[1]), _ptr(root_token),
                                      _ptr(cand), _ptr(cand_len), _ptr(tokens), _ptr(parent),
                                      _ptr(n_nodes), _ptr(node_of), _ptr(status), _stream(stream))
    if check:
        _check(code, "clv_build_token_tree")
    return code


def clv_lm_head_argmax(hidden, weight, argmax_ids, status, workspace, stream=None, check=True) -> int:
    """hidden bf16 [rows, hidden_dim], weight bf16 [vocab, hidden_dim] (row strides taken from the
    tensors), argmax_ids int32 [rows], status int32 [1]."""
    rows, hidden_dim = hidden.shape
    vocab = weight.shape[0]
    code = lib().clv_lm_head_argmax(_ptr(hidden), int(hidden.stride(0)), _ptr(weight),
                                    int(weight.stride(0)), int(rows), int(hidden_dim), int(vocab),
                                    _ptr(argmax_ids), _ptr(status), _ptr(workspace),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _stream(stream))
    if check:
        _check(code, "clv_lm_head_argmax")
    return code


def clv_accept_walk(shape, parent, tokens, argmax_ids, accept_len, accept_idx, next_token, status,
                    stream=None, check=True) -> int:
    code = lib().clv_accept_walk(_ref(shape), _ptr(parent), _ptr(tokens), _ptr(argmax_ids),
                                 _ptr(accept_len), _ptr(accept_idx), _ptr(next_token), _ptr(status),
                                 _stream(stream))
    if check:
        _check(code, "clv_accept_walk")
    return code


def clv_kv_commit(shape, cache, k_tree, v_tree, accept_idx, accept_len, ctx_len, ctx_len_out, status,
                  stream=None, check=True) -> int:
    code = lib().clv_kv_commit(_ref(shape), _ref(cache), _ptr(k_tree), _ptr(v_tree),
                               _ptr(accept_idx), _ptr(accept_len), _ptr(ctx_len), _ptr(ctx_len_out),
                               _ptr(status), _stream(stream))
    if check:
        _check(code, "clv_kv_commit")
    return code


def clv_staging_bytes(shape: ClvShape, ld: int) -> int:
    return int(lib().clv_staging_bytes(_ref(shape), int(ld)))


def clv_verify_step_host(shape, cache, host_in: ClvHostInputs, host_out: ClvHostOutputs, ctx_len,
                         max_ctx_len, softmax_scale, staging, workspace, stream=None,
                         check=True) -> int:
    code = lib().clv_verify_step_host(_ref(shape), _ref(cache), _ref(host_in), _ref(host_out),
                                      _ptr(ctx_len), int(max_ctx_len), float(softmax_scale),
                                      _ptr(staging), staging.numel() * staging.element_size(),
                                      _ptr(workspace),
                                      0 if workspace is None else workspace.numel() * workspace.element_size(),
                                      _stream(stream))
    if check:
        _check(code, "clv_verify_step_host")
    return code


def clv_version() -> int:
    return int(lib().clv_version())


def clv_status_string(code: int) -> str:
    return lib().clv_status_string(int(code)).decode()


def clv_test_set_wait_limit(sm_cycles: int) -> None:
    """Tests only: SM cycles after which a bounded on-chip wait gives up (<= 0: the default)."""
    lib().clv_test_set_wait_limit(int(sm_cycles))
