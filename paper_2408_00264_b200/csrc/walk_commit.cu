// Greedy acceptance walk (Sec. 2.1 verification phase) and KV commit (equivalence requirement of
// Sec. 2.1).  Both are latency-bound: one warp per sequence for the walk, one thread block per
// sequence for the row copies.
#include <limits.h>

#include "clv_internal.cuh"

namespace clv {
namespace {

// ------------------------------------------------------------------------------------ walk
struct WalkSmem {
  int sp[CLV_MAX_NODES], st[CLV_MAX_NODES], si[CLV_MAX_NODES], path[CLV_MAX_NODES];
};

// The walk of sequence b by one warp; returns the accepted length (0 if the tree is malformed).
// The path is left in sm.path[0 .. len) for the caller (visible after a __syncwarp / barrier).
__device__ __forceinline__ int walk_sequence(WalkSmem& sm, int b, int lane, int N, int path_cap,
                                             const int32_t* parent, const int32_t* tokens,
                                             const int32_t* ids, int32_t* accept_len, int32_t* accept_idx,
                                             int32_t* next_token, int32_t* status) {
  int* sp = sm.sp; int* st = sm.st; int* si = sm.si; int* path = sm.path;
  const int64_t o = (int64_t)b * N;
  bool bad = false;
  for (int i = lane; i < N; i += 32) {
    const int p = parent[o + i];
    sp[i] = p;
    st[i] = tokens[o + i];
    si[i] = ids[o + i];
    bad |= (i == 0) ? (p != -1) : (p < 0 || p >= i);  // node 0 is the only root
  }
  bad = __any_sync(0xFFFFFFFFu, bad) || path_cap < 1;
  __syncwarp();
  int len = 0, cur = 0;
  if (!bad) {
    if (lane == 0) path[0] = 0;
    len = 1;
    for (int step = 1; step < N; ++step) {  // a path has at most N nodes
      const int want = si[cur];
      int found = INT_MAX;
      for (int c = cur + 1 + lane; c < N; c += 32)
        if (sp[c] == cur && st[c] == want) { found = c; break; }
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) found = min(found, __shfl_xor_sync(0xFFFFFFFFu, found, s));
      if (found == INT_MAX) break;
      if (len == path_cap || len == CLV_MAX_NODES) { bad = true; break; }
      if (lane == 0) path[len] = found;
      ++len;
      cur = found;
    }
  }
  __syncwarp();
  if (bad) len = 0;
  for (int j = lane; j < path_cap; j += 32)
    accept_idx[(int64_t)b * path_cap + j] = (j < len) ? path[j] : -1;
  if (lane == 0) {
    accept_len[b] = len;
    next_token[b] = bad ? -1 : si[cur];
    status[b] = bad ? CLV_ERR_TREE : CLV_OK;
  }
  return len;
}

__global__ void __launch_bounds__(32) walk_kernel(int N, int path_cap, const int32_t* parent,
                                                  const int32_t* tokens, const int32_t* ids,
                                                  int32_t* accept_len, int32_t* accept_idx,
                                                  int32_t* next_token, int32_t* status) {
  __shared__ WalkSmem sm;
  // Launched with programmatic stream serialisation: this grid may be set up while the previous
  // kernel of the stream is still draining, so wait for that kernel's results here, and let the
  // next kernel (the commit) start its own set-up right away.
  cudaGridDependencySynchronize();
  cudaTriggerProgrammaticLaunchCompletion();
  walk_sequence(sm, blockIdx.x, threadIdx.x, N, path_cap, parent, tokens, ids, accept_len, accept_idx,
                next_token, status);
}

// ------------------------------------------------------------------------------------ commit
struct CommitParams {
  uint4* kc;
  uint4* vc;
  const uint4* k_tree;
  const uint4* v_tree;
  const int32_t* block_table;
  const int32_t* accept_idx;
  const int32_t* accept_len;
  const int32_t* ctx_len;
  int32_t* ctx_len_out;
  int32_t* status;
  int N, path_cap, paged, cap_tokens, n_pages, max_pages;
  int row_vec;  // 16-byte vectors per token row: Hkv * 128 * 2 / 16
};

struct CommitSmem {
  int src[CLV_MAX_NODES];
  long long dst[CLV_MAX_NODES];  // destination token row (global row index)
  int ok;
};

// The commit of sequence b by one thread block (accept_len / accept_idx are read from memory).
__device__ __forceinline__ void commit_sequence(CommitSmem& sm, const CommitParams& p, int b, int tid) {
  int* s_src = sm.src;
  long long* s_dst = sm.dst;
  int& s_ok = sm.ok;
  const int L = p.ctx_len[b];
  const int len = p.accept_len[b];
  if (tid == 0) s_ok = (L >= 0 && len >= 0 && len <= p.path_cap && len <= CLV_MAX_NODES) ? 1 : 0;
  __syncthreads();
  if (s_ok) {
    for (int j = tid; j < len; j += blockDim.x) {
      const int a = p.accept_idx[(int64_t)b * p.path_cap + j];
      const long long t = (long long)L + j;
      long long row = -1;
      if (p.paged) {
        const long long lp = t / CLV_PAGE_SIZE;
        if (lp < p.max_pages) {
          const int pg = p.block_table[(int64_t)b * p.max_pages + lp];
          if (pg >= 0 && pg < p.n_pages) row = (long long)pg * CLV_PAGE_SIZE + t % CLV_PAGE_SIZE;
        }
      } else if (t < p.cap_tokens) {
        row = (long long)b * p.cap_tokens + t;
      }
      if (a < 0 || a >= p.N || row < 0) s_ok = 0;  // benign race: every writer stores 0
      s_src[j] = a;
      s_dst[j] = row;
    }
  }
  __syncthreads();
  if (!s_ok) {
    if (tid == 0) { p.ctx_len_out[b] = L; p.status[b] = CLV_ERR_TREE; }
    return;
  }
  const int per_row = 2 * p.row_vec;  // K then V
  for (int w = tid; w < len * per_row; w += blockDim.x) {
    const int j = w / per_row, r = w - j * per_row;
    const int c = (r < p.row_vec) ? r : r - p.row_vec;
    const int64_t src = ((int64_t)b * p.N + s_src[j]) * p.row_vec + c;
    const int64_t dst = s_dst[j] * p.row_vec + c;
    if (r < p.row_vec) p.kc[dst] = p.k_tree[src];
    else p.vc[dst] = p.v_tree[src];
  }
  if (tid == 0) { p.ctx_len_out[b] = L + len; p.status[b] = CLV_OK; }
}

__global__ void __launch_bounds__(256) commit_kernel(CommitParams p) {
  __shared__ CommitSmem sm;
  cudaGridDependencySynchronize();  // programmatic launch: the walk's outputs are complete after this
  cudaTriggerProgrammaticLaunchCompletion();  // a following kernel may set up; it waits for this grid itself
  commit_sequence(sm, p, blockIdx.x, threadIdx.x);
}

// Walk and commit of a sequence in one launch: warp 0 walks, then the whole block copies the rows.
struct WalkArgs {
  int N, path_cap;
  const int32_t* parent;
  const int32_t* tokens;
  const int32_t* ids;
  int32_t* accept_len;
  int32_t* accept_idx;
  int32_t* next_token;
  int32_t* status;
};
__global__ void __launch_bounds__(256) walk_commit_kernel(WalkArgs w, CommitParams p) {
  __shared__ WalkSmem wsm;
  __shared__ CommitSmem csm;
  cudaGridDependencySynchronize();
  cudaTriggerProgrammaticLaunchCompletion();
  if (threadIdx.x < 32)
    walk_sequence(wsm, blockIdx.x, threadIdx.x, w.N, w.path_cap, w.parent, w.tokens, w.ids, w.accept_len,
                  w.accept_idx, w.next_token, w.status);
  __syncthreads();  // the walk's results, written by this block, are visible to all of it
  commit_sequence(csm, p, blockIdx.x, threadIdx.x);
}

// The commit of every layer of a model in one launch: block (b, layer) copies the accepted rows of
// sequence b in that layer's tree buffers into that layer's cache.  All layers share the accepted
// path, the context lengths and (paged) the block table, so every block of a sequence reaches the
// same verdict; ctx_len_out and status are written by each of them with the same values.
__global__ void __launch_bounds__(256) commit_layers_kernel(CommitParams p, long long cache_stride_vec,
                                                            long long tree_stride_vec) {
  __shared__ CommitSmem sm;
  cudaGridDependencySynchronize();
  cudaTriggerProgrammaticLaunchCompletion();
  const long long layer = blockIdx.y;
  p.kc += layer * cache_stride_vec;
  p.vc += layer * cache_stride_vec;
  p.k_tree += layer * tree_stride_vec;
  p.v_tree += layer * tree_stride_vec;
  commit_sequence(sm, p, blockIdx.x, threadIdx.x);
}

}  // namespace

cudaError_t launch_walk(const clv_shape& s, const int32_t* parent, const int32_t* tokens,
                        const int32_t* ids, int32_t* accept_len, int32_t* accept_idx,
                        int32_t* next_token, int32_t* status, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)s.batch, 1, 1);
  cfg.blockDim = dim3(32, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, walk_kernel, (int)s.n_nodes, (int)s.path_cap, parent, tokens, ids, accept_len,
                            accept_idx, next_token, status);
}

namespace {
CommitParams commit_params(const clv_shape& s, const clv_kv_cache& c, const void* k_tree, const void* v_tree,
                           const int32_t* accept_idx, const int32_t* accept_len, const int32_t* ctx_len,
                           int32_t* ctx_len_out, int32_t* status) {
  CommitParams p;
  p.kc = static_cast<uint4*>(c.k);
  p.vc = static_cast<uint4*>(c.v);
  p.k_tree = static_cast<const uint4*>(k_tree);
  p.v_tree = static_cast<const uint4*>(v_tree);
  p.block_table = c.block_table;
  p.accept_idx = accept_idx;
  p.accept_len = accept_len;
  p.ctx_len = ctx_len;
  p.ctx_len_out = ctx_len_out;
  p.status = status;
  p.N = s.n_nodes;
  p.path_cap = s.path_cap;
  p.paged = c.paged;
  p.cap_tokens = c.cap_tokens;
  p.n_pages = c.n_pages;
  p.max_pages = c.max_pages_per_seq;
  p.row_vec = s.n_kv_heads * CLV_HEAD_DIM * 2 / 16;
  return p;
}
}  // namespace

cudaError_t launch_commit(const clv_shape& s, const clv_kv_cache& c, const void* k_tree,
                          const void* v_tree, const int32_t* accept_idx, const int32_t* accept_len,
                          const int32_t* ctx_len, int32_t* ctx_len_out, int32_t* status,
                          cudaStream_t stream) {
  const CommitParams p = commit_params(s, c, k_tree, v_tree, accept_idx, accept_len, ctx_len, ctx_len_out, status);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)s.batch, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, commit_kernel, p);
}

cudaError_t launch_walk_commit(const clv_shape& s, const clv_kv_cache& c, const int32_t* parent,
                               const int32_t* tokens, const int32_t* ids, const void* k_tree,
                               const void* v_tree, const int32_t* ctx_len, int32_t* accept_len,
                               int32_t* accept_idx, int32_t* next_token, int32_t* ctx_len_out,
                               int32_t* walk_status, int32_t* commit_status, cudaStream_t stream) {
  const CommitParams p =
      commit_params(s, c, k_tree, v_tree, accept_idx, accept_len, ctx_len, ctx_len_out, commit_status);
  WalkArgs w;
  w.N = s.n_nodes;
  w.path_cap = s.path_cap;
  w.parent = parent;
  w.tokens = tokens;
  w.ids = ids;
  w.accept_len = accept_len;
  w.accept_idx = accept_idx;
  w.next_token = next_token;
  w.status = walk_status;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)s.batch, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, walk_commit_kernel, w, p);
}

cudaError_t launch_commit_layers(const clv_shape& s, const clv_kv_cache& c, int n_layers, int64_t cache_layer_stride,
                                 const void* k_tree, const void* v_tree, int64_t tree_layer_stride,
                                 const int32_t* accept_idx, const int32_t* accept_len, const int32_t* ctx_len,
                                 int32_t* ctx_len_out, int32_t* status, cudaStream_t stream) {
  const CommitParams p = commit_params(s, c, k_tree, v_tree, accept_idx, accept_len, ctx_len, ctx_len_out, status);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)s.batch, (unsigned)n_layers, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, commit_layers_kernel, p, (long long)(cache_layer_stride / 8),
                            (long long)(tree_layer_stride / 8));
}

}  // namespace clv
