// Token tree from speculated sequences (Sec. 2.1, Fig. 2 caption: several speculations are merged
// by prefix matching into a tree).  One thread block per sequence; the sizes are tiny (at most 128
// candidates of at most 16 tokens), so the kernel is latency bound like the walk.
//
// A node is a distinct non-empty prefix of some candidate; node 0 is the root (the token the target
// emitted last).  Nodes are numbered by depth first, then by the lowest candidate that contains
// the prefix, which makes the numbering unique and topological (parent[i] < i).  Unused slots up
// to node_cap become children of the root with token -1: they never match a target token, so the
// arrays can go into a verify step of fixed size as they are.
#include "clv_internal.cuh"

namespace clv {
namespace {

constexpr int kMaxCand = CLV_TREE_MAX_CAND;   // 128
constexpr int kMaxLen = CLV_TREE_MAX_LEN;     // 16
constexpr int kThreads = 128;

struct Params {
  int n_cand, max_len, node_cap;
  const int32_t* root_token;
  const int32_t* cand;
  const int32_t* cand_len;
  int32_t* tokens;
  int32_t* parent;
  int32_t* n_nodes;
  int32_t* node_of;
  int32_t* status;
};

__global__ void __launch_bounds__(kThreads) token_tree_kernel(Params p) {
  // rep[d][c]: lowest candidate whose first d+1 tokens equal those of candidate c (-1: c is shorter)
  __shared__ int s_rep[kMaxLen][kMaxCand];
  __shared__ short s_node[kMaxLen][kMaxCand];   // node number of (depth d, candidate c) if c is its own rep
  __shared__ int s_cand[kMaxCand * kMaxLen];     // this sequence's candidates, [c][d]
  __shared__ int s_len[kMaxCand];
  __shared__ int s_total;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int C = p.n_cand, D = p.max_len;
  cudaGridDependencySynchronize();  // programmatic launch: the previous kernel's results are complete
  const int32_t* cand_g = p.cand + (int64_t)b * C * D;
  for (int w = tid; w < C * D; w += kThreads) s_cand[w] = cand_g[w];
  const int* cand = s_cand;
  bool bad = false;
  for (int c = tid; c < C; c += kThreads) {
    const int len = p.cand_len[(int64_t)b * C + c];
    bad |= (len < 0 || len > D);
    s_len[c] = min(max(len, 0), D);
  }
  bad = __syncthreads_or(bad ? 1 : 0) != 0;

  // ---- prefix matching, one depth after the other: candidate c' shares c's prefix of length d+1
  //      iff it shared the prefix of length d and carries the same token at depth d --------------
  // Every candidate's scan over the earlier ones is shared by `parts` threads (interleaved), which
  // combine with a shared-memory minimum.
  const int parts = max(1, kThreads / C);
  for (int d = 0; d < D; ++d) {
    for (int c = tid; c < C; c += kThreads) s_rep[d][c] = d < s_len[c] ? c : -1;
    __syncthreads();
    for (int w = tid; w < C * parts; w += kThreads) {
      const int c = w / parts, part = w - c * parts;
      if (d >= s_len[c]) continue;
      const int tok = cand[c * D + d];
      const int up = d == 0 ? 0 : s_rep[d - 1][c];
      int rep = c;
      const int* prev = s_rep[d == 0 ? 0 : d - 1];
#pragma unroll 4
      for (int o = part; o < c; o += parts) {
        // all three loads are issued whatever they return, so that the iterations overlap
        const bool match = (d < s_len[o]) & ((d == 0) | (prev[o] == up)) & (cand[o * D + d] == tok);
        rep = (match && o < rep) ? o : rep;
      }
      if (rep < c) atomicMin(&s_rep[d][c], rep);
    }
    __syncthreads();
  }

  // ---- number the nodes: depth major, candidate minor; one warp scans 32 positions at a time ----
  if (tid < 32) {
    int base = 1;  // node 0 is the root
    for (int d = 0; d < D; ++d) {
      for (int c0 = 0; c0 < C; c0 += 32) {
        const int c = c0 + tid;
        const bool is_new = c < C && s_rep[d][c] == c;
        const unsigned m = __ballot_sync(0xFFFFFFFFu, is_new);
        if (c < C) s_node[d][c] = is_new ? (short)min(base + __popc(m & ((1u << tid) - 1u)), 32767) : (short)-1;
        base += __popc(m);
      }
    }
    if (tid == 0) s_total = base;
  }
  __syncthreads();
  const int total = s_total;
  const bool fail = bad || total > p.node_cap;

  int32_t* tokens = p.tokens + (int64_t)b * p.node_cap;
  int32_t* parent = p.parent + (int64_t)b * p.node_cap;
  int32_t* node_of = p.node_of + (int64_t)b * C * D;
  // every slot first: the root, then padding that hangs off the root with a token nothing matches
  for (int i = tid; i < p.node_cap; i += kThreads) {
    tokens[i] = i == 0 ? p.root_token[b] : -1;
    parent[i] = i == 0 ? -1 : 0;
  }
  __syncthreads();
  for (int w = tid; w < C * D; w += kThreads) {
    const int c = w / D, d = w - c * D;
    const int rep = s_rep[d][c];
    int node = -1;
    if (!fail && rep >= 0) {
      node = s_node[d][rep];
      if (rep == c) {  // this candidate introduces the node
        tokens[node] = cand[c * D + d];
        parent[node] = d == 0 ? 0 : s_node[d - 1][s_rep[d - 1][c]];
      }
    }
    node_of[w] = node;
  }
  if (tid == 0) {
    p.n_nodes[b] = fail ? 1 : total;
    p.status[b] = fail ? CLV_ERR_TREE : CLV_OK;
  }
}

}  // namespace

cudaError_t launch_token_tree(int batch, int n_cand, int max_len, int node_cap, const int32_t* root_token,
                              const int32_t* cand, const int32_t* cand_len, int32_t* tokens, int32_t* parent,
                              int32_t* n_nodes, int32_t* node_of, int32_t* status, cudaStream_t stream) {
  Params p;
  p.n_cand = n_cand;
  p.max_len = max_len;
  p.node_cap = node_cap;
  p.root_token = root_token;
  p.cand = cand;
  p.cand_len = cand_len;
  p.tokens = tokens;
  p.parent = parent;
  p.n_nodes = n_nodes;
  p.node_of = node_of;
  p.status = status;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)batch, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, token_tree_kernel, p);
}

}  // namespace clv
