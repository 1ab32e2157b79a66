// The compressed, linear form of the tree mask (App. A.1 speaks of a tree mask that is a numerical
// comparison instead of an N x N matrix; its figure is missing, the encoding taken is depth-first
// entry/exit labels): tin = position of a node in a depth-first walk that visits children in
// increasing node index, tout = tin + size of its subtree.  Node j is an ancestor of node i, or i
// itself, exactly if tin[j] <= tin[i] < tout[j].  Both directions, one block of 128 threads per
// sequence (N <= 128: latency bound like the walk).
#include "clv_internal.cuh"

namespace clv {
namespace {

constexpr int kThreads = CLV_MAX_NODES;   // 128: one thread per node

__global__ void __launch_bounds__(kThreads) to_intervals_kernel(int N, const int32_t* parent, int32_t* tin,
                                                                int32_t* tout, int32_t* status) {
  __shared__ int sp[CLV_MAX_NODES], ssize[CLV_MAX_NODES], sin[CLV_MAX_NODES], soff[CLV_MAX_NODES];
  __shared__ int s_bad;
  const int b = blockIdx.x, i = threadIdx.x;
  cudaGridDependencySynchronize();
  if (i == 0) s_bad = 0;
  __syncthreads();
  if (i < N) {
    const int par = parent[(int64_t)b * N + i];
    sp[i] = par;
    ssize[i] = 1;
    soff[i] = 0;
    if (par < -1 || par >= i) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (i < N) { tin[(int64_t)b * N + i] = -1; tout[(int64_t)b * N + i] = -1; }
    if (i == 0) status[b] = CLV_ERR_TREE;
    return;
  }
  if (i == 0) {
    // parents come before children: sizes from the last node down, entry labels from the first up
    // (a node's label = its parent's + 1 + the sizes of its earlier siblings; roots follow each other)
    for (int v = N - 1; v >= 1; --v) if (sp[v] >= 0) ssize[sp[v]] += ssize[v];
    int root_off = 0;
    for (int v = 0; v < N; ++v) {
      const int par = sp[v];
      if (par < 0) { sin[v] = root_off; root_off += ssize[v]; }
      else { sin[v] = sin[par] + 1 + soff[par]; soff[par] += ssize[v]; }
    }
    status[b] = CLV_OK;
  }
  __syncthreads();
  if (i < N) { tin[(int64_t)b * N + i] = sin[i]; tout[(int64_t)b * N + i] = sin[i] + ssize[i]; }
}

__global__ void __launch_bounds__(kThreads) from_intervals_kernel(int N, const int32_t* tin, const int32_t* tout,
                                                                  int32_t* parent, int32_t* status) {
  __shared__ long long s0[CLV_MAX_NODES], s1[CLV_MAX_NODES];
  __shared__ int s_bad;
  const int b = blockIdx.x, i = threadIdx.x;
  cudaGridDependencySynchronize();
  if (i == 0) s_bad = 0;
  if (i < N) { s0[i] = tin[(int64_t)b * N + i]; s1[i] = tout[(int64_t)b * N + i]; }
  __syncthreads();
  int best = -1;
  if (i < N) {
    const long long a0 = s0[i], a1 = s1[i];
    bool bad = !(a1 > a0);
    for (int j = 0; j < N; ++j) {
      if (j == i) continue;
      const long long b0 = s0[j], b1 = s1[j];
      bad |= (b0 == a0);                         // two nodes with the same entry label
      bad |= (a0 < b0 && b0 < a1 && a1 < b1);    // overlap without nesting
      if (b0 <= a0 && a0 < b1 && (best < 0 || b1 - b0 < s1[best] - s0[best])) best = j;   // narrowest interval around i
    }
    bad |= (best >= i);                          // a parent must come before its child
    if (bad) s_bad = 1;
  }
  __syncthreads();
  if (i < N) parent[(int64_t)b * N + i] = s_bad ? -1 : best;
  if (i == 0) status[b] = s_bad ? CLV_ERR_TREE : CLV_OK;
}

template <class K, class... A>
cudaError_t launch_per_sequence(K kernel, int batch, cudaStream_t stream, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)batch, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

}  // namespace

cudaError_t launch_tree_to_intervals(int batch, int n_nodes, const int32_t* parent, int32_t* tin, int32_t* tout,
                                     int32_t* status, cudaStream_t stream) {
  return launch_per_sequence(to_intervals_kernel, batch, stream, n_nodes, parent, tin, tout, status);
}

cudaError_t launch_tree_from_intervals(int batch, int n_nodes, const int32_t* tin, const int32_t* tout,
                                       int32_t* parent, int32_t* status, cudaStream_t stream) {
  return launch_per_sequence(from_intervals_kernel, batch, stream, n_nodes, tin, tout, parent, status);
}

}  // namespace clv
