// One step of a Clover-2 draft head (Sec. 3.1; App. A.3 prints the Attention Decoder) for a few
// rows (one per sequence and candidate):
//   Attention Decoder:  x = RMSNorm(h; norm1);  q = x Wq^T + bq;  k = e Wk^T + bk;  v = e Wv^T + bv;
//     per head j: gate_j = <q_j, k_j> / max(|q_j| |k_j|, 1e-8);  a = h + v * gate   (no activation)
//   output projector:   p = [a, e] Wfc^T + bfc        (fully connected, over a and the token embedding)
//   proposals:          logits = RMSNorm(p; norm2) lm_head^T;  the k largest per row
// h = hidden state (of the target, or of the previous head), e = embedding of the last token.
// The five products run on the tensor cores (the row-block GEMM of the LM head kernel with its
// accumulators written out, fp32): with a handful of rows they stream their weights once, which
// is what bounds the step (1.22 GB at hidden 4096, vocabulary 128256).  The operands of a product
// are bf16 (x, a, e, RMSNorm(p) are rounded once, like the activations of a bf16 model); sums,
// gates and logits stay fp32.  The small kernels here do the rest: one block per row.
#include <limits.h>
#include <math.h>

#include "clv_internal.cuh"

namespace clv {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float bf16f(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t f2bf(float x) {
  const __nv_bfloat16 v = __float2bfloat16_rn(x);
  return *reinterpret_cast<const uint16_t*>(&v);
}
__device__ __forceinline__ float block_sum(float v, float* s_red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  __syncthreads();   // s_red may still be read from the previous use
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < kThreads / 32; ++w) t += s_red[w];
  return t;
}

// the sum of the `parts` partial products of one element (a product's K axis may be cut in parts)
__device__ __forceinline__ float sum_parts(const float* x, int64_t i, int parts, int64_t stride) {
  float v = x[i];
  for (int s = 1; s < parts; ++s) v += x[i + s * stride];
  return v;
}

// y = RMSNorm(x; gain) rounded to bf16; x is bf16 (x32 == NULL) or fp32 in `parts` parts.
// Optionally also x itself rounded to bf16 (the head's hidden state, handed to the next head).
__global__ void __launch_bounds__(kThreads) rmsnorm_rows_kernel(int H, const uint16_t* x16, const float* x32,
                                                                int parts, int64_t stride, const uint16_t* gain,
                                                                float eps, uint16_t* y, uint16_t* x_out) {
  __shared__ float s_red[kThreads / 32];
  const int r = blockIdx.x;
  cudaGridDependencySynchronize();
  float ss = 0.f;
  for (int i = threadIdx.x; i < H; i += kThreads) {
    const float v = x32 ? sum_parts(x32, (int64_t)r * H + i, parts, stride) : bf16f(x16[(int64_t)r * H + i]);
    ss += v * v;
  }
  const float inv = rsqrtf(block_sum(ss, s_red) / (float)H + eps);
  for (int i = threadIdx.x; i < H; i += kThreads) {
    const float v = x32 ? sum_parts(x32, (int64_t)r * H + i, parts, stride) : bf16f(x16[(int64_t)r * H + i]);
    y[(int64_t)r * H + i] = f2bf(v * inv * bf16f(gain[i]));
    if (x_out) x_out[(int64_t)r * H + i] = f2bf(v);
  }
}

// a = h + v * gate (per head: cosine of q and k), written with e behind it: cat[r] = [a, e] (bf16).
// One warp per head, eight heads per block; q, k, v arrive in `parts` parts.
__global__ void __launch_bounds__(kThreads) gate_residual_kernel(int H, int n_heads, const float* q, const float* k,
                                                                 const float* v, int parts, int64_t stride,
                                                                 const uint16_t* h, const uint16_t* e, uint16_t* cat) {
  const int r = blockIdx.x, hd = H / n_heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.y * (kThreads / 32) + warp;
  cudaGridDependencySynchronize();
  if (j < n_heads) {
    const int64_t o = (int64_t)r * H + (int64_t)j * hd;
    float qk = 0.f, qq = 0.f, kk = 0.f;
    for (int i = lane; i < hd; i += 32) {
      const float a = sum_parts(q, o + i, parts, stride), b = sum_parts(k, o + i, parts, stride);
      qk += a * b; qq += a * a; kk += b * b;
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
      qk += __shfl_xor_sync(0xFFFFFFFFu, qk, s);
      qq += __shfl_xor_sync(0xFFFFFFFFu, qq, s);
      kk += __shfl_xor_sync(0xFFFFFFFFu, kk, s);
    }
    const float gate = qk / fmaxf(sqrtf(qq) * sqrtf(kk), 1e-8f);
    for (int i = lane; i < hd; i += 32) {
      cat[(int64_t)r * 2 * H + (int64_t)j * hd + i] = f2bf(bf16f(h[o + i]) + sum_parts(v, o + i, parts, stride) * gate);
      cat[(int64_t)r * 2 * H + H + (int64_t)j * hd + i] = e[o + i];
    }
  }
}

// The k largest logits of a row, highest first, lower index first among equals.  Up to 16: one
// pass in which every thread keeps the k best of its share in registers (sorted; an element that
// does not beat the thread's k-th costs one comparison), then k rounds of a block-wide argmax over
// the 256 heads of those lists.  More than 16: k passes over the row (it stays in L2), each
// excluding what the passes before it took.
constexpr int kListMax = 16;
__device__ __forceinline__ bool before(float v, int i, float bv, int bi) {   // order: value desc, index asc
  return (v > bv) || (v == bv && i < bi);
}
__global__ void __launch_bounds__(kThreads) topk_rows_kernel(int V, int64_t ld, int k_top, const float* logits,
                                                             int32_t* ids, float* vals) {
  __shared__ float s_v[kThreads / 32];
  __shared__ int s_i[kThreads / 32];
  __shared__ int s_win;
  __shared__ float s_last_v;
  __shared__ int s_last_i;
  const int r = blockIdx.x, tid = threadIdx.x;
  const float* row = logits + (int64_t)r * ld;
  cudaGridDependencySynchronize();
  if (k_top <= kListMax) {
    float lv[kListMax];
    int li[kListMax];
#pragma unroll
    for (int t = 0; t < kListMax; ++t) { lv[t] = -INFINITY; li[t] = INT_MAX; }
    for (int i = tid; i < V; i += kThreads) {
      float x = row[i];
      if (x != x) x = -INFINITY;   // NaN: last
      if (!before(x, i, lv[kListMax - 1], li[kListMax - 1])) continue;
      // insert: shift everything that comes after (x, i) down by one
#pragma unroll
      for (int t = kListMax - 1; t >= 0; --t) {
        const bool here = (t == 0) || !before(x, i, lv[t - 1], li[t - 1]);
        if (before(x, i, lv[t], li[t])) {
          if (here) { lv[t] = x; li[t] = i; }
          else { lv[t] = lv[t - 1]; li[t] = li[t - 1]; }
        }
      }
    }
    // note: only the first k_top entries of a list can matter
    int head = 0;   // this thread's next candidate
    for (int t = 0; t < k_top; ++t) {
      float bv = -INFINITY;
      int bi = INT_MAX;
#pragma unroll
      for (int u = 0; u < kListMax; ++u) if (u == head) { bv = lv[u]; bi = li[u]; }
      int who = tid;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
        const int ow = __shfl_xor_sync(0xFFFFFFFFu, who, o);
        if (before(ov, oi, bv, bi)) { bv = ov; bi = oi; who = ow; }
      }
      __syncthreads();   // the previous round's s_win has been read
      if ((tid & 31) == 0) { s_v[tid >> 5] = bv; s_i[tid >> 5] = bi; }
      __syncthreads();
      if (tid == 0) {
        for (int w = 1; w < kThreads / 32; ++w)
          if (before(s_v[w], s_i[w], bv, bi)) { bv = s_v[w]; bi = s_i[w]; }
        ids[(int64_t)r * k_top + t] = (bi == INT_MAX) ? -1 : bi;   // fewer than k entries
        vals[(int64_t)r * k_top + t] = bv;
        s_win = bi;
      }
      __syncthreads();
      const int win = s_win;
      bool mine = false;
#pragma unroll
      for (int u = 0; u < kListMax; ++u) mine |= (u == head && li[u] == win && win != INT_MAX);
      if (mine) ++head;
    }
    return;
  }
  float last_v = INFINITY;
  int last_i = -1;
  for (int t = 0; t < k_top; ++t) {
    // candidates: everything that comes after (last_v, last_i) in the order (value desc, index asc)
    float bv = -INFINITY;
    int bi = INT_MAX;
    for (int i = tid; i < V; i += kThreads) {
      float x = row[i];
      if (x != x) x = -INFINITY;
      const bool after = (x < last_v) || (x == last_v && i > last_i);
      if (after && before(x, i, bv, bi)) { bv = x; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
      if (before(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if ((tid & 31) == 0) { s_v[tid >> 5] = bv; s_i[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < kThreads / 32; ++w)
        if (before(s_v[w], s_i[w], bv, bi)) { bv = s_v[w]; bi = s_i[w]; }
      s_last_v = bv;
      s_last_i = bi;
      ids[(int64_t)r * k_top + t] = (bi == INT_MAX) ? -1 : bi;
      vals[(int64_t)r * k_top + t] = bv;
    }
    __syncthreads();
    last_v = s_last_v;
    last_i = s_last_i;
    if (last_i == INT_MAX) last_v = -INFINITY;
  }
}

template <class K, class... A>
cudaError_t launch_rows(K kernel, dim3 grid, cudaStream_t stream, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

// scratch layout (after the workspace's fixed part): x bf16 [R,H] | q, k, v fp32 [S1][R,H] each |
// cat bf16 [R,2H] | p fp32 [S2][R,H] | y bf16 [R,H] | logits fp32 [R, ldl]   (S1, S2: parts of the K axis)
size_t draft_head_scratch_bytes(int rows, int hidden, int vocab) {
  const size_t R = rows, H = hidden, ldl = (vocab + 7) / 8 * 8;
  const size_t s1 = rows_linear_splits(rows, hidden, hidden), s2 = rows_linear_splits(rows, 2 * hidden, hidden);
  return up256(R * H * 2) + 3 * up256(s1 * R * H * 4) + up256(R * 2 * H * 2) + up256(s2 * R * H * 4) +
         up256(R * H * 2) + up256(R * ldl * 4);
}

cudaError_t launch_draft_head_step(const clv_draft_head& w, int rows, const void* h, const void* e, int k_top,
                                   void* hidden_out, int32_t* top_ids, float* top_logits, int32_t* status,
                                   unsigned* tickets, void* scratch, cudaStream_t stream) {
  const int H = w.hidden_dim, V = w.vocab;
  const size_t R = rows, ldl = (V + 7) / 8 * 8;
  const int s1 = rows_linear_splits(rows, H, H), s2 = rows_linear_splits(rows, 2 * H, H);
  const int64_t part = (int64_t)R * H;   // elements between the parts of a product
  char* s = static_cast<char*>(scratch);
  uint16_t* x = reinterpret_cast<uint16_t*>(s); s += up256(R * H * 2);
  float* q = reinterpret_cast<float*>(s); s += up256(s1 * R * H * 4);
  float* k = reinterpret_cast<float*>(s); s += up256(s1 * R * H * 4);
  float* v = reinterpret_cast<float*>(s); s += up256(s1 * R * H * 4);
  uint16_t* cat = reinterpret_cast<uint16_t*>(s); s += up256(R * 2 * H * 2);
  float* p = reinterpret_cast<float*>(s); s += up256(s2 * R * H * 4);
  uint16_t* y = reinterpret_cast<uint16_t*>(s); s += up256(R * H * 2);
  float* logits = reinterpret_cast<float*>(s);
  const uint16_t* h16 = static_cast<const uint16_t*>(h);
  const uint16_t* e16 = static_cast<const uint16_t*>(e);
  cudaError_t err;
#define CLV_TRY(call) if ((err = (call)) != cudaSuccess) return err
  // status words: one per product (a wait of the GEMM kernel that ran out)
  CLV_TRY(launch_rows(rmsnorm_rows_kernel, dim3((unsigned)rows), stream, H, h16, (const float*)nullptr, 1, (int64_t)0,
                      static_cast<const uint16_t*>(w.norm1), w.rms_eps, x, (uint16_t*)nullptr));
  CLV_TRY(launch_rows_linear(x, H, w.wq, H, w.bq, rows, H, H, q, H, s1, part, status + 0, tickets, stream));
  CLV_TRY(launch_rows_linear(e16, H, w.wk, H, w.bk, rows, H, H, k, H, s1, part, status + 1, tickets, stream));
  CLV_TRY(launch_rows_linear(e16, H, w.wv, H, w.bv, rows, H, H, v, H, s1, part, status + 2, tickets, stream));
  CLV_TRY(launch_rows(gate_residual_kernel, dim3((unsigned)rows, (unsigned)((w.n_heads + 7) / 8)), stream, H,
                      (int)w.n_heads, (const float*)q, (const float*)k, (const float*)v, s1, part, h16, e16, cat));
  CLV_TRY(launch_rows_linear(cat, 2 * H, w.wfc, 2 * H, w.bfc, rows, 2 * H, H, p, H, s2, part, status + 3, tickets, stream));
  CLV_TRY(launch_rows(rmsnorm_rows_kernel, dim3((unsigned)rows), stream, H, (const uint16_t*)nullptr, (const float*)p,
                      s2, part, static_cast<const uint16_t*>(w.norm2), w.rms_eps, y, static_cast<uint16_t*>(hidden_out)));
  CLV_TRY(launch_rows_linear(y, H, w.lm_head, H, nullptr, rows, H, V, logits, (int64_t)ldl, 1, 0, status + 4, tickets,
                             stream));
  CLV_TRY(launch_rows(topk_rows_kernel, dim3((unsigned)rows), stream, V, (int64_t)ldl, k_top, (const float*)logits,
                      top_ids, top_logits));
#undef CLV_TRY
  return cudaSuccess;
}

}  // namespace clv
