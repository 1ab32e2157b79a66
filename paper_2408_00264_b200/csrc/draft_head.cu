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

constexpr int kThreads = 256;       // gate and top-k kernels
constexpr int kNormThreads = 512;
constexpr int kNormCache = 4;       // groups of 4 elements a thread keeps between the two passes

__device__ __forceinline__ float bf16f(uint32_t b) { return __uint_as_float(b << 16); }
__device__ __forceinline__ uint32_t f2bf(float x) {
  const __nv_bfloat16 v = __float2bfloat16_rn(x);
  return (uint32_t)*reinterpret_cast<const uint16_t*>(&v);
}
__device__ __forceinline__ float4 bf16x4(uint2 b) {
  return make_float4(__uint_as_float(b.x << 16), __uint_as_float(b.x & 0xFFFF0000u), __uint_as_float(b.y << 16),
                     __uint_as_float(b.y & 0xFFFF0000u));
}
__device__ __forceinline__ uint2 to_bf16x4(float4 v) {
  return make_uint2(f2bf(v.x) | (f2bf(v.y) << 16), f2bf(v.z) | (f2bf(v.w) << 16));
}

// four neighbouring elements of a product whose K axis was cut in `parts` parts (up to 8): the
// parts added up in their order
__device__ __forceinline__ float4 sum_parts4(const float* x, int64_t i, int parts, int64_t stride) {
  float4 p[8];
#pragma unroll
  for (int s = 0; s < 8; ++s)
    if (s < parts) p[s] = *reinterpret_cast<const float4*>(x + i + s * stride);
  float4 v = p[0];
#pragma unroll
  for (int s = 1; s < 8; ++s)
    if (s < parts) { v.x += p[s].x; v.y += p[s].y; v.z += p[s].z; v.w += p[s].w; }
  return v;
}

// y = RMSNorm(x; gain) rounded to bf16; x is bf16 (x32 == NULL) or fp32 in `parts` parts.
// Optionally also x itself rounded to bf16 (the head's hidden state, handed to the next head).
// One block per row; a thread keeps its first 16 elements in registers between the two passes
// (hidden sizes up to 8192 are read once), later ones are read again.
__global__ void __launch_bounds__(kNormThreads) rmsnorm_rows_kernel(int H, const uint16_t* x16, const float* x32,
                                                                    int parts, int64_t stride, const uint16_t* gain,
                                                                    float eps, uint16_t* y, uint16_t* x_out) {
  __shared__ float s_red[kNormThreads / 32];
  const int r = blockIdx.x, tid = threadIdx.x, n4 = H / 4;
  const int64_t row = (int64_t)r * H;
  cudaGridDependencySynchronize();
  auto load = [&](int i) {
    return x32 ? sum_parts4(x32, row + 4 * (int64_t)i, parts, stride)
               : bf16x4(*reinterpret_cast<const uint2*>(x16 + row + 4 * (int64_t)i));
  };
  float4 c[kNormCache];
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < kNormCache; ++j) {
    const int i = tid + j * kNormThreads;
    if (i < n4) {
      c[j] = load(i);
      ss += c[j].x * c[j].x + c[j].y * c[j].y + c[j].z * c[j].z + c[j].w * c[j].w;
    }
  }
  for (int i = tid + kNormCache * kNormThreads; i < n4; i += kNormThreads) {
    const float4 v = load(i);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  if ((tid & 31) == 0) s_red[tid >> 5] = ss;
  __syncthreads();
  float total = 0.f;
  for (int w = 0; w < kNormThreads / 32; ++w) total += s_red[w];
  const float inv = rsqrtf(total / (float)H + eps);
  auto emit = [&](int i, float4 v) {
    const float4 g = bf16x4(*reinterpret_cast<const uint2*>(gain + 4 * (int64_t)i));
    *reinterpret_cast<uint2*>(y + row + 4 * (int64_t)i) =
        to_bf16x4(make_float4(v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w));
    if (x_out) *reinterpret_cast<uint2*>(x_out + row + 4 * (int64_t)i) = to_bf16x4(v);
  };
#pragma unroll
  for (int j = 0; j < kNormCache; ++j) {
    const int i = tid + j * kNormThreads;
    if (i < n4) emit(i, c[j]);
  }
  for (int i = tid + kNormCache * kNormThreads; i < n4; i += kNormThreads) emit(i, load(i));
}

// a = h + v * gate (per head: cosine of q and k), written with e behind it: cat[r] = [a, e] (bf16).
// One warp per head, eight heads per block; q, k, v arrive in `parts` parts; a lane takes four
// neighbouring elements at a time (the head size is a multiple of 4).
__global__ void __launch_bounds__(kThreads) gate_residual_kernel(int H, int n_heads, const float* q, const float* k,
                                                                 const float* v, int parts, int64_t stride,
                                                                 const uint16_t* h, const uint16_t* e, uint16_t* cat) {
  const int r = blockIdx.x, hd = H / n_heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.y * (kThreads / 32) + warp;
  cudaGridDependencySynchronize();
  if (j >= n_heads) return;
  const int64_t o = (int64_t)r * H + (int64_t)j * hd;
  float qk = 0.f, qq = 0.f, kk = 0.f;
  for (int i = 4 * lane; i < hd; i += 128) {
    const float4 a = sum_parts4(q, o + i, parts, stride), b = sum_parts4(k, o + i, parts, stride);
    qk += a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w;
    qq += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
    kk += b.x * b.x + b.y * b.y + b.z * b.z + b.w * b.w;
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    qk += __shfl_xor_sync(0xFFFFFFFFu, qk, s);
    qq += __shfl_xor_sync(0xFFFFFFFFu, qq, s);
    kk += __shfl_xor_sync(0xFFFFFFFFu, kk, s);
  }
  const float gate = qk / fmaxf(sqrtf(qq) * sqrtf(kk), 1e-8f);
  uint16_t* dst = cat + (int64_t)r * 2 * H + (int64_t)j * hd;
  for (int i = 4 * lane; i < hd; i += 128) {
    const float4 hv = bf16x4(*reinterpret_cast<const uint2*>(h + o + i));
    const float4 vv = sum_parts4(v, o + i, parts, stride);
    *reinterpret_cast<uint2*>(dst + i) =
        to_bf16x4(make_float4(hv.x + vv.x * gate, hv.y + vv.y * gate, hv.z + vv.z * gate, hv.w + vv.w * gate));
    *reinterpret_cast<uint2*>(dst + H + i) = *reinterpret_cast<const uint2*>(e + o + i);
  }
}

// ---- the k largest of a row: highest first, lower index first among equals ----------------------
// A row is cut in slices of 2048 entries, one block each: a thread sorts its 8 entries, each warp
// picks the k best of its 256 (k rounds of a shuffle argmax over the lanes' current best; the
// winning lane moves on to its next), warp 0 picks the k best of the 8 warps' picks.  The
// slices' picks (value, index) are the entries of the next level, until one slice is left.
constexpr int kSliceLen = 2048, kPerThread = kSliceLen / kThreads, kListK = 32;
static_assert(kPerThread == 8 && (kThreads / 32) * kListK <= 32 * kPerThread, "warp 0 holds all warps' picks");

__device__ __forceinline__ bool before(float v, int i, float bv, int bi) {   // order: value desc, index asc
  return (v > bv) || (v == bv && i < bi);
}
__device__ __forceinline__ void sort8(float (&v)[kPerThread], int (&ix)[kPerThread]) {
#pragma unroll
  for (int a = 1; a < kPerThread; ++a)
#pragma unroll
    for (int b = a; b > 0; --b)
      if (before(v[b], ix[b], v[b - 1], ix[b - 1])) {
        const float tv = v[b]; v[b] = v[b - 1]; v[b - 1] = tv;
        const int ti = ix[b]; ix[b] = ix[b - 1]; ix[b - 1] = ti;
      }
}
// the k best of the warp's sorted lists, in order, to out_v / out_i (absent entries: -inf, INT_MAX)
__device__ __forceinline__ void warp_select(float (&v)[kPerThread], int (&ix)[kPerThread], int k, float* out_v,
                                            int* out_i) {
  const int lane = threadIdx.x & 31;
  for (int t = 0; t < k; ++t) {
    float bv = v[0];
    int bi = ix[0];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
      if (before(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { out_v[t] = bv; out_i[t] = bi; }
    if (bi != INT_MAX && ix[0] == bi) {   // indices are distinct: this lane won
#pragma unroll
      for (int u = 0; u + 1 < kPerThread; ++u) { v[u] = v[u + 1]; ix[u] = ix[u + 1]; }
      v[kPerThread - 1] = -INFINITY;
      ix[kPerThread - 1] = INT_MAX;
    }
  }
}

// in_i == NULL: the entries' indices are their positions.  last: results go to ids / vals as the
// caller wants them (-1 for an absent entry); otherwise out_v / out_i [rows, out_stride] get k per slice.
__global__ void __launch_bounds__(kThreads) topk_slices_kernel(int n, int64_t ld, const float* in_v, const int* in_i,
                                                               int k, float* out_v, int* out_i, int64_t out_stride,
                                                               int last) {
  __shared__ float s_v[(kThreads / 32) * kListK];
  __shared__ int s_i[(kThreads / 32) * kListK];
  const int r = blockIdx.x, slice = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  cudaGridDependencySynchronize();
  float v[kPerThread];
  int ix[kPerThread];
  {
    const int j0 = slice * kSliceLen + tid * kPerThread;
    const int64_t at = (int64_t)r * ld + j0;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    int4 ia = make_int4(0, 0, 0, 0), ib = ia;
    if (j0 < n) {   // rows are padded to a multiple of 8 entries: the loads stay inside
      a = *reinterpret_cast<const float4*>(in_v + at);
      b = *reinterpret_cast<const float4*>(in_v + at + 4);
      if (in_i) {
        ia = *reinterpret_cast<const int4*>(in_i + at);
        ib = *reinterpret_cast<const int4*>(in_i + at + 4);
      }
    }
    const float lv[kPerThread] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    const int li[kPerThread] = {ia.x, ia.y, ia.z, ia.w, ib.x, ib.y, ib.z, ib.w};
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
      const bool have = j0 + u < n && (!in_i || li[u] != INT_MAX);
      float x = lv[u];
      if (x != x) x = -INFINITY;   // NaN: after everything else
      v[u] = have ? x : -INFINITY;
      ix[u] = have ? (in_i ? li[u] : j0 + u) : INT_MAX;
    }
  }
  sort8(v, ix);
  warp_select(v, ix, k, s_v + warp * k, s_i + warp * k);
  __syncthreads();
  if (warp != 0) return;
  const int have = (kThreads / 32) * k;
#pragma unroll
  for (int u = 0; u < kPerThread; ++u) {
    const int j = lane * kPerThread + u;
    v[u] = j < have ? s_v[j] : -INFINITY;
    ix[u] = j < have ? s_i[j] : INT_MAX;
  }
  sort8(v, ix);
  float* ov = out_v + (int64_t)r * out_stride + (last ? 0 : slice * k);
  int* oi = out_i + (int64_t)r * out_stride + (last ? 0 : slice * k);
  warp_select(v, ix, k, ov, oi);
  __syncwarp();
  if (last)
    for (int t = lane; t < k; t += 32)
      if (oi[t] == INT_MAX) oi[t] = -1;
}

// More than 32 per row: k passes over the row (it stays in L2), each taking the best of what
// comes after the previous pass's pick.
__global__ void __launch_bounds__(kThreads) topk_passes_kernel(int V, int64_t ld, int k_top, const float* logits,
                                                               int32_t* ids, float* vals) {
  __shared__ float s_v[kThreads / 32];
  __shared__ int s_i[kThreads / 32];
  __shared__ float s_last_v;
  __shared__ int s_last_i;
  const int r = blockIdx.x, tid = threadIdx.x;
  const float* row = logits + (int64_t)r * ld;
  cudaGridDependencySynchronize();
  float last_v = INFINITY;
  int last_i = -1;
  for (int t = 0; t < k_top; ++t) {
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
cudaError_t launch_rows(K kernel, dim3 grid, int threads, cudaStream_t stream, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

// top-k candidates one level leaves per row (a multiple of 8, so that rows stay 32-byte aligned)
size_t topk_candidates(int vocab, int k_top) {
  const size_t slices = ((size_t)vocab + kSliceLen - 1) / kSliceLen;
  return (slices * (size_t)(k_top < kListK ? k_top : kListK) + 7) / 8 * 8;
}

}  // namespace

// scratch layout (after the workspace's fixed part): x bf16 [R,H] | q, k, v fp32 [S1][R,H] each |
// cat bf16 [R,2H] | p fp32 [S2][R,H] | y bf16 [R,H] | logits fp32 [R, ldl] | two levels of top-k
// candidates, values then indices [R, cand] each   (S1, S2: parts of the K axis)
size_t draft_head_scratch_bytes(int rows, int hidden, int vocab) {
  const size_t R = rows, H = hidden, ldl = (vocab + 7) / 8 * 8;
  const size_t s1 = rows_linear_splits(rows, hidden, hidden, 3), s2 = rows_linear_splits(rows, 2 * hidden, hidden, 1);
  return up256(R * H * 2) + 3 * up256(s1 * R * H * 4) + up256(R * 2 * H * 2) + up256(s2 * R * H * 4) +
         up256(R * H * 2) + up256(R * ldl * 4) + 4 * up256(R * topk_candidates(vocab, kListK) * 4);
}

cudaError_t launch_draft_head_step(const clv_draft_head& w, int rows, const void* h, const void* e, int k_top,
                                   void* hidden_out, int32_t* top_ids, float* top_logits, int32_t* status,
                                   unsigned* tickets, void* scratch, cudaStream_t stream) {
  const int H = w.hidden_dim, V = w.vocab;
  const size_t R = rows, ldl = (V + 7) / 8 * 8;
  const int s1 = rows_linear_splits(rows, H, H, 3), s2 = rows_linear_splits(rows, 2 * H, H, 1);
  const int64_t part = (int64_t)R * H;   // elements between the parts of a product
  const size_t cand = topk_candidates(V, kListK);
  char* s = static_cast<char*>(scratch);
  uint16_t* x = reinterpret_cast<uint16_t*>(s); s += up256(R * H * 2);
  float* q = reinterpret_cast<float*>(s); s += up256(s1 * R * H * 4);
  float* k = reinterpret_cast<float*>(s); s += up256(s1 * R * H * 4);
  float* v = reinterpret_cast<float*>(s); s += up256(s1 * R * H * 4);
  uint16_t* cat = reinterpret_cast<uint16_t*>(s); s += up256(R * 2 * H * 2);
  float* p = reinterpret_cast<float*>(s); s += up256(s2 * R * H * 4);
  uint16_t* y = reinterpret_cast<uint16_t*>(s); s += up256(R * H * 2);
  float* logits = reinterpret_cast<float*>(s); s += up256(R * ldl * 4);
  float* cand_v[2];
  int* cand_i[2];
  for (int b = 0; b < 2; ++b) {
    cand_v[b] = reinterpret_cast<float*>(s); s += up256(R * cand * 4);
    cand_i[b] = reinterpret_cast<int*>(s); s += up256(R * cand * 4);
  }
  const uint16_t* h16 = static_cast<const uint16_t*>(h);
  const uint16_t* e16 = static_cast<const uint16_t*>(e);
  const dim3 per_row((unsigned)rows);
  cudaError_t err;
#define CLV_TRY(call) if ((err = (call)) != cudaSuccess) return err
  // status words: one per product (a wait of the GEMM kernel that ran out)
  CLV_TRY(launch_rows(rmsnorm_rows_kernel, per_row, kNormThreads, stream, H, h16, (const float*)nullptr, 1, (int64_t)0,
                      static_cast<const uint16_t*>(w.norm1), w.rms_eps, x, (uint16_t*)nullptr));
  {   // q = x wq^T + bq, k = e wk^T + bk, v = e wv^T + bv: one launch
    const void* const xs[3] = {x, e16, e16};
    const void* const ws[3] = {w.wq, w.wk, w.wv};
    const void* const bs[3] = {w.bq, w.bk, w.bv};
    float* const outs[3] = {q, k, v};
    CLV_TRY(launch_rows_linear(3, xs, H, ws, H, bs, rows, H, H, outs, H, s1, part, status + 0, tickets, stream));
  }
  CLV_TRY(launch_rows(gate_residual_kernel, dim3((unsigned)rows, (unsigned)((w.n_heads + 7) / 8)), kThreads, stream, H,
                      (int)w.n_heads, (const float*)q, (const float*)k, (const float*)v, s1, part, h16, e16, cat));
  {
    const void* const xs[1] = {cat};
    const void* const bs[1] = {w.bfc};
    float* const outs[1] = {p};
    CLV_TRY(launch_rows_linear(1, xs, 2 * H, &w.wfc, 2 * H, bs, rows, 2 * H, H, outs, H, s2, part, status + 3, tickets,
                               stream));
  }
  CLV_TRY(launch_rows(rmsnorm_rows_kernel, per_row, kNormThreads, stream, H, (const uint16_t*)nullptr, (const float*)p,
                      s2, part, static_cast<const uint16_t*>(w.norm2), w.rms_eps, y, static_cast<uint16_t*>(hidden_out)));
  {
    const void* const xs[1] = {y};
    const void* const bs[1] = {nullptr};
    float* const outs[1] = {logits};
    CLV_TRY(launch_rows_linear(1, xs, H, &w.lm_head, H, bs, rows, H, V, outs, (int64_t)ldl, 1, 0, status + 4, tickets,
                               stream));
  }
  if (k_top > kListK) {
    CLV_TRY(launch_rows(topk_passes_kernel, per_row, kThreads, stream, V, (int64_t)ldl, k_top, (const float*)logits,
                        top_ids, top_logits));
  } else {
    int n = V, level = 0;
    int64_t ld = (int64_t)ldl;
    const float* in_v = logits;
    const int* in_i = nullptr;
    for (;; ++level) {
      const int slices = (n + kSliceLen - 1) / kSliceLen;
      const int last = slices == 1;
      float* out_v = last ? top_logits : cand_v[level & 1];
      int* out_i = last ? top_ids : cand_i[level & 1];
      CLV_TRY(launch_rows(topk_slices_kernel, dim3((unsigned)rows, (unsigned)slices), kThreads, stream, n, ld, in_v, in_i,
                          k_top, out_v, out_i, last ? (int64_t)k_top : (int64_t)cand, last));
      if (last) break;
      n = slices * k_top;
      ld = (int64_t)cand;
      in_v = out_v;
      in_i = out_i;
    }
  }
#undef CLV_TRY
  return cudaSuccess;
}

}  // namespace clv
