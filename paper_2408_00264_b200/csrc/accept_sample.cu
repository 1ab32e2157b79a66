// Stochastic acceptance at temperature T > 0 (Sec. 4.1 / 4.2, Table 1 lower half: the paper adopts
// its baseline's tree sampling algorithm and prints no formula; taken here as speculative sampling
// for drafts that are proposed deterministically, one token per child).
//
// At the current node the target's distribution is p = softmax(logits / T).  The children are
// tried in increasing node index: child c with token x is accepted if
//   u[c] < p(x) / (1 - mass of the tokens rejected at this node so far);
// a rejected token is struck from the distribution; when every child is rejected (or there is
// none) the next token is the first v, in vocabulary order and not struck, whose running sum of p
// exceeds u[N] * (what is left).  The uniforms are the caller's.
//
// Two launches.  (1) One pass over all logits (an HBM stream like the argmax): every block
// reduces a piece of a row to (maximum, sum of exponentials relative to it) with an online
// update, in base-2 units.  (2) One block per sequence walks the tree: per level it combines the
// pieces of the current row, fetches the logits of all children's tokens at once (one round trip
// to memory), and one thread runs the accept chain; the final draw sums 256 slices of the row,
// locates the slice by a running sum and then scans that slice with the whole block.
#include <limits.h>
#include <math.h>

#include "clv_internal.cuh"

namespace clv {
namespace {

constexpr int kThreads = 256;
constexpr int kPiece = 32768;   // logits per block of the statistics pass (64 KB)
constexpr int kUnroll = 8;

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// (m, s): s = sum of 2^(x - m) over the values seen so far, m their maximum (s = 0 while m = -inf)
struct Stat {
  float m, s;
};
__device__ __forceinline__ void stat_merge(Stat& a, const Stat& b) {
  const float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return;   // both empty
  a.s = a.s * ex2(a.m - m) + b.s * ex2(b.m - m);   // 2^(-inf) = 0 for an empty side
  a.m = m;
}
__device__ __forceinline__ void stat_take8(Stat& st, const uint4& w, float k) {
  float x[8] = {bf16_lo(w.x) * k, bf16_hi(w.x) * k, bf16_lo(w.y) * k, bf16_hi(w.y) * k,
                bf16_lo(w.z) * k, bf16_hi(w.z) * k, bf16_lo(w.w) * k, bf16_hi(w.w) * k};
  float mx = x[0];
#pragma unroll
  for (int j = 1; j < 8; ++j) mx = fmaxf(mx, x[j]);   // NaN operands are dropped
  if (!(mx > -INFINITY)) return;                        // nothing but -inf (or NaN): no mass
  if (mx > st.m) { st.s *= ex2(st.m - mx); st.m = mx; }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float e = ex2(x[j] - st.m);
    st.s += (x[j] == x[j]) ? e : 0.f;                   // a NaN logit carries no mass
  }
}

struct StatParams {
  const uint16_t* logits;
  int64_t ld;
  int vocab, pieces;
  float k;           // log2(e) / T
  float2* partial;   // [rows][pieces]
};

__global__ void __launch_bounds__(kThreads) softmax_stats_kernel(StatParams p) {
  const int row = blockIdx.x / p.pieces;
  const int piece = blockIdx.x - row * p.pieces;
  const int begin = piece * kPiece;
  const int end = min(p.vocab, begin + kPiece);
  const uint16_t* base = p.logits + (int64_t)row * p.ld;
  const int nvec = (end - begin) >> 3;
  const uint4* vp = reinterpret_cast<const uint4*>(base + begin);
  const int tid = threadIdx.x;
  cudaGridDependencySynchronize();
  Stat st = {-INFINITY, 0.f};
  int i = tid;
  for (; i + (kUnroll - 1) * kThreads < nvec; i += kUnroll * kThreads) {
    uint4 w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) w[u] = ld_stream16(vp + i + u * kThreads);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) stat_take8(st, w[u], p.k);
  }
  for (; i < nvec; i += kThreads) stat_take8(st, ld_stream16(vp + i), p.k);
  {  // ragged end of the row: at most 7 scalars
    const int t0 = begin + 8 * nvec + tid;
    if (t0 < end) {
      const float x = __uint_as_float((uint32_t)base[t0] << 16) * p.k;
      if (x > -INFINITY) { Stat one = {x, 1.f}; stat_merge(st, one); }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Stat other = {__shfl_xor_sync(0xFFFFFFFFu, st.m, o), __shfl_xor_sync(0xFFFFFFFFu, st.s, o)};
    stat_merge(st, other);
  }
  __shared__ float sm[kThreads / 32], ss[kThreads / 32];
  if ((tid & 31) == 0) { sm[tid >> 5] = st.m; ss[tid >> 5] = st.s; }
  __syncthreads();
  if (tid != 0) return;
  for (int w = 1; w < kThreads / 32; ++w) { Stat other = {sm[w], ss[w]}; stat_merge(st, other); }
  p.partial[(int64_t)row * p.pieces + piece] = make_float2(st.m, st.s);
}

struct WalkParams {
  const uint16_t* logits;
  int64_t ld;
  int vocab, pieces, N, path_cap;
  float k;
  const float2* partial;
  const int32_t* parent;
  const int32_t* tokens;
  const float* uniforms;   // [B][N + 1]
  int32_t* accept_len;
  int32_t* accept_idx;
  int32_t* next_token;
  int32_t* status;
};

__global__ void __launch_bounds__(kThreads) sample_walk_kernel(WalkParams p) {
  __shared__ int sp[CLV_MAX_NODES], st[CLV_MAX_NODES], path[CLV_MAX_NODES];
  __shared__ float su[CLV_MAX_NODES + 1], se[CLV_MAX_NODES];
  __shared__ float s_slice[kThreads];
  __shared__ float s_m, s_S, s_before, s_target;
  __shared__ int s_found, s_bad, s_pick, s_lastv;
  const int b = blockIdx.x, tid = threadIdx.x, N = p.N;
  const int64_t o = (int64_t)b * N;
  cudaGridDependencySynchronize();
  if (tid == 0) s_bad = (p.path_cap < 1) ? 1 : 0;
  __syncthreads();
  for (int i = tid; i < N; i += kThreads) {
    const int par = p.parent[o + i];
    sp[i] = par;
    st[i] = p.tokens[o + i];
    if ((i == 0) ? (par != -1) : (par < 0 || par >= i)) s_bad = 1;   // node 0 is the only root
  }
  for (int i = tid; i <= N; i += kThreads) su[i] = p.uniforms[(int64_t)b * (N + 1) + i];
  __syncthreads();
  int len = 1, cur = 0;
  bool bad = s_bad != 0;
  if (tid == 0) path[0] = 0;
  while (!bad) {
    // ---- the current row's maximum and sum from its pieces
    if (tid < 32) {
      Stat a = {-INFINITY, 0.f};
      for (int i = tid; i < p.pieces; i += 32) {
        const float2 v = p.partial[(o + cur) * p.pieces + i];
        Stat other = {v.x, v.y};
        stat_merge(a, other);
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        Stat other = {__shfl_xor_sync(0xFFFFFFFFu, a.m, off), __shfl_xor_sync(0xFFFFFFFFu, a.s, off)};
        stat_merge(a, other);
      }
      if (tid == 0) { s_m = a.m; s_S = a.s; }
    }
    __syncthreads();
    const float m = s_m, S = s_S;
    // ---- the weights 2^(x - m) of all children's tokens, fetched together
    const uint16_t* row = p.logits + (o + cur) * p.ld;
    for (int c = cur + 1 + tid; c < N; c += kThreads) {
      float e = 0.f;
      if (sp[c] == cur) {
        const int x = st[c];
        if (x >= 0 && x < p.vocab && m > -INFINITY) {
          const float l = __uint_as_float((uint32_t)row[x] << 16) * p.k;
          e = (l == l) ? ex2(l - m) : 0.f;
        }
      }
      se[c] = e;
    }
    __syncthreads();
    if (tid == 0) {   // the accept chain, in node order
      float rej = 0.f;
      int found = -1;
      for (int c = cur + 1; c < N; ++c) {
        if (sp[c] != cur) continue;
        float e = se[c];
        for (int d = cur + 1; d < c; ++d)   // a token that was struck already carries nothing
          if (sp[d] == cur && st[d] == st[c]) e = 0.f;
        const float left = S - rej;
        const float a = (left > 0.f) ? e / left : 0.f;
        if (su[c] < a) { found = c; break; }
        rej += e;
      }
      s_found = found;
    }
    __syncthreads();
    const int found = s_found;
    if (found < 0) break;
    if (len == p.path_cap || len == CLV_MAX_NODES) { bad = true; break; }
    if (tid == 0) path[len] = found;
    ++len;
    cur = found;
    __syncthreads();   // se[] and the scalars are rewritten on the next level
  }
  if (!bad) {
    // ---- draw the next token from what is left of row `cur`: all of its children were rejected,
    //      their tokens are struck.  256 slices of the row, each a multiple of 8 logits.
    const float m = s_m;
    const uint16_t* row = p.logits + (o + cur) * p.ld;
    const int per = ((p.vocab + kThreads - 1) / kThreads + 7) & ~7;
    const int v0 = min(p.vocab, tid * per), v1 = min(p.vocab, v0 + per);
    auto weight = [&](int v) -> float {
      const float l = __uint_as_float((uint32_t)row[v] << 16) * p.k;
      return (l == l && m > -INFINITY) ? ex2(l - m) : 0.f;
    };
    // the slice's sum with 16-byte reads, four in flight (v0 is a multiple of 8, rows are 16-byte
    // aligned); the weights of struck tokens inside the slice are taken out again afterwards
    float sum = 0.f;
    {
      int v = v0;
      for (; v + 32 <= v1; v += 32) {
        uint4 w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) w[q] = *reinterpret_cast<const uint4*>(row + v + 8 * q);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float x[8] = {bf16_lo(w[q].x), bf16_hi(w[q].x), bf16_lo(w[q].y), bf16_hi(w[q].y),
                              bf16_lo(w[q].z), bf16_hi(w[q].z), bf16_lo(w[q].w), bf16_hi(w[q].w)};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float l = x[j] * p.k;
            sum += (l == l && m > -INFINITY) ? ex2(l - m) : 0.f;
          }
        }
      }
      for (; v < v1; ++v) sum += weight(v);
      for (int c = cur + 1; c < N; ++c) {
        if (sp[c] != cur || st[c] < v0 || st[c] >= v1) continue;
        bool repeat = false;   // a token carried by two siblings is struck once
        for (int d = cur + 1; d < c; ++d) repeat |= (sp[d] == cur && st[d] == st[c]);
        if (!repeat) sum -= weight(st[c]);
      }
      sum = fmaxf(sum, 0.f);
    }
    s_slice[tid] = sum;
    __syncthreads();
    if (tid == 0) {
      // what is left, by the sums of this pass (the first pass's sum minus the rejected weights
      // differs from it by rounding only)
      float total = 0.f;
      for (int j = 0; j < kThreads; ++j) total += s_slice[j];
      const float target = su[N] * total;
      float run = 0.f;
      int pick = -1, last = -1;
      for (int j = 0; j < kThreads; ++j) {
        if (s_slice[j] > 0.f) last = j;
        if (pick < 0 && s_slice[j] > 0.f && run + s_slice[j] > target) { pick = j; s_before = run; }
        if (pick < 0) run += s_slice[j];
      }
      if (pick < 0 && last >= 0) {   // rounding: the target lies at the very end
        pick = last;
        s_before = total - s_slice[last];
      }
      s_pick = pick;
      s_target = target;
      s_found = INT_MAX;   // first element of the slice whose running sum exceeds the target
      s_lastv = -1;        // last element of the slice that carries any weight
    }
    __syncthreads();
    const int pick = s_pick;
    if (pick >= 0) {
      // ---- the whole block walks the chosen slice, 256 elements at a time: weights, a running sum
      //      across the block (warp scans + the warps' totals), the first element past the target
      const float target = s_target;
      const int q0 = min(p.vocab, pick * per), q1 = min(p.vocab, q0 + per);
      const int lane = tid & 31, warp = tid >> 5;
      float before = s_before;
      for (int base = q0; base < q1; base += kThreads) {
        const int v = base + tid;
        float e = 0.f;
        if (v < q1) {
          bool hit = false;
          for (int c = cur + 1; c < N; ++c) hit |= (sp[c] == cur && st[c] == v);
          e = hit ? 0.f : weight(v);
        }
        float incl = e;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const float up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
          if (lane >= off) incl += up;
        }
        if (lane == 31) s_slice[warp] = incl;
        __syncthreads();
        float wbase = before;
        for (int w = 0; w < warp; ++w) wbase += s_slice[w];
        float round_total = 0.f;
        for (int w = 0; w < kThreads / 32; ++w) round_total += s_slice[w];
        if (e > 0.f) {
          atomicMax(&s_lastv, v);
          if (wbase + incl > target) atomicMin(&s_found, v);
        }
        __syncthreads();
        if (s_found != INT_MAX) break;   // same verdict in every thread
        before += round_total;
      }
      if (tid == 0) p.next_token[b] = (s_found != INT_MAX) ? s_found : s_lastv;
    } else if (tid == 0) {
      p.next_token[b] = -1;   // a row without any mass
    }
  }
  __syncthreads();
  if (bad) len = 0;
  for (int j = tid; j < p.path_cap; j += kThreads)
    p.accept_idx[(int64_t)b * p.path_cap + j] = (j < len) ? path[j] : -1;
  if (tid == 0) {
    p.accept_len[b] = len;
    if (bad) p.next_token[b] = -1;
    p.status[b] = bad ? CLV_ERR_TREE : CLV_OK;
  }
}

int sample_pieces(int vocab) { return (vocab + kPiece - 1) / kPiece; }

}  // namespace

size_t sample_scratch_bytes(int rows, int vocab) { return sizeof(float2) * (size_t)rows * sample_pieces(vocab); }

cudaError_t launch_accept_sample(const clv_shape& s, const void* logits, int64_t ld, const int32_t* parent,
                                 const int32_t* tokens, const float* uniforms, float temperature,
                                 int32_t* accept_len, int32_t* accept_idx, int32_t* next_token, int32_t* status,
                                 void* scratch, cudaStream_t stream) {
  const int rows = s.batch * s.n_nodes;
  const float k = 1.4426950408889634f / temperature;
  StatParams a;
  a.logits = static_cast<const uint16_t*>(logits);
  a.ld = ld;
  a.vocab = s.vocab;
  a.pieces = sample_pieces(s.vocab);
  a.k = k;
  a.partial = static_cast<float2*>(scratch);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((int64_t)rows * a.pieces), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, softmax_stats_kernel, a);
  if (e != cudaSuccess) return e;
  WalkParams w;
  w.logits = a.logits;
  w.ld = ld;
  w.vocab = s.vocab;
  w.pieces = a.pieces;
  w.N = s.n_nodes;
  w.path_cap = s.path_cap;
  w.k = k;
  w.partial = a.partial;
  w.parent = parent;
  w.tokens = tokens;
  w.uniforms = uniforms;
  w.accept_len = accept_len;
  w.accept_idx = accept_idx;
  w.next_token = next_token;
  w.status = status;
  cfg.gridDim = dim3((unsigned)s.batch, 1, 1);
  return cudaLaunchKernelEx(&cfg, sample_walk_kernel, w);
}

}  // namespace clv
