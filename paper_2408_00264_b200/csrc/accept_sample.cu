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
// Two launches.  (1) One pass over all logits (an HBM stream like the argmax): every warp
// reduces a slice of 4096 consecutive logits of a row to (maximum, sum of exponentials relative
// to it) with an online update, in base-2 units.  (2) One block per sequence walks the tree: per
// level it combines the slices of the current row, fetches the logits of all children's tokens
// at once (one round trip to memory), and one thread runs the accept chain; the final draw
// locates the slice by a running sum over the slices' weights (the weights of struck tokens
// taken out) and then scans that one slice with the whole block, 16 logits per thread.
#include <limits.h>
#include <math.h>

#include "clv_internal.cuh"

namespace clv {
namespace {

constexpr int kThreads = 256;
constexpr int kPiece = 32768;   // logits per block of the statistics pass (64 KB)
constexpr int kUnroll = 8;
constexpr int kSlice = kPiece / (kThreads / 32);   // 4096 logits per warp: the unit of the running sums
constexpr int kPerThread = kSlice / kThreads;       // 16: what a thread scans of the chosen slice
static_assert(kSlice == 4096 && kPerThread == 16, "a slice is scanned in one round of the block");

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

// A batch of kUnroll vectors at once: one maximum and at most one rescale for the 64 values, then
// their exponentials into four running sums (no long chain of dependent additions).
__device__ __forceinline__ void stat_take_batch(Stat& st, const uint4 (&w)[kUnroll], float k) {
  float mx = -INFINITY;
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    const uint32_t r[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) mx = fmaxf(mx, fmaxf(bf16_lo(r[j]) * k, bf16_hi(r[j]) * k));   // NaN operands are dropped
  }
  if (!(mx > -INFINITY)) return;   // nothing but -inf (or NaN): no mass
  if (mx > st.m) { st.s *= ex2(st.m - mx); st.m = mx; }
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    const uint32_t r[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = bf16_lo(r[j]) * k, b = bf16_hi(r[j]) * k;
      acc[j] += ((a == a) ? ex2(a - st.m) : 0.f) + ((b == b) ? ex2(b - st.m) : 0.f);   // a NaN logit carries no mass
    }
  }
  st.s += (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

struct StatParams {
  const uint16_t* logits;
  int64_t ld;
  int vocab, pieces;
  float k;           // log2(e) / T
  float2* partial;   // [rows][pieces * 8]: one (maximum, sum) per slice
};

__global__ void __launch_bounds__(kThreads) softmax_stats_kernel(StatParams p) {
  const int row = blockIdx.x / p.pieces;
  const int piece = blockIdx.x - row * p.pieces;
  const int begin = piece * kPiece;
  const int end = min(p.vocab, begin + kPiece);
  const uint16_t* base = p.logits + (int64_t)row * p.ld;
  const int nvec = (end - begin) >> 3;
  const uint4* vp = reinterpret_cast<const uint4*>(base + begin);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  cudaGridDependencySynchronize();
  // warp w takes the vectors [512 w, 512 (w + 1)) of the piece: 4096 consecutive logits
  Stat st = {-INFINITY, 0.f};
  const int lim = min(nvec, (warp + 1) * (kSlice / 8));
  int i = warp * (kSlice / 8) + lane;
  for (; i + (kUnroll - 1) * 32 < lim; i += kUnroll * 32) {
    uint4 w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) w[u] = ld_stream16(vp + i + u * 32);
    stat_take_batch(st, w, p.k);
  }
  for (; i < lim; i += 32) stat_take8(st, ld_stream16(vp + i), p.k);
  {  // ragged end of the row: at most 7 scalars, taken by the warp whose slice holds them
    const int t0 = begin + 8 * nvec + lane;
    if (t0 < end && (t0 - begin) / kSlice == warp) {
      const float x = __uint_as_float((uint32_t)base[t0] << 16) * p.k;
      if (x > -INFINITY) { Stat one = {x, 1.f}; stat_merge(st, one); }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Stat other = {__shfl_xor_sync(0xFFFFFFFFu, st.m, o), __shfl_xor_sync(0xFFFFFFFFu, st.s, o)};
    stat_merge(st, other);
  }
  if (lane == 0) p.partial[((int64_t)row * p.pieces + piece) * (kThreads / 32) + warp] = make_float2(st.m, st.s);
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
  const int n_sl = p.pieces * (kPiece / kSlice);   // slices of a row
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
      for (int i = tid; i < n_sl; i += 32) {
        const float2 v = p.partial[(o + cur) * n_sl + i];
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
    //      their tokens are struck.  The slices' weights come from the statistics pass.
    const float m = s_m;
    const uint16_t* row = p.logits + (o + cur) * p.ld;
    auto weight = [&](int v) -> float {
      const float l = __uint_as_float((uint32_t)row[v] << 16) * p.k;
      return (l == l && m > -INFINITY) ? ex2(l - m) : 0.f;
    };
    // what is left, slice by slice (the first pass's sums minus the struck weights differ from a
    // fresh sum by rounding only); thread 0 walks the slices in vocabulary order
    for (int j = tid; j < n_sl; j += kThreads) {
      const float2 sl = p.partial[(o + cur) * n_sl + j];
      float sum = (sl.x > -INFINITY && m > -INFINITY) ? sl.y * ex2(sl.x - m) : 0.f;
      const int v0 = j * kSlice, v1 = min(p.vocab, v0 + kSlice);
      for (int c = cur + 1; c < N; ++c) {
        if (sp[c] != cur || st[c] < v0 || st[c] >= v1) continue;
        bool repeat = false;   // a token carried by two siblings is struck once
        for (int d = cur + 1; d < c; ++d) repeat |= (sp[d] == cur && st[d] == st[c]);
        if (!repeat) sum -= weight(st[c]);
      }
      sum = fmaxf(sum, 0.f);
      if (j < kThreads) s_slice[j] = sum;
    }
    __syncthreads();
    if (tid == 0) {
      const int n_here = n_sl;   // at most one slice per thread: larger vocabularies are refused by the host
      float total = 0.f;
      for (int j = 0; j < n_here; ++j) total += s_slice[j];
      const float target = su[N] * total;
      float run = 0.f;
      int pick = -1, last = -1;
      for (int j = 0; j < n_here; ++j) {
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
      // ---- the whole block scans the chosen slice in one round: a thread takes 16 consecutive
      //      logits (two 16-byte reads), strikes the children's tokens among them, adds them up;
      //      a running sum across the block (warp scan + the warps' totals) gives every thread
      //      its start, and the first element whose running sum exceeds the target wins
      const float target = s_target;
      const int q0 = pick * kSlice, q1 = min(p.vocab, q0 + kSlice);
      const int lane = tid & 31, warp = tid >> 5;
      const int v_base = q0 + tid * kPerThread;
      float e[kPerThread];
      {
        uint4 w[2];
#pragma unroll
        for (int h = 0; h < 2; ++h)   // past the row's end: the last vector again (cut by index below)
          w[h] = ld_stream16(row + min(v_base + 8 * h, (q1 - 1) & ~7));
        uint32_t struck = 0;
        for (int c = cur + 1; c < N; ++c)
          if (sp[c] == cur && st[c] >= v_base && st[c] < v_base + kPerThread) struck |= 1u << (st[c] - v_base);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float x[8] = {bf16_lo(w[h].x), bf16_hi(w[h].x), bf16_lo(w[h].y), bf16_hi(w[h].y),
                              bf16_lo(w[h].z), bf16_hi(w[h].z), bf16_lo(w[h].w), bf16_hi(w[h].w)};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float l = x[j] * p.k;
            const bool in = (v_base + 8 * h + j < q1) && !((struck >> (8 * h + j)) & 1u) && l == l && m > -INFINITY;
            e[8 * h + j] = in ? ex2(l - m) : 0.f;
          }
        }
      }
      float mine = 0.f;
#pragma unroll
      for (int j = 0; j < kPerThread; ++j) mine += e[j];
      float incl = mine;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const float up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += up;
      }
      if (lane == 31) s_slice[warp] = incl;
      __syncthreads();
      float run = s_before + (incl - mine);   // the running sum before this thread's first element
      for (int w = 0; w < warp; ++w) run += s_slice[w];
      int first = INT_MAX, lastv = -1;
#pragma unroll
      for (int j = 0; j < kPerThread; ++j) {
        run += e[j];
        if (e[j] > 0.f) {
          lastv = v_base + j;
          if (first == INT_MAX && run > target) first = v_base + j;
        }
      }
      if (lastv >= 0) atomicMax(&s_lastv, lastv);
      if (first != INT_MAX) atomicMin(&s_found, first);
      __syncthreads();
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

int sample_max_vocab() { return kThreads * kSlice; }   // one slice per thread of the walk's block

size_t sample_scratch_bytes(int rows, int vocab) {
  return sizeof(float2) * (size_t)rows * sample_pieces(vocab) * (kPiece / kSlice);
}

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
