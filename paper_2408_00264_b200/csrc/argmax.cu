// Per-node greedy choice: argmax over the vocabulary of each logits row (Sec. 4.2, T = 0).
//
// Pure HBM stream: every logit is read once with 16-byte loads that bypass L1.  A row is cut into
// `chunks` pieces so that the grid covers the machine even for few rows; each block reduces its
// piece to one (value, lowest index) pair, packs it into a 64-bit key whose unsigned order is
// "higher value first, then lower index", and the last block to arrive for a row takes the
// maximum key.  The result is independent of the chunking and of block scheduling.
#include <limits.h>

#include "clv_internal.cuh"

namespace clv {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 8;  // 16-byte loads in flight per thread (32 KB per block)

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t u) {
  return *reinterpret_cast<__nv_bfloat162*>(&u);
}

// Per-thread state: for each of the 8 positions inside a 16-byte vector, the running maximum (bf16)
// and the number of the visit at which it was first reached, both packed two per register.
// Updating is branch free (compare mask, max, bit select): a data-dependent branch would be taken
// by some lane of the warp at almost every step, because a thread only sees a few dozen vectors.
struct Track {
  __nv_bfloat162 m[4];
  uint32_t at[4];  // two 16-bit visit numbers; 0xFFFF = nothing above -inf seen yet
};
__device__ __forceinline__ void track_init(Track& t) {
#pragma unroll
  for (int j = 0; j < 4; ++j) { t.m[j] = as_bf162(0xFF80FF80u); t.at[j] = 0xFFFFFFFFu; }
}
__device__ __forceinline__ void take_vec(Track& t, const uint4& w, uint32_t visit2) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const __nv_bfloat162 x = as_bf162(u[j]);
    const uint32_t gt = __hgt2_mask(x, t.m[j]);  // strictly greater (false for NaN): first hit stays
    t.m[j] = __hmax2(t.m[j], x);                 // NaN operands are dropped
    t.at[j] = (t.at[j] & ~gt) | (visit2 & gt);
  }
}
struct Best {
  float v;
  int i;
};

__device__ __forceinline__ bool better(float v, int i, float bv, int bi) {
  return (v > bv) || (v == bv && i < bi);
}

__device__ __forceinline__ unsigned long long pack_key(float v, int i) {
  if (v == 0.0f) v = 0.0f;  // -0 and +0 are the same value: one bit pattern
  uint32_t f = __float_as_uint(v);
  uint32_t ord = (f & 0x80000000u) ? ~f : (f | 0x80000000u);
  return ((unsigned long long)ord << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
}

struct Params {
  const uint16_t* logits;
  int64_t ld;
  int vocab;
  int chunks;
  int chunk_elems;
  int32_t* ids;
  unsigned* tickets;
  unsigned long long* partial;
};

__global__ void __launch_bounds__(kThreads) argmax_kernel(Params p) {
  const int row = blockIdx.x / p.chunks;
  const int chunk = blockIdx.x - row * p.chunks;
  const int begin = chunk * p.chunk_elems;
  const int end = min(p.vocab, begin + p.chunk_elems);
  const uint16_t* base = p.logits + (int64_t)row * p.ld;
  const int nvec = (end - begin) >> 3;
  const uint4* vp = reinterpret_cast<const uint4*>(base + begin);
  const int tid = threadIdx.x;
  // programmatic launch: the grid may be set up while the previous kernel of the stream drains;
  // nothing is read or written before that kernel's results are complete
  cudaGridDependencySynchronize();

  Track trk;
  track_init(trk);
  int i = tid;
  uint32_t visit2 = 0;  // visit number in both halves
  for (; i + (kUnroll - 1) * kThreads < nvec; i += kUnroll * kThreads) {
    uint4 w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) w[u] = ld_stream16(vp + i + u * kThreads);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) { take_vec(trk, w[u], visit2); visit2 += 0x00010001u; }
  }
  for (; i < nvec; i += kThreads) { take_vec(trk, ld_stream16(vp + i), visit2); visit2 += 0x00010001u; }
  // the thread's best of its 8 positions: visit k of this thread is vector tid + k * kThreads
  Best best = {-INFINITY, INT_MAX};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
#pragma unroll
    for (int hlf = 0; hlf < 2; ++hlf) {
      const uint32_t k = hlf ? (trk.at[j] >> 16) : (trk.at[j] & 0xFFFFu);
      if (k == 0xFFFFu) continue;
      const float v = hlf ? __high2float(trk.m[j]) : __low2float(trk.m[j]);
      const int idx = begin + 8 * (tid + (int)k * kThreads) + 2 * j + hlf;
      if ((v > best.v) || (v == best.v && idx < best.i)) { best.v = v; best.i = idx; }
    }
  }
  // ragged end of the row (vocab not a multiple of 8): at most 7 scalars, after all vectors
  {
    const int t0 = begin + 8 * nvec + tid;
    if (t0 < end) {
      float x = __uint_as_float((uint32_t)base[t0] << 16);
      if (x > best.v) { best.v = x; best.i = t0; }
    }
  }

  // block reduction in the order (value descending, index ascending)
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xFFFFFFFFu, best.v, o);
    int oi = __shfl_xor_sync(0xFFFFFFFFu, best.i, o);
    if (better(ov, oi, best.v, best.i)) { best.v = ov; best.i = oi; }
  }
  __shared__ float sv[kThreads / 32];
  __shared__ int si[kThreads / 32];
  if ((tid & 31) == 0) { sv[tid >> 5] = best.v; si[tid >> 5] = best.i; }
  __syncthreads();
  if (tid != 0) return;
  for (int w = 1; w < kThreads / 32; ++w)
    if (better(sv[w], si[w], best.v, best.i)) { best.v = sv[w]; best.i = si[w]; }

  unsigned long long key = pack_key(best.v, best.i);
  if (p.chunks > 1) {
    unsigned long long* mine = p.partial + (size_t)row * p.chunks;
    __stcg(mine + chunk, key);
    __threadfence();
    const unsigned arrived = atomicInc(p.tickets + row, (unsigned)p.chunks - 1);  // wraps to 0
    if (arrived != (unsigned)p.chunks - 1) return;
    __threadfence();
    for (int c = 0; c < p.chunks; ++c) {
      unsigned long long k = __ldcg(mine + c);
      key = k > key ? k : key;
    }
  }
  int idx = (int)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
  p.ids[row] = (idx == INT_MAX) ? 0 : idx;  // a row of only -inf / NaN: first index
}

}  // namespace

ArgmaxPlan argmax_plan(int rows, int vocab) {
  ArgmaxPlan pl;
  pl.rows = rows;
  // 32768 logits (64 KB) per block = two batches of kUnroll loads per thread (measured best on
  // 128256-wide rows: 1024 blocks = one wave of 7 blocks per SM); fewer, smaller pieces only when
  // there are too few rows to cover the machine.
  const int unit = kThreads * 8;  // elements one pass of the block covers
  int chunk_elems = 2 * kUnroll * unit;
  const int want_blocks = 4 * sm_count();
  while (chunk_elems > unit && (int64_t)rows * ((vocab + chunk_elems - 1) / chunk_elems) < want_blocks)
    chunk_elems >>= 1;
  pl.chunk_elems = chunk_elems;
  pl.chunks = (vocab + chunk_elems - 1) / chunk_elems;
  pl.scratch_bytes = pl.chunks > 1 ? sizeof(unsigned long long) * (size_t)rows * pl.chunks : 0;
  return pl;
}

cudaError_t launch_argmax(const ArgmaxPlan& plan, const void* logits, int64_t ld, int vocab,
                          int32_t* ids, unsigned* tickets, void* scratch, cudaStream_t stream) {
  Params p;
  p.logits = static_cast<const uint16_t*>(logits);
  p.ld = ld;
  p.vocab = vocab;
  p.chunks = plan.chunks;
  p.chunk_elems = plan.chunk_elems;
  p.ids = ids;
  p.tickets = tickets;
  p.partial = static_cast<unsigned long long*>(scratch);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((int64_t)plan.rows * plan.chunks), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, argmax_kernel, p);
}

// ---- variant whose scratch lives in the library image ------------------------------------------
// For callers that cannot allocate device memory at all.  The scratch (arrival counters followed
// by the per-chunk keys) is a fixed array in this module's device image: every GPU that loads the
// library holds it until the process exits, and every call on that GPU shares it.
namespace {
constexpr int kStaticMaxRows = 4096;         // B * N
constexpr int kStaticMaxKeys = 131072;       // rows * chunks
constexpr size_t kStaticTicketBytes = sizeof(unsigned) * (size_t)kStaticMaxRows;
constexpr size_t kStaticBytes = kStaticTicketBytes + sizeof(unsigned long long) * (size_t)kStaticMaxKeys;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

unsigned char* g_static_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device
}  // namespace

bool argmax_static_fits(int rows, int vocab) {
  if (rows > kStaticMaxRows) return false;
  const ArgmaxPlan plan = argmax_plan(rows, vocab);
  return (int64_t)rows * plan.chunks <= kStaticMaxKeys;
}

cudaError_t launch_argmax_static(const void* logits, int64_t ld, int rows, int vocab, int32_t* ids,
                                 cudaStream_t stream) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_static_ptr[dev] == nullptr) {
    // In host code the array's name is only a handle; the address the kernel can use has to be
    // asked for, with the device that will run the kernel current.
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
  }
  unsigned char* base = g_static_ptr[dev];
  const ArgmaxPlan plan = argmax_plan(rows, vocab);
  if (plan.chunks > 1) {
    // the counters must start at zero whatever an earlier (possibly aborted) call left behind
    e = cudaMemsetAsync(base, 0, sizeof(unsigned) * (size_t)rows, stream);
    if (e != cudaSuccess) return e;
  }
  return launch_argmax(plan, logits, ld, vocab, ids, reinterpret_cast<unsigned*>(base),
                       base + kStaticTicketBytes, stream);
}

}  // namespace clv
