// LM head fused with the per-node greedy choice (Sec. 3.1: final norm and LM head of the target;
// Sec. 4.2: greedy decoding at T = 0): ids[r] = argmax_v round_bf16(<hidden[r, :], W[v, :]>), lowest
// v on ties.  The logits are never written: each 256 x 256 tile of them lives in tensor memory
// only, and its row maxima go to one 64-bit key per row with atomicMax.
//
// A persistent block per SM walks (vocabulary tile, row block) pairs.  Warp 0 streams 64-wide
// K chunks of the weight tile ([256 vocabulary rows][64]) and of the hidden rows ([2 x 128][64])
// through a three-deep TMA ring, warp 1 issues tcgen05.mma (M 128, N 256, K 16; two accumulators
// of 256 columns fill the tensor memory), warps 2..9 are the epilogue: one thread per row scans
// the accumulator for the row's best (value, lowest index).  The weight matrix is read from HBM
// once per row block; the hidden rows are re-read from L2 by every block.
#include <cuda_bf16.h>
#include <limits.h>
#include <math.h>

#include "clv_internal.cuh"
#include "tc_ptx.cuh"
#include "tmem_access.cuh"

namespace clv {
namespace {

constexpr int kThreads = 320;
constexpr int BM = 128;              // rows per accumulator
constexpr int MB = 2 * BM;           // rows per block step (two accumulators)
constexpr int BN = 256;              // vocabulary entries per tile
constexpr int BK = 64;               // K elements per ring stage (one 128-byte swizzle row)
constexpr int kStages = 3;
constexpr int kMaxProb = 3;          // products of one shape that one launch can take
constexpr uint32_t kATile = BM * BK * 2;      // 16 KB
constexpr uint32_t kWTile = BN * BK * 2;      // 32 KB
constexpr uint32_t kStageBytes = 2 * kATile + kWTile;
constexpr uint32_t kSmem = kStages * kStageBytes + 1024;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kIdesc = make_idesc(BM, BN, false);
constexpr uint32_t kIdescHalf = make_idesc(BM, BN / 2, false);

struct Params {
  int M, K, V;
  int n_tiles, m_blocks;
  int full_items;   // work items that are whole tiles; the rest are half tiles (128 vocabulary entries)
  int n_items;
  int32_t* ids;
  float* out;                 // not NULL: the products (+ bias) are written here, fp32 [M, ld_out], and no argmax is taken
  int n_prob;                 // with `out`: up to kMaxProb products of one shape in one launch, each with its own
  float* outs[3];             //   operands (tensor maps), destination and bias; out == outs[0]
  const uint16_t* biases[3];
  int64_t ld_out;
  int k_splits;               // with `out`: the K axis is cut in this many parts, part s writes its partial
  int64_t out_split_stride;   //   products to out + s * out_split_stride (the reader adds the parts up)
  int out_vec;                // `out`, its strides and `bias` allow 16-byte accesses
  int two_acc;                // M <= 128: the two accumulators alternate between tiles, so that the
                              //   epilogue of one tile runs under the MMAs of the next
  uint32_t a_tile_bytes;      // bytes one load of the row operand brings (a box of 8..128 rows)
  unsigned long long* keys;   // [M], zero between calls
  unsigned* counter;          // zero between calls
  unsigned* aborts;           // blocks that gave up a wait; zero between calls
  int32_t* status;            // one word: CLV_OK or CLV_ERR_TIMEOUT
  long long wait_limit;       // SM cycles a bounded wait may last
};

__device__ __forceinline__ unsigned long long pack_key(float v, int i) {
  if (v == 0.0f) v = 0.0f;  // -0 and +0 are the same value: one bit pattern
  const uint32_t f = __float_as_uint(v);
  const uint32_t ord = (f & 0x80000000u) ? ~f : (f | 0x80000000u);
  return ((unsigned long long)ord << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
}
__device__ __forceinline__ float round_bf16(float x) {
  return __bfloat162float(__float2bfloat16_rn(x));
}

// Work item -> (first vocabulary entry, entries, row block).  Items are whole tiles, all row
// blocks of a tile in a row so that a weight tile is read from HBM once and from L2 afterwards;
// when the last round would leave more than half of the blocks idle, its tiles are cut in two
// halves of 128 entries so that twice as many blocks share it.
struct Item {
  int col0, cols, mb;
};
__device__ __forceinline__ Item decode_item(const Params& p, int item) {
  int tile = item, half = -1;
  if (item >= p.full_items) {
    const int j = item - p.full_items;
    tile = p.full_items + (j >> 1);
    half = j & 1;
  }
  const int n = tile / p.m_blocks;
  Item it;
  it.mb = tile - n * p.m_blocks;
  it.col0 = n * BN + (half > 0 ? BN / 2 : 0);
  it.cols = half < 0 ? BN : BN / 2;
  return it;
}

struct Maps {
  CUtensorMap a[kMaxProb], w[kMaxProb], w_half;   // w_half: 128-entry boxes of w[0] (single product only)
};

__global__ void __launch_bounds__(kThreads, 1)
lm_head_argmax_kernel(const __grid_constant__ Maps tm, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) unsigned long long s_bar[2 * kStages + 5];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ int s_last;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar0 = smem_u32(&s_bar[0]);
  auto bar_full = [&](int s) { return bar0 + 8u * s; };
  auto bar_empty = [&](int s) { return bar0 + 8u * (kStages + s); };
  // a tile's accumulators are complete / the epilogue has read them; index 1 only with two_acc
  auto bar_acc_full = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto bar_acc_empty = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  const uint32_t bar_drain = bar0 + 8u * (2 * kStages + 4);
  if (tid == 0) {
    for (int i = 0; i < 2 * kStages; ++i) mbar_init(bar0 + 8u * i, 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full(b), 1);
      mbar_init(bar_acc_empty(b), p.two_acc ? BM : 2 * BM);
    }
    mbar_init(bar_drain, 1);
    s_abort = 0;
    fence_barrier_init();
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(&s_tmem), kTmemCols);
  if (tid >= 64 && tid < 64 + p.n_prob) {
    tma_prefetch_desc(&tm.a[tid - 64]);
    tma_prefetch_desc(&tm.w[tid - 64]);
    if (tid == 64) tma_prefetch_desc(&tm.w_half);
  }
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  if (p.a_tile_bytes < kATile) {
    // a box of fewer than 128 rows leaves the rest of the operand tile as it was: make that zeros
    uint8_t* base = smem_raw + (smem_base - smem_u32(smem_raw));
    for (int s = 0; s < kStages; ++s)
      for (uint32_t o = (uint32_t)tid * 16u; o < kATile; o += kThreads * 16u)
        *reinterpret_cast<uint4*>(base + (size_t)s * kStageBytes + o) = make_uint4(0u, 0u, 0u, 0u);
    fence_async_smem();
  }
  cudaGridDependencySynchronize();  // programmatic launch: the previous kernel's results are complete
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abort_flag = &s_abort;
  const long long wlim = p.wait_limit;

  auto sA = [&](int s, int mt) { return smem_base + (uint32_t)s * kStageBytes + (uint32_t)mt * kATile; };
  auto sW = [&](int s) { return smem_base + (uint32_t)s * kStageBytes + 2 * kATile; };

  // work item -> (tile and row block, part of the K axis, product): products innermost, so that
  // blocks working side by side read different weights
  const int per_tile = p.k_splits * p.n_prob;
  const int n_items = p.n_items * per_tile;
  const int k_chunks = p.K / BK / p.k_splits;
  int issued = 0;  // ring stages filled by the producer (for the drain)

  if (warp == 0) {
    // =========================== TMA producer ===============================================
    if (lane == 0) {
      bool ok = true;
      int it = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const Item wi = decode_item(p, item / per_tile);
        const int sub = item % per_tile, prob = sub % p.n_prob;
        const int kc0 = (sub / p.n_prob) * k_chunks;
        const int mb = wi.mb;
        const int rows_left = p.M - mb * MB;
        const int m_tiles = rows_left > BM ? 2 : 1;
        const uint32_t w_bytes = (uint32_t)wi.cols * BK * 2;
        for (int kc = 0; kc < k_chunks && ok; ++kc, ++it) {
          const int s = it % kStages;
          if (it >= kStages) ok = mbar_wait(bar_empty(s), ((it / kStages) - 1) & 1, abort_flag, wlim);
          if (!ok) break;
          mbar_expect_tx(bar_full(s), w_bytes + (uint32_t)m_tiles * p.a_tile_bytes);
          tma_load_2d(sW(s), wi.cols == BN ? &tm.w[prob] : &tm.w_half, (kc0 + kc) * BK, wi.col0, bar_full(s));
          for (int mt = 0; mt < m_tiles; ++mt)
            tma_load_2d(sA(s, mt), &tm.a[prob], (kc0 + kc) * BK, mb * MB + mt * BM, bar_full(s));
          issued = it + 1;
        }
      }
    }
  } else if (warp == 1) {
    // =========================== MMA issuer ===================================================
    if (lane == 0) {
      bool ok = true;
      int it = 0, tile = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tile) {
        const Item wi = decode_item(p, item / per_tile);
        const int m_tiles = (p.M - wi.mb * MB) > BM ? 2 : 1;
        const uint32_t idesc = wi.cols == BN ? kIdesc : kIdescHalf;
        const int acc = p.two_acc ? (tile & 1) : 0;          // accumulator (pair) of this tile
        const int use = p.two_acc ? (tile >> 1) : tile;      // how often it has been used before
        if (use > 0) {  // the epilogue has taken its previous tile out of tensor memory
          ok = mbar_wait(bar_acc_empty(acc), (use - 1) & 1, abort_flag, wlim);
          if (!ok) break;
          tc_fence_after();
        }
        for (int kc = 0; kc < k_chunks && ok; ++kc, ++it) {
          const int s = it % kStages;
          ok = mbar_wait(bar_full(s), (it / kStages) & 1, abort_flag, wlim);
          if (!ok) break;
          tc_fence_after();
          const uint64_t wd = smem_desc(sW(s), 16, 1024);
          for (int mt = 0; mt < m_tiles; ++mt) {
            const uint64_t ad = smem_desc(sA(s, mt), 16, 1024);
#pragma unroll
            for (int ks = 0; ks < BK / 16; ++ks)
              umma_bf16(tmem + (uint32_t)((mt + acc) * BN), ad + (uint64_t)((ks * 32) >> 4), wd + (uint64_t)((ks * 32) >> 4),
                        idesc, (kc > 0 || ks > 0) ? 1u : 0u);
          }
          umma_commit(bar_empty(s));  // the stage is free once these MMAs have read it
        }
        if (ok) umma_commit(bar_acc_full(acc));
      }
    }
  } else {
    // =========================== epilogue: one thread per row ==================================
    const int mt = (warp - 2) >> 2;          // accumulator of this group
    const int quarter = warp & 3;            // tensor-memory lanes this warp may touch
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    bool ok = true;
    int tile = 0;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tile) {
      const Item wi = decode_item(p, item / per_tile);
      const int sub = item % per_tile, prob = sub % p.n_prob, part = sub / p.n_prob;
      const int mb = wi.mb;
      if (p.two_acc && (tile & 1) != mt) continue;   // the other group's tile
      const int acc = p.two_acc ? mt : 0;
      const int row = mb * MB + (p.two_acc ? 0 : mt * BM) + row_in_tile;
      const bool row_valid = row < p.M;
      ok = mbar_wait(bar_acc_full(acc), (p.two_acc ? (tile >> 1) : tile) & 1, abort_flag, wlim);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      // the second accumulator is unused for a short row block
      const bool group_used = p.two_acc || (p.M - mb * MB) > mt * BM;
      float best_v = -INFINITY;
      int best_i = INT_MAX;
      if (group_used) {
        const int col0 = wi.col0;
#pragma unroll 1
        for (int c = 0; c < wi.cols; c += 32) {
          uint32_t x[32];
          tmem_ld_x32(tmem + lane_addr + (uint32_t)(mt * BN + c), x);
          tmem_wait_ld();
          if (p.out != nullptr) {   // plain product: this row's 32 values (+ bias) go to memory
            if (row_valid) {
              const uint16_t* bias = p.biases[0];
              float* dst = p.outs[0];
              if (prob == 1) { bias = p.biases[1]; dst = p.outs[1]; }
              if (prob == 2) { bias = p.biases[2]; dst = p.outs[2]; }
              dst += part * p.out_split_stride + (int64_t)row * p.ld_out + col0 + c;
              const bool add_bias = bias != nullptr && part == 0;
              if (p.out_vec && col0 + c + 32 <= p.V) {   // 128 bytes of this row in eight stores
                if (add_bias) {
                  const uint4* b4 = reinterpret_cast<const uint4*>(bias + col0 + c);
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    const uint4 b = b4[j];
                    const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                      x[8 * j + 2 * t] = __float_as_uint(__uint_as_float(x[8 * j + 2 * t]) + __uint_as_float(w[t] << 16));
                      x[8 * j + 2 * t + 1] =
                          __float_as_uint(__uint_as_float(x[8 * j + 2 * t + 1]) + __uint_as_float(w[t] & 0xFFFF0000u));
                    }
                  }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j)
                  reinterpret_cast<uint4*>(dst)[j] = make_uint4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  if (col0 + c + j >= p.V) continue;
                  float v = __uint_as_float(x[j]);
                  if (add_bias) v += __uint_as_float((uint32_t)bias[col0 + c + j] << 16);
                  dst[j] = v;
                }
              }
            }
            continue;
          }
          // rounding to bf16 is monotonic: the chunk's maximum first, the position only if it wins
          float m = -INFINITY;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float v = (col0 + c + j < p.V) ? __uint_as_float(x[j]) : -INFINITY;
            x[j] = __float_as_uint(v);
            m = fmaxf(m, v);   // NaN operands are dropped
          }
          const float mr = round_bf16(m);
          if (mr > best_v) {
            int first = 31;
#pragma unroll
            for (int j = 31; j >= 0; --j)
              if (round_bf16(__uint_as_float(x[j])) == mr) first = j;
            best_v = mr;
            best_i = col0 + c + first;
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar_acc_empty(acc));
      if (row_valid && best_i != INT_MAX) atomicMax(p.keys + row, pack_key(best_v, best_i));
    }
  }

  // ---- teardown --------------------------------------------------------------------------------
  __syncwarp();
  if (*abort_flag) {
    if (warp == 0 && lane == 0)
      for (int i = max(0, issued - kStages); i < issued; ++i) mbar_drain(bar_full(i % kStages), (i / kStages) & 1);
    if (warp == 1 && lane == 0) {
      umma_commit(bar_drain);
      mbar_drain(bar_drain, 0);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, kTmemCols);
  if (tid == 0) {
    if (*abort_flag) atomicAdd(p.aborts, 1u);
    __threadfence();
    const unsigned arrived = atomicInc(p.counter, gridDim.x - 1);  // wraps to 0
    s_last = (arrived == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  // the last block turns the keys into indices and leaves keys and counters zero for the next call
  __threadfence();
  if (tid == 0) {   // one status word per product
    const int verdict = atomicExch(p.aborts, 0u) ? (int)CLV_ERR_TIMEOUT : (int)CLV_OK;
    for (int i = 0; i < p.n_prob; ++i) p.status[i] = verdict;
  }
  if (p.out != nullptr) return;   // no keys were written
  for (int r = tid; r < p.M; r += kThreads) {
    const unsigned long long key = atomicExch(p.keys + r, 0ull);
    const int idx = (int)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
    p.ids[r] = (key == 0ull) ? 0 : idx;  // a row of only -inf / NaN logits: first index
  }
}

bool make_map_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t k, int64_t ld, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)k, rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool lm_head_supported(int rows, int hidden, int vocab) {
  // keys share the zero-initialised counter area of the workspace: 2 words per row after the counter
  return rows > 0 && vocab > 0 && hidden > 0 && (hidden % BK) == 0 && 2 * (int64_t)rows + 2 <= kTickets &&
         encode_fn() != nullptr;
}

namespace {
struct Product {   // one product of a launch: rows x[rows, K] times weight[vocab, K]^T (+ bias) -> out
  const void* x;
  const void* weight;
  const void* bias;
  float* out;
};

cudaError_t launch_rows_times_weights(int n_prob, const Product* pr, int64_t ld_hidden, int64_t ld_weight, int rows,
                                      int hidden_dim, int vocab, int32_t* ids, int64_t ld_out, int k_splits,
                                      int64_t out_split_stride, int32_t* status, unsigned* tickets,
                                      cudaStream_t stream) {
  static OncePerDevice once;
  cudaError_t e0 = run_once_per_device(once, [] {
    return cudaFuncSetAttribute(lm_head_argmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
  });
  if (e0 != cudaSuccess) return e0;
  if (n_prob < 1 || n_prob > kMaxProb) return cudaErrorInvalidValue;
  Maps tm;
  int a_box = BM;   // rows one load of the row operand brings: the power of two that covers them, 8..128
  while (a_box > 8 && a_box / 2 >= rows) a_box /= 2;
  Params p;
  bool vec = (ld_out % 4) == 0 && (out_split_stride % 4) == 0;
  for (int i = 0; i < kMaxProb; ++i) {
    const Product& q = pr[i < n_prob ? i : 0];   // unused slots repeat the first product
    if (!make_map_2d(&tm.a[i], q.x, (uint64_t)rows, (uint64_t)hidden_dim, ld_hidden, (uint32_t)a_box) ||
        !make_map_2d(&tm.w[i], q.weight, (uint64_t)vocab, (uint64_t)hidden_dim, ld_weight, BN))
      return cudaErrorInvalidValue;
    p.outs[i] = q.out;
    p.biases[i] = static_cast<const uint16_t*>(q.bias);
    vec = vec && (reinterpret_cast<uintptr_t>(q.out) % 16) == 0 && (reinterpret_cast<uintptr_t>(q.bias) % 16) == 0;
  }
  if (!make_map_2d(&tm.w_half, pr[0].weight, (uint64_t)vocab, (uint64_t)hidden_dim, ld_weight, BN / 2))
    return cudaErrorInvalidValue;
  p.M = rows;
  p.K = hidden_dim;
  p.V = vocab;
  p.n_tiles = (vocab + BN - 1) / BN;
  p.m_blocks = (rows + MB - 1) / MB;
  p.ids = ids;
  p.out = pr[0].out;
  p.n_prob = n_prob;
  p.ld_out = ld_out;
  p.k_splits = k_splits;
  p.out_split_stride = out_split_stride;
  p.out_vec = p.out != nullptr && vec;
  p.two_acc = rows <= BM;
  p.a_tile_bytes = (uint32_t)a_box * BK * 2;
  p.counter = tickets;
  p.aborts = tickets + 1;
  p.keys = reinterpret_cast<unsigned long long*>(tickets + 2);
  p.status = status;
  p.wait_limit = wait_limit_cycles();
  const int tiles = p.n_tiles * p.m_blocks;
  const int work = tiles * k_splits * n_prob;
  const int grid = work < sm_count() ? work : sm_count();
  const int rem = tiles % grid;   // tiles of the last, incomplete round
  const int split = (k_splits == 1 && n_prob == 1 && rem > 0 && 2 * rem <= grid) ? rem : 0;
  p.full_items = tiles - split;
  p.n_items = tiles + split;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, lm_head_argmax_kernel, tm, p);
}
}  // namespace

cudaError_t launch_lm_head_argmax(const void* hidden, int64_t ld_hidden, const void* weight, int64_t ld_weight,
                                  int rows, int hidden_dim, int vocab, int32_t* ids, int32_t* status,
                                  unsigned* tickets, cudaStream_t stream) {
  const Product pr = {hidden, weight, nullptr, nullptr};
  return launch_rows_times_weights(1, &pr, ld_hidden, ld_weight, rows, hidden_dim, vocab, ids, 0, 1, 0, status,
                                   tickets, stream);
}

// How many parts the K axis of a product with few output features is cut into, so that the launch
// covers the machine: a power of two up to 8 that divides the number of 64-wide K chunks.
// `n` products of one shape share the launch; up to three rounds of blocks are accepted.
int rows_linear_splits(int rows, int in_dim, int out_dim, int n) {
  const int tiles = ((out_dim + BN - 1) / BN) * ((rows + MB - 1) / MB) * n;
  int s = 1;
  while (s < 8 && tiles * s * 2 <= 3 * sm_count() && (in_dim / BK) % (s * 2) == 0) s *= 2;
  return s;
}

// out[i][part][r][o] = sum over part's share of k of x[i][r][k] * weight[i][o][k] (+ bias[i][o] in
// part 0) for n products of one shape (n <= 3) in one launch: the same kernel with its
// accumulators written out (fp32) instead of reduced to an argmax.  The reader adds the `splits`
// parts up (a fixed order: the result does not depend on scheduling).  status gets one word per
// product.
cudaError_t launch_rows_linear(int n, const void* const* x, int64_t ld_x, const void* const* weight,
                               int64_t ld_weight, const void* const* bias, int rows, int in_dim, int out_dim,
                               float* const* out, int64_t ld_out, int splits, int64_t split_stride, int32_t* status,
                               unsigned* tickets, cudaStream_t stream) {
  if (n < 1 || n > kMaxProb) return cudaErrorInvalidValue;
  Product pr[kMaxProb];
  for (int i = 0; i < n; ++i) pr[i] = Product{x[i], weight[i], bias[i], out[i]};
  return launch_rows_times_weights(n, pr, ld_x, ld_weight, rows, in_dim, out_dim, nullptr, ld_out, splits,
                                   split_stride, status, tickets, stream);
}

}  // namespace clv
