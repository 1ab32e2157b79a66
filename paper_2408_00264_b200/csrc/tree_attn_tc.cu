// Tree attention (Sec. 2.1) on the 5th-generation tensor cores: tcgen05.mma with accumulators in
// tensor memory, K/V/Q tiles staged by TMA into 128-byte-swizzled shared memory.
//
// Query row = (tree node, head-in-group) pair, so all G heads of a GQA group and all tree nodes
// reuse every K/V byte.  A row tile of 128 rows holds whole nodes: 128 / G of them (rounded down;
// its other rows idle).  One thread block owns ONE row tile of one (sequence, kv head) and a
// contiguous range of the key axis (cache keys first, then the tree's own), walked in tiles of
// 128 keys that are loaded as 64-key pieces (also the page size of a paged cache).
// Roles: warp 0 = TMA producer, warp 1 = MMA issuer and owner of the tensor-memory allocation;
// warps 2-9 = softmax, two threads per query row: thread `ch` of a
// row takes the 64 columns of piece `ch` of every key tile.
// Tensor memory: three score buffers of 128 columns and one output accumulator of 128.  The
// issuer runs Q K^T up to three tiles ahead, so the softmax threads find the next scores ready
// when they finish a tile, and P V of a tile runs beside the softmax of the next one.
// Per tile: S = Q K^T -> the row's two threads read their halves, mask, exponentiate against a
// lazily updated reference maximum and add up the row -> P (bf16) overwrites consumed score
// columns -> O += P V (A operand from tensor memory).  The tree columns are masked with per-node
// ancestor bitsets derived from parent[] on chip; masked scores are replaced, not added to, so
// they contribute exactly zero.
// Split-KV: the blocks that share a row tile form one thread-block cluster; each stages
// its accumulator in its own shared memory and every block finalises a share of the rows by
// reading its peers' staging areas (distributed shared memory): no partial result touches global
// memory.  Every wait is bounded: on expiry the block raises a flag, all roles leave their loops,
// in-flight copies and MMAs are drained, the cluster meets, tensor memory is released and
// CLV_ERR_TIMEOUT is reported for the sequence.
#include <cooperative_groups.h>
#include <cuda.h>
#include <cuda_fp16.h>
#include <math.h>

#include "clv_internal.cuh"
#include "tc_ptx.cuh"
#include "tmem_access.cuh"

namespace cg = cooperative_groups;

namespace clv {
namespace {

constexpr int PG = CLV_PAGE_SIZE;      // 64: keys per TMA piece (= page size)
constexpr int HD = CLV_HEAD_DIM;       // 128
constexpr int BM = 128;                // rows per block
constexpr int BN = 128;                // keys per tile
constexpr int PPT = BN / PG;           // pieces per tile
constexpr int NSB = 3;                 // score buffers (= depth of the K ring)
constexpr int kThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr uint32_t kQTile = BM * HD * 2;      // 32 KB: two [128 rows][64 d] swizzled halves
constexpr uint32_t kPiece = PG * 64 * 2;       // 8 KB: [64 keys][64 d] swizzled, one TMA box
constexpr uint32_t kTmemCols = 512;
constexpr float kRowSumLimit = 256.0f;        // a thread's part of a row of P may sum to 2^8 before the reference is replaced

struct Cfg {
  static constexpr int KST = NSB;                   // a K buffer and a score buffer free together
  static constexpr int VST = 2;                     // depth of the V ring
  static constexpr uint32_t kStage = BN * HD * 2;   // bytes of a K (or V) tile
  static constexpr uint32_t kSmem = kQTile + (KST + VST) * kStage + 1024;
};

struct Params {
  const int32_t* block_table;
  const int32_t* parent;
  const int32_t* ctx_len;
  uint16_t* out;
  float* lse;
  int32_t* status;
  int B, N, Hq, Hkv, G;
  int paged, cap_tokens, n_pages, max_pages;
  int longest_first;  // hand out sequences in order of decreasing context length
  int pair_boxes;     // the 4-D tensor maps exist: a whole 128-key tile of a contiguous cache is one copy
  int tiles;       // row tiles per (sequence, kv head); each is worked by one cluster
  int splits;      // blocks along the key axis = cluster size
  float scale_log2;
  long long wait_limit;   // SM cycles a bounded wait may last
  unsigned* tickets;      // per sequence: [2b] blocks that have finished, [2b+1] error bits; zero between calls
  int blocks_per_seq;
};

// Distributed shared memory: 8- and 16-byte loads from a peer's shared memory.  Volatile asm, so
// that a batch of them is issued back to back (all in flight) before the first result is used.
__device__ __forceinline__ float4 dsmem_ld16(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 dsmem_ld8u(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared::cluster.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float2 half2_bits_to_float2(uint32_t u) {
  return __half22float2(*reinterpret_cast<const __half2*>(&u));
}
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// The same loads from this block's own shared memory (volatile asm too, so that they join the batch).
__device__ __forceinline__ float4 smem_ld16(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 smem_ld8u(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

// Final combination of NSRC accumulators per output row, for the rows [first_row, first_row +
// per_rank) of the tile that this block finalises.  The staged accumulators are fp16 (each row
// scaled by a power of two of its own, which the weight undoes), 256 bytes per row; source q of a
// row lives in cluster rank q (this block's own share is read locally).  One warp takes 16 / NSRC
// rows at a time: lane i < 16 fetches the (maximum, sum, scale) of one (row, source) pair and
// every lane 16 8-byte pieces of the rows, all in flight together (one round trip through
// distributed shared memory); the normalised weights then come from shuffles.  Lane j owns output
// columns 4j .. 4j+3.
template <int NSRC>
__device__ __forceinline__ void merge_rows(uint32_t sO_addr, uint32_t ml_addr, int my_rank, int first_row,
                                           int per_rank, int warp, int lane, const long long* row_off,
                                           uint16_t* out, float* lse) {
  constexpr int RB = 16 / NSRC;
  const float kLn2 = 0.6931471805599453f;
  const int rot = my_rank + 1;   // first source read: the next rank's (every block starts at a different peer)
  for (int k0 = warp * RB; k0 < per_rank; k0 += RB * (kThreads / 32)) {
    const int mu_ = (lane & 15) / NSRC, mj = (lane & 15) % NSRC;   // this lane's (row, source) pair
    float4 ml;
    {
      const int trow = first_row + min(k0 + mu_, per_rank - 1);
      const uint32_t a = ml_addr + (uint32_t)trow * 16u;
      ml = (mj == my_rank) ? smem_ld16(a) : dsmem_ld16(cluster_map(a, (uint32_t)mj));
    }
    uint2 x[RB * NSRC];
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      const int trow = first_row + min(k0 + u, per_rank - 1);
      const uint32_t off = (uint32_t)(trow * (HD * 2) + (((lane >> 1) ^ (trow & 15)) << 4) + ((lane & 1) << 3));
#pragma unroll
      for (int j = 0; j < NSRC; ++j) {
        const int q = (j + rot) & (NSRC - 1);
        x[u * NSRC + j] = (q == my_rank) ? smem_ld8u(sO_addr + off) : dsmem_ld8u(cluster_map(sO_addr + off, (uint32_t)q));
      }
    }
    // weights: the NSRC lanes of a row sit side by side
    float mmax = ml.x;
#pragma unroll
    for (int o = 1; o < NSRC; o <<= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xFFFFFFFFu, mmax, o));
    const float mu = (mmax == -INFINITY) ? 0.f : mmax;
    const float wgt = (ml.y > 0.f) ? ex2(ml.x - mu) : 0.f;
    float lsum = wgt * ml.y;
#pragma unroll
    for (int o = 1; o < NSRC; o <<= 1) lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, o);
    const float wn = wgt * (lsum > 0.f ? 1.f / lsum : 0.f) * ml.z;  // the staged row is 1 / ml.z times O
    if (lse != nullptr && lane < 16 && mj == 0 && k0 + mu_ < per_rank) {
      const long long o = row_off[first_row + k0 + mu_];   // where the row's output starts, -1 for an idle row
      if (o >= 0) lse[o / HD] = (mmax + log2f(lsum)) * kLn2;
    }
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int j = 0; j < NSRC; ++j) {
        const float wq = __shfl_sync(0xFFFFFFFFu, wn, u * NSRC + ((j + rot) & (NSRC - 1)));
        const float2 lo = half2_bits_to_float2(x[u * NSRC + j].x), hi = half2_bits_to_float2(x[u * NSRC + j].y);
        acc.x += wq * lo.x; acc.y += wq * lo.y; acc.z += wq * hi.x; acc.w += wq * hi.y;
      }
      if (k0 + u >= per_rank) continue;
      const long long o = row_off[first_row + k0 + u];
      if (o < 0) continue;
      *reinterpret_cast<uint2*>(out + o + lane * 4) = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    }
  }
}

// ------------------------------------------------------------------------------------ kernel
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc,
                    const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kt,
                    const __grid_constant__ CUtensorMap tm_vt, const __grid_constant__ CUtensorMap tm_kc2,
                    const __grid_constant__ CUtensorMap tm_vc2, const Params p) {
  constexpr int KST = Cfg::KST, VST = Cfg::VST;
  constexpr uint32_t kStage = Cfg::kStage;
  constexpr uint32_t kHalf = kStage / 2;    // a stage holds [64-wide half of d][128 keys][64 d]
  constexpr uint32_t kIdescQK = make_idesc(BM, BN, false);  // S[128 rows x 128 keys] = Q K^T
  constexpr uint32_t kIdescPV = make_idesc(BM, HD, true);   // O[128 rows x 128 d] += P V
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t s_anc[CLV_MAX_NODES][4];
  __shared__ int s_parent[CLV_MAX_NODES];
  // barriers: K full [KST] | V full [VST] | S full [NSB] | P full [NSB] | P V done [NSB] | V empty [VST] | Q | drain
  constexpr int B_KF = 0, B_VF = B_KF + KST, B_SF = B_VF + VST, B_PF = B_SF + NSB, B_PV = B_PF + NSB,
                B_VE = B_PV + NSB, B_Q = B_VE + VST, B_DR = B_Q + 1, NBAR = B_DR + 1;
  __shared__ __align__(8) unsigned long long s_bar[NBAR];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ int s_redo[8];        // per softmax warp: the last tile in which one of its row sums was suspect
  __shared__ int s_fail[8];        // per softmax warp: one of its waits has run out
  __shared__ float s_xch[2][BM];   // values exchanged between the two threads of a row
  __shared__ float s_xch2[2][BM];
  __shared__ float4 s_ml[BM];      // (reference maximum, row sum, 1 / staging scale, -) for the merge
  __shared__ int s_seq;
  __shared__ long long s_rowoff[BM];   // per row of the tile: element offset of its output row, -1 for an idle row

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int CS = p.splits;                            // cluster size
  const int split = (int)(blockIdx.x % (unsigned)CS); // rank in the cluster (clusters are laid along x)
  const int cluster_id = (int)(blockIdx.x / (unsigned)CS);
  const int unit = cluster_id / p.tiles, tile_idx = cluster_id - unit * p.tiles;   // this block's row tile
  int b = unit / p.Hkv;
  const int kvh = unit - b * p.Hkv;
  const int N = p.N, G = p.G, rows_total = G * N;
  const int RT = (BM / G) * G;                        // rows of a tile that hold whole nodes

  // ---- set-up that reads no global memory: barriers, tensor memory, descriptor prefetch.  The
  //      kernel is launched with programmatic stream serialisation, so this part may run while the
  //      previous kernel of the stream drains.
  const uint32_t bar0 = smem_u32(&s_bar[0]);
  auto bar = [&](int idx) { return bar0 + 8u * (uint32_t)idx; };
  if (tid == 0) {
    for (int i = 0; i < KST; ++i) mbar_init(bar(B_KF + i), 1);
    for (int i = 0; i < VST; ++i) { mbar_init(bar(B_VF + i), 1); mbar_init(bar(B_VE + i), 1); }
    for (int i = 0; i < NSB; ++i) {
      mbar_init(bar(B_SF + i), 1);
      mbar_init(bar(B_PF + i), 8);   // one arrival per softmax warp
      mbar_init(bar(B_PV + i), 1);
    }
    mbar_init(bar(B_Q), 1);
    mbar_init(bar(B_DR), 1);
    s_abort = 0;
    for (int i = 0; i < 8; ++i) { s_redo[i] = -1; s_fail[i] = 0; }
    fence_barrier_init();
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(&s_tmem), kTmemCols);
  if (tid == 64) {
    tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_kc); tma_prefetch_desc(&tm_vc);
    tma_prefetch_desc(&tm_kt); tma_prefetch_desc(&tm_vt);
    if (p.pair_boxes) { tma_prefetch_desc(&tm_kc2); tma_prefetch_desc(&tm_vc2); }
  }
  cudaGridDependencySynchronize();

  if (p.longest_first) {
    // More blocks than SMs and contexts of different lengths (ragged batch): hand the sequences
    // out longest first, so that the block scheduler packs the short ones into the gaps.  Block
    // group `b` takes the sequence whose length has rank b (ties by index).
    const int want = b;
    for (int i = tid; i < p.B; i += kThreads) {
      const int Li = p.ctx_len[i];
      int rank = 0;
      for (int j = 0; j < p.B; ++j) {
        const int Lj = __ldg(p.ctx_len + j);
        rank += (Lj > Li) || (Lj == Li && j < i);
      }
      if (rank == want) s_seq = i;
    }
    __syncthreads();
    b = s_seq;
  }

  // ---- the sequence's length, this block's range of the key axis ------------------------------
  // The key axis is cut in 64-key pieces: p_cache pieces of context, then the tree's own pieces.
  // A split takes a contiguous range of pieces and walks it in tiles of two pieces; the last tile
  // of a range may hold one piece only.
  const int L = p.ctx_len[b];
  const bool len_bad = (L < 0) || (p.paged ? ((L + PG - 1) / PG > p.max_pages) : (L > p.cap_tokens));
  const int p_cache = (!len_bad && L > 0) ? (L + PG - 1) / PG : 0;  // 64-key pieces (pages) of the context
  const int p_total = p_cache + (N + PG - 1) / PG;
  const int pc_begin = (int)((unsigned)split * (unsigned)p_total / (unsigned)p.splits);
  const int pc_end = (int)((unsigned)(split + 1) * (unsigned)p_total / (unsigned)p.splits);
  const int T = (pc_end - pc_begin + PPT - 1) / PPT;   // tiles of this block

  // ---- shared memory carve-up (1024-byte aligned tiles for the 128-byte swizzle) ------------
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem_base;
  const uint32_t sK = sQ + kQTile;           // ring of KST K stages
  const uint32_t sV = sK + KST * kStage;     // ring of VST V stages
  uint8_t* const sV_gen = smem_raw + (sV - smem_u32(smem_raw));

  volatile int* abort_flag = &s_abort;
  const long long wlim = p.wait_limit;

  // ---- the producer's two steps (whole warp 0): the copies of K tile kt / V tile vt.  Lane j
  //      caches the pool page of context piece (base + j) for each ring (paged cache).
  int issued_k = 0, issued_v = 0;  // bookkeeping for the drain
  int pk_page = 0, pk_base = -64, pv_page = 0, pv_base = -64;
  auto issue_tile = [&](int t, bool is_k, int& page, int& page_base) {
    const int g0 = pc_begin + t * PPT;
    if (p.paged && g0 < p_cache && g0 + PPT > page_base + 32) {
      page_base = g0;
      const int pc = g0 + lane;
      page = (pc < p_cache) ? p.block_table[(int64_t)b * p.max_pages + pc] : 0;
    }
    int row0[PPT];
    bool is_tree[PPT];
#pragma unroll
    for (int j = 0; j < PPT; ++j) {
      const int g = g0 + j;
      int pg = __shfl_sync(0xFFFFFFFFu, page, (g - page_base) & 31);
      is_tree[j] = g >= p_cache;
      if (g >= pc_end) row0[j] = -1;     // the range ended inside this tile
      else if (is_tree[j]) row0[j] = b * N + (g - p_cache) * PG;
      else if (p.paged) {
        if (pg < 0 || pg >= p.n_pages) pg = 0;   // the reporter flags the sequence; any page will do
        row0[j] = pg * PG;
      } else row0[j] = b * p.cap_tokens + g * PG;
    }
    if (lane == 0) {
      const int st = is_k ? t % KST : t % VST;
      const uint32_t full = is_k ? bar(B_KF + st) : bar(B_VF + st);
      const uint32_t stage = (is_k ? sK : sV) + (uint32_t)st * kStage;
      if (p.pair_boxes && row0[0] >= 0 && !is_tree[1] && row0[1] == row0[0] + PG) {
        // both pieces are neighbours in the cache: the whole tile, both halves of d, in one copy
        mbar_expect_tx(full, kStage);
        tma_load_4d(stage, is_k ? &tm_kc2 : &tm_vc2, 0, row0[0], 0, kvh, full);
      } else {
        int n_pieces = 0;
#pragma unroll
        for (int j = 0; j < PPT; ++j) n_pieces += row0[j] >= 0;
        mbar_expect_tx(full, (uint32_t)n_pieces * 2u * kPiece);  // 0 bytes: a plain arrival
#pragma unroll
        for (int j = 0; j < PPT; ++j) {
          if (row0[j] < 0) continue;
          const CUtensorMap* m = is_tree[j] ? (is_k ? &tm_kt : &tm_vt) : (is_k ? &tm_kc : &tm_vc);
          const uint32_t dst = stage + (uint32_t)j * kPiece;
          tma_load_3d(dst, m, 0, kvh, row0[j], full);
          tma_load_3d(dst + kHalf, m, 64, kvh, row0[j], full);
        }
      }
    }
    if (is_k) issued_k = t + 1;
    else issued_v = t + 1;
  };
  // The Q tile and the first tiles of both rings go out before the block's first barrier: they
  // need the sequence's length only (a bad length reads the tree's own rows, which exist; the
  // block then waits for these copies before it leaves).
  int kt0 = 0, vt0 = 0;
  if (warp == 0 && T > 0) {
    if (lane == 0) {
      mbar_expect_tx(bar(B_Q), (uint32_t)(RT * HD * 2));   // the boxes hold RT rows
      const int node0 = b * N + tile_idx * (BM / G);
      tma_load_3d(sQ, &tm_q, 0, kvh * G, node0, bar(B_Q));
      tma_load_3d(sQ + kQTile / 2, &tm_q, 64, kvh * G, node0, bar(B_Q));
    }
    const int nk = min(T, KST), nv = min(T, VST);
    while (kt0 < nk || vt0 < nv) {
      if (kt0 < nk) { issue_tile(kt0, true, pk_page, pk_base); ++kt0; }
      if (vt0 < nv) { issue_tile(vt0, false, pv_page, pv_base); ++vt0; }
    }
  }

  // ---- per-sequence checks (the threads of warps 2 and up) ----------------------------------
  bool bad = len_bad;
  for (int i = tid - 64; i < N; i += kThreads - 64) {
    if (i < 0) continue;
    const int par = p.parent[(int64_t)b * N + i];
    s_parent[i] = par;
    bad |= (par < -1 || par >= i);
  }
  tc_fence_before();
  const int seq_bad = __syncthreads_or(bad ? 1 : 0);  // same verdict in every block of the sequence
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const bool reporter = (tile_idx == 0 && split == 0 && kvh == 0);
  // status[b] is written once, by whichever block of the sequence finishes last: every block adds
  // its error bits (1 malformed input, 2 a wait ran out) to the sequence's word in the workspace
  // and then takes a ticket; the holder of the last ticket turns the bits into the status code and
  // leaves both words zero for the next call.
  auto report = [&](unsigned bits) -> unsigned {   // one thread per block; returns the ticket
    if (bits) atomicOr(p.tickets + 2 * b + 1, bits);
    __threadfence();
    return atomicInc(p.tickets + 2 * b, (unsigned)p.blocks_per_seq - 1);  // wraps to 0
  };
  auto publish = [&](unsigned ticket) {
    if (ticket != (unsigned)p.blocks_per_seq - 1) return;
    __threadfence();
    const unsigned bits = atomicExch(p.tickets + 2 * b + 1, 0u);
    p.status[b] = (bits & 1u) ? CLV_ERR_TREE : (bits & 2u) ? CLV_ERR_TIMEOUT : CLV_OK;
  };
  auto release_tmem = [&]() { tmem_dealloc(tmem, kTmemCols); };   // warp 1
  if (seq_bad) {  // the whole cluster leaves together, once the copies that are under way have landed
    if (tid == 0) {
      for (int i = 0; i < kt0; ++i) mbar_drain(bar(B_KF + i), 0);
      for (int i = 0; i < vt0; ++i) mbar_drain(bar(B_VF + i), 0);
      if (T > 0) mbar_drain(bar(B_Q), 0);
    }
    if (warp == 1) release_tmem();
    if (tid == 0) publish(report(1u));
    return;
  }

  auto tmem_S = [&](int buf) { return tmem + (uint32_t)(buf * BN); };   // P overwrites columns 0-31 and 64-95
  const uint32_t tmem_O = tmem + (uint32_t)(NSB * BN);

  // per-thread state of the softmax threads (warps 2..9); declared here because the epilogue runs
  // after block-wide synchronisation points that all roles must reach together
  const int sw = warp >= 2 ? warp - 2 : 0;
  const int ch = sw >> 2;                        // which 64-key piece of every tile (= column half)
  const int quarter = warp & 3;                  // TMEM lanes this warp may touch
  const int row = quarter * 32 + lane;           // row inside the 128-row tile
  const int r_glob = tile_idx * RT + row;
  const bool row_valid = row < RT && r_glob < rows_total;
  const int node = row_valid ? r_glob / G : 0;
  const int gq = row_valid ? r_glob - node * G : 0;
  const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
  const int pair_bar = 2 + quarter;              // named barrier of the two warps that share rows
  float m_ref = -INFINITY, l_run = 0.f;
  if (warp >= 2 && ch == 0)   // read by the merge, after several block-wide barriers
    s_rowoff[row] = row_valid ? (((int64_t)b * N + node) * p.Hq + kvh * G + gq) * HD : -1ll;

  if (warp == 0) {
    // =========================== TMA producer ===============================================
    // K and V advance independently: whichever ring has a free buffer gets its next tile.
    int kt = kt0, vt = vt0;
    long long t_idle = clock64();
    bool ok = true;
    while (ok && (kt < T || vt < T)) {
      bool progress = false;
      if (kt < T) {
        const int st = kt % KST;
        int ready = 1;
        if (kt >= KST && lane == 0) ready = mbar_test(bar(B_SF + st), ((kt / KST) - 1) & 1) ? 1 : 0;
        ready = __shfl_sync(0xFFFFFFFFu, ready, 0);
        if (ready) {
          issue_tile(kt, true, pk_page, pk_base);
          ++kt;
          progress = true;
        }
      }
      if (vt < T) {
        const int st = vt % VST;
        int ready = 1;
        if (vt >= VST && lane == 0)
          ready = mbar_test(bar(B_VE + st), ((vt / VST) - 1) & 1) ? 1 : 0;
        ready = __shfl_sync(0xFFFFFFFFu, ready, 0);
        if (ready) {
          issue_tile(vt, false, pv_page, pv_base);
          ++vt;
          progress = true;
        }
      }
      if (progress) {
        t_idle = clock64();
      } else {
        int stop = 0;
        if (lane == 0) {
          if (*abort_flag) stop = 1;
          else if (clock64() - t_idle > wlim) { *abort_flag = 1; stop = 1; }
        }
        if (__shfl_sync(0xFFFFFFFFu, stop, 0)) ok = false;
      }
    }
  } else if (warp == 1) {
    // =========================== MMA issuer ===================================================
    if (lane == 0 && T > 0) {
      bool ok = mbar_wait(bar(B_Q), 0, abort_flag, wlim);
      tc_fence_after();
      // Descriptors are built once; inside the loops an operand's descriptor is a base plus a
      // constant (the address field counts 16-byte units and never carries out of its 14 bits).
      const uint64_t q_desc = smem_desc(sQ, 16, 1024);
      const uint64_t k_desc = smem_desc(sK, 16, 1024);
      const uint64_t v_desc = smem_desc(sV, kHalf, 1024);   // lbo: the other half of d
      auto issue_qk = [&](int t) -> bool {
        const int st = t % KST;
        if (!mbar_wait(bar(B_KF + st), (t / KST) & 1, abort_flag, wlim)) return false;
        tc_fence_after();
        const uint64_t kd = k_desc + (uint64_t)((st * kStage) >> 4);
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const uint32_t qo = (ks >> 2) * (kQTile / 2) + (ks & 3) * 32;
          const uint32_t ko = (ks >> 2) * kHalf + (ks & 3) * 32;
          umma_bf16(tmem_S(t % NSB), q_desc + (qo >> 4), kd + (ko >> 4), kIdescQK, ks > 0 ? 1u : 0u);
        }
        umma_commit(bar(B_SF + t % NSB));   // scores ready; this K buffer is free
        return true;
      };
      for (int t = 0; t < NSB && t < T && ok; ++t) ok = issue_qk(t);
      for (int t = 0; t < T && ok; ++t) {
        const int buf = t % NSB, st = t % VST;
        // both tests are issued together; the bounded waits follow only if one of them fails
        const bool p_in = mbar_test(bar(B_PF + buf), (t / NSB) & 1);
        const bool v_in = mbar_test(bar(B_VF + st), (t / VST) & 1);
        if (!p_in) ok = mbar_wait(bar(B_PF + buf), (t / NSB) & 1, abort_flag, wlim);
        if (ok && !v_in) ok = mbar_wait(bar(B_VF + st), (t / VST) & 1, abort_flag, wlim);
        if (!ok) break;
        tc_fence_after();
        const int n_kk = min(PPT, pc_end - (pc_begin + t * PPT)) * (PG / 16);   // a missing piece is skipped
        const uint64_t vd = v_desc + (uint64_t)((st * kStage) >> 4);
        // P of piece j of the tile sits in the first 32 columns of that piece's 64 score columns
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk)
          if (kk < n_kk)
            umma_bf16_ts(tmem_O, tmem_S(buf) + (kk >> 2) * 64 + (kk & 3) * 8, vd + (uint64_t)((kk * 2048) >> 4),
                         kIdescPV, (t > 0 || kk > 0) ? 1u : 0u);
        umma_commit(bar(B_PV + buf));   // O holds tile t
        umma_commit(bar(B_VE + st));    // this V buffer is free
        if (t + NSB < T) ok = issue_qk(t + NSB);
      }
    }
  } else {
    // =========================== softmax threads ==============================================
    // ancestor bitsets (row i of the tree's topology matrix), built while the first tiles are on
    // their way; the 256 threads meet at a named barrier of their own
    for (int i = tid - 64; i < N; i += kSoftmaxThreads) {
      uint32_t w[4] = {0, 0, 0, 0};
      int j = i;
      for (int hop = 0; hop < N && j >= 0; ++hop) {
        w[j >> 5] |= 1u << (j & 31);
        j = s_parent[j];
      }
      s_anc[i][0] = w[0]; s_anc[i][1] = w[1]; s_anc[i][2] = w[2]; s_anc[i][3] = w[3];
    }
    if (reporter && warp == 2) {  // one warp per sequence reports: block table of the context
      bool pbad = false;
      if (p.paged) {
        for (int pg = lane; pg < p_cache; pg += 32) {
          const int e = p.block_table[(int64_t)b * p.max_pages + pg];
          pbad |= (e < 0 || e >= p.n_pages);
        }
      }
      pbad = __any_sync(0xFFFFFFFFu, pbad);
      if (lane == 0 && pbad) atomicOr(p.tickets + 2 * b + 1, 1u);  // before this block's ticket
    }
    named_barrier(1, kSoftmaxThreads);

    // A wait that runs out raises the block's abort flag and sets `fail`; the thread then skips
    // the work but keeps walking through the named barriers it shares with its partner warp, and
    // both leave the loop together at the next exchange (a warp must never be left alone at a
    // named barrier, which has no time limit).
    bool fail = false;
    auto wait_all = [&](uint32_t barrier, uint32_t parity) {   // warp-uniform verdict
      if (fail) return;
      const bool w_ok = mbar_wait(barrier, parity, abort_flag, wlim);
      fail = !__all_sync(0xFFFFFFFFu, w_ok);
    };
    const bool warp_rows_valid = __all_sync(0xFFFFFFFFu, row_valid);
    // tiles [0, t_plain) of this block consist of two complete pieces of context: nothing to mask
    const int t_plain = max(0, (min(pc_end, L / PG) - pc_begin) / PPT);
    // The scores of a tile (this thread's 64) are fetched into registers while the previous tile's
    // P is on its way to tensor memory; they stay there until the tile is done, so a tile can be
    // redone against a new reference without another read.
    uint32_t sv[64];
    auto fetch_scores = [&](int t, int sbuf) {
      if (pc_begin + t * PPT + ch < pc_end && !fail) tmem_ld_x64(tmem_S(sbuf) + lane_addr + ch * 64, sv);
    };
    int buf = 0;
    uint32_t ph = 0;   // score buffer of tile t and the parity of its phase
    if (T > 0) {
      wait_all(bar(B_SF), 0);
      tc_fence_after();
      fetch_scores(0, 0);
    }
    for (int t = 0; t < T; ++t) {
      const int g0 = pc_begin + t * PPT;
      const int g = g0 + ch;
      const bool present = g < pc_end;
      // real keys in each piece of the tile, and the allowed columns of this thread's piece
      int valid[PPT] = {PG, PG};
      bool short_tile = false, need_mask = !warp_rows_valid;
      uint32_t allow0 = row_valid ? 0xFFFFFFFFu : 0u, allow1 = allow0;
      if (t >= t_plain) {
#pragma unroll
        for (int j = 0; j < PPT; ++j) {
          const int gj = g0 + j;
          if (gj >= pc_end) valid[j] = -1;                       // no such piece: P V skips it
          else if (gj < p_cache) valid[j] = min(PG, L - gj * PG);
          else valid[j] = min(PG, N - (gj - p_cache) * PG);
          short_tile |= (valid[j] >= 0 && valid[j] < PG);
        }
        need_mask = true;
        allow0 = allow1 = 0;
        if (present && row_valid) {
          if (g < p_cache) {
            const uint64_t bits = valid[ch] >= 64 ? ~0ull : ((1ull << valid[ch]) - 1ull);
            allow0 = (uint32_t)bits; allow1 = (uint32_t)(bits >> 32);
          } else {
            const int tp = g - p_cache;
            allow0 = s_anc[node][2 * tp]; allow1 = s_anc[node][2 * tp + 1];
          }
        }
      }
      if (present && !fail) {
        tmem_wait_ld();   // the scores of this tile
        if (need_mask) {  // columns that are not allowed become -inf
#pragma unroll
          for (int j = 0; j < 64; ++j) {
            const uint32_t wbits = (j < 32) ? allow0 : allow1;
            if (!((wbits >> (j & 31)) & 1u)) sv[j] = 0xFF800000u;
          }
        }
      }
      // One pass with the reference maximum as it stands: exponentiate, pack P and add up.  P goes
      // to tensor memory as soon as 32 keys are done: keys 64 ch + 32 h .. + 31 of the tile land in
      // columns 64 ch + 16 h .. + 15 of the score buffer (two bf16 per column), i.e. on top of
      // scores that this very thread has already taken.  No per-element maximum is tracked: a sum
      // of at most 2^8 proves that no probability exceeded 2^8, i.e. that the reference is still
      // good.  Otherwise (rare after the first tile; inf or NaN from an overflow also lands here)
      // the true maximum of the row is taken from the scores, the reference replaced, O rescaled
      // and the tile redone from the registers.  The two threads of a row decide together.
      float sum = 0.f;
      float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      auto exp_pass = [&]() {
        sum = 0.f;
        if (!present || fail) return;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float p0 = ex2(fmaf(__uint_as_float(sv[32 * h + 2 * j]), p.scale_log2, neg_m));
            const float p1 = ex2(fmaf(__uint_as_float(sv[32 * h + 2 * j + 1]), p.scale_log2, neg_m));
            sum += p0 + p1;
            pk[j] = pack_bf16(p0, p1);
          }
          tmem_st_x16(tmem_S(buf) + lane_addr + ch * 64 + h * 16, pk);
        }
      };
      if (t > 0) {
        exp_pass();
        // a row without a reference yet must take one as soon as it sees a score
        const bool suspect = !(sum <= kRowSumLimit) || (m_ref == -INFINITY && sum != 0.f);
        if (__any_sync(0xFFFFFFFFu, suspect) && lane == 0) *(volatile int*)&s_redo[sw] = t;
      }
      if (fail && lane == 0) *(volatile int*)&s_fail[sw] = 1;
      named_barrier(pair_bar, 64);
      if (*(volatile int*)&s_fail[sw] | *(volatile int*)&s_fail[sw ^ 4]) break;   // both warps see the same
      const bool redo = (t == 0) ||   // no reference yet
                        (*(volatile int*)&s_redo[sw] == t) || (*(volatile int*)&s_redo[sw ^ 4] == t);
      if (redo) {
        float mx = -INFINITY;
        if (present && !fail) {
#pragma unroll
          for (int j = 0; j < 64; ++j) mx = fmaxf(mx, __uint_as_float(sv[j]));
          mx *= p.scale_log2;   // scale > 0; -inf (no allowed key) stays -inf
        }
        s_xch[ch][row] = mx;
        named_barrier(pair_bar, 64);
        mx = fmaxf(mx, s_xch[ch ^ 1][row]);
        const bool need = mx > m_ref;
        if (t > 0) {  // O must be at rest: P V of the previous tile has completed
          wait_all(bar(B_PV + (t - 1) % NSB), ((t - 1) / NSB) & 1);
          tc_fence_after();
        }
        const float alpha = need ? ex2(m_ref - mx) : 1.0f;  // ex2(-inf) = 0
        if (need) { m_ref = mx; l_run *= alpha; }
        if (t > 0 && !fail) {
          if (present) tmem_wait_st();   // this thread's stores of the first pass, before it touches O
#pragma unroll 1
          for (int cc = 0; cc < 64; cc += 32) {
            uint32_t ov[32];
            tmem_ld_x32(tmem_O + lane_addr + ch * 64 + cc, ov);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
            tmem_st_x32(tmem_O + lane_addr + ch * 64 + cc, ov);
          }
          tmem_wait_st();
        }
        neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
        exp_pass();
      }
      l_run += sum;
      // the next tile's scores travel to the registers while this tile's P travels the other way
      const int nbuf = (buf == NSB - 1) ? 0 : buf + 1;
      const uint32_t nph = (buf == NSB - 1) ? ph ^ 1u : ph;
      if (t + 1 < T) {
        wait_all(bar(B_SF + nbuf), nph);
        tc_fence_after();
        fetch_scores(t + 1, nbuf);
      }
      if (present && !fail) tmem_wait_st();

      if (short_tile) {
        // Rows of a V piece beyond its real keys hold whatever lies behind them in memory; their
        // probabilities are exactly 0, but 0 * NaN would poison O: clear them.
        const int vst = t % VST;
        wait_all(bar(B_VF + vst), (t / VST) & 1);
        if (!fail) {
          uint8_t* vt = sV_gen + vst * kStage;
          const int me = tid - 64;   // 0 .. 255 among the softmax threads
          constexpr int kHalves = 2;   // halves of the head dimension
#pragma unroll
          for (int j = 0; j < PPT; ++j) {
            if (valid[j] < 0) continue;
            const int per_half = (PG - valid[j]) * 8;  // 16-byte chunks per half of the head dimension
            for (int cidx = me; cidx < kHalves * per_half; cidx += kSoftmaxThreads) {
              const int half = cidx / per_half, rem = cidx - half * per_half;
              const int vr = j * PG + valid[j] + (rem >> 3), chk = rem & 7;
              *reinterpret_cast<uint4*>(vt + half * kHalf + vr * 128 + chk * 16) = make_uint4(0, 0, 0, 0);
            }
          }
          fence_async_smem();   // cleared V rows visible to the tensor core's reads
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !fail) mbar_arrive(bar(B_PF + buf));
      buf = nbuf;
      ph = nph;
    }

    if (!fail && !*abort_flag && T > 0) {  // the last P V has landed in O
      const bool w_ok = mbar_wait(bar(B_PV + (T - 1) % NSB), ((T - 1) / NSB) & 1, abort_flag, wlim);
      (void)__all_sync(0xFFFFFFFFu, w_ok);
    }
  }

  // ---- every role meets here: all MMAs and copies of this block are complete -----------------
  __syncwarp();
  if (*abort_flag) {
    if (warp == 0 && lane == 0) {
      // TMA copies that were issued land on their own; wait for the newest phase of each stage
      for (int i = max(0, issued_k - KST); i < issued_k; ++i) mbar_drain(bar(B_KF + i % KST), (i / KST) & 1);
      for (int i = max(0, issued_v - VST); i < issued_v; ++i) mbar_drain(bar(B_VF + i % VST), (i / VST) & 1);
    }
    if (warp == 2 && lane == 0 && T > 0) mbar_drain(bar(B_Q), 0);
    if (warp == 1 && lane == 0) {
      umma_commit(bar(B_DR));
      mbar_drain(bar(B_DR), 0);  // completes when every MMA issued so far has finished
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const bool aborted = *abort_flag != 0;
  // the ticket is taken here and looked at when the block leaves, so that its round trip is hidden
  // behind the epilogue (no wait can run out after this point)
  unsigned my_ticket = 0;
  if (tid == 0) my_ticket = report(aborted ? 2u : 0u);
  const int n_src = p.splits;   // accumulators that cover one output row
  const float kLn2 = 0.6931471805599453f;
  // staging area for the merge: O as fp16 [128 rows][128], every row scaled by a power of two that
  // puts its largest magnitude in [2^13, 2^14) (half the bytes of fp32 through distributed shared
  // memory, at a relative rounding error of 2^-11, far below that of the bf16 output; the scale
  // travels with the row's maximum and sum).  The 16-byte chunk c of row r is stored at chunk
  // (c ^ (r & 15)) so that row-per-thread writes and row-per-warp reads are both conflict free.
  // The area reuses the tile memory, which nothing reads any more.
  uint8_t* const sO = smem_raw + (sQ - smem_u32(smem_raw));

  if (!aborted && warp >= 2) {
    // the row's two threads add up their sums (and, for staging, agree on the row's scale)
    float amax = 0.f;
    if (n_src > 1 && T > 0) {
#pragma unroll 1
      for (int cc = 0; cc < 64; cc += 32) {
        uint32_t ov[32];
        tmem_ld_x32(tmem_O + lane_addr + ch * 64 + cc, ov);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(__uint_as_float(ov[j])));
      }
    }
    s_xch[ch][row] = l_run;
    s_xch2[ch][row] = amax;
    named_barrier(1, kSoftmaxThreads);
    const float l_tot = l_run + s_xch[ch ^ 1][row];
    amax = fmaxf(amax, s_xch2[ch ^ 1][row]);
    if (n_src == 1) {
      // only accumulator of these rows: normalise and store this thread's 64 columns
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      uint16_t* dst = p.out + (((int64_t)b * N + node) * p.Hq + kvh * G + gq) * HD + ch * 64;
#pragma unroll 1
      for (int cc = 0; cc < 64; cc += 32) {
        uint32_t ov[32];
        tmem_ld_x32(tmem_O + lane_addr + ch * 64 + cc, ov);
        tmem_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(ov[q4 * 8 + 0]) * inv, __uint_as_float(ov[q4 * 8 + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(ov[q4 * 8 + 2]) * inv, __uint_as_float(ov[q4 * 8 + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(ov[q4 * 8 + 4]) * inv, __uint_as_float(ov[q4 * 8 + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(ov[q4 * 8 + 6]) * inv, __uint_as_float(ov[q4 * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + cc + q4 * 8) = v;
          }
        }
      }
      if (p.lse != nullptr && row_valid && ch == 0)
        p.lse[((int64_t)b * N + node) * p.Hq + kvh * G + gq] = (m_ref + log2f(l_tot)) * kLn2;
    } else {
      uint8_t* orow = sO + (size_t)row * (HD * 2);
      // scale 2^lc with amax * 2^lc in [2^13, 2^14); lc is clamped so that the scale and its
      // inverse are normal numbers (a zero row keeps zeros, inf or NaN stay what they are)
      const int biased = (int)((__float_as_uint(amax) >> 23) & 255u);
      const int lc = max(-100, min(100, 140 - biased));
      const float cscale = __uint_as_float((uint32_t)(127 + lc) << 23);
      const float cinv = __uint_as_float((uint32_t)(127 - lc) << 23);
#pragma unroll 1
      for (int cc = 0; cc < 64; cc += 32) {
        uint32_t ov[32];
        if (T > 0) {
          tmem_ld_x32(tmem_O + lane_addr + ch * 64 + cc, ov);
          tmem_wait_ld();
        } else {  // a block without tiles contributes zeros with weight zero
#pragma unroll
          for (int j = 0; j < 32; ++j) ov[j] = 0u;
        }
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t h[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const __half2 v = __floats2half2_rn(__uint_as_float(ov[q4 * 8 + 2 * e]) * cscale,
                                                __uint_as_float(ov[q4 * 8 + 2 * e + 1]) * cscale);
            h[e] = *reinterpret_cast<const uint32_t*>(&v);
          }
          const int chunk = ((ch * 64 + cc) >> 3) + q4;
          *reinterpret_cast<uint4*>(orow + ((chunk ^ (row & 15)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
        }
      }
      if (ch == 0) s_ml[row] = make_float4(T > 0 ? m_ref : -INFINITY, T > 0 ? l_tot : 0.f, cinv, 0.f);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CS == 1) {  // a block that is its own cluster
    if (warp == 1) release_tmem();
    if (tid == 0) publish(my_ticket);
    return;
  }

  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();  // every block's staging area is complete and its MMAs are done (also reached by an aborted block)
  if (n_src > 1 && !aborted) {
    // ---- merge across the key splits through distributed shared memory: split j finalises rows
    //      [j, j+1) * 128 / splits of the tile; source q of a row lives in cluster rank q ----
    const int per_rank = BM / p.splits;
    const int first_row = split * per_rank;
    {
      const uint32_t sO_addr = smem_u32(sO), ml_addr = smem_u32(&s_ml[0]);
      switch (n_src) {
        case 2: merge_rows<2>(sO_addr, ml_addr, split, first_row, per_rank, warp, lane, s_rowoff, p.out, p.lse); break;
        case 4: merge_rows<4>(sO_addr, ml_addr, split, first_row, per_rank, warp, lane, s_rowoff, p.out, p.lse); break;
        default: merge_rows<8>(sO_addr, ml_addr, split, first_row, per_rank, warp, lane, s_rowoff, p.out, p.lse); break;
      }
    }
  }
  cluster.sync();  // no block may leave while a peer still reads its shared memory
  if (warp == 1) release_tmem();
  if (tid == 0) publish(my_ticket);
}

// ------------------------------------------------------------------------------------ host side
// bf16 tensor [rows][heads][128]; box = 64 elements x box_heads x box_rows, 128-byte swizzle
bool make_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t heads, uint32_t box_heads,
              uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)HD, heads, rows};
  const cuuint64_t strides[2] = {(cuuint64_t)HD * 2, (cuuint64_t)HD * 2 * heads};
  const cuuint32_t box[3] = {64, box_heads, box_rows};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same tensor seen as [rows][heads][2 halves of d][64]: a box of 64 x box_rows x 2 x 1 in the
// order (d, row, half, head) lands in shared memory as [half][row][64], the layout of a K or V
// stage, so a tile of 128 neighbouring rows is one copy instead of four.
bool make_map_halves(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t heads, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {64, rows, 2, heads};
  const cuuint64_t strides[3] = {(cuuint64_t)HD * 2 * heads, 128, (cuuint64_t)HD * 2};
  const cuuint32_t box[4] = {64, box_rows, 2, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int row_tiles(const clv_shape& s) {
  const int G = s.n_q_heads / s.n_kv_heads;
  return (s.n_nodes + BM / G - 1) / (BM / G);   // row tiles of BM / G whole nodes
}

}  // namespace

bool tc_attn_supported(const clv_shape& s, const clv_kv_cache& c) {
  const int G = s.n_q_heads / s.n_kv_heads;
  if (G > BM) return false;                            // a row tile must hold at least one whole node
  const int64_t cache_rows = c.paged ? (int64_t)c.n_pages * CLV_PAGE_SIZE : (int64_t)s.batch * c.cap_tokens;
  if (cache_rows >= (1ll << 31) || (int64_t)s.batch * s.n_nodes >= (1ll << 31)) return false;
  return encode_fn() != nullptr;
}

AttnPlan tc_attn_plan(const clv_shape& s, int max_ctx_len) {
  AttnPlan pl;
  pl.m_tiles = row_tiles(s);
  const int64_t ctas = (int64_t)s.batch * s.n_kv_heads * pl.m_tiles;
  const int key_tiles = (max_ctx_len > 0 ? (max_ctx_len + BN - 1) / BN : 0) + (s.n_nodes + BN - 1) / BN;
  // The key axis is split over a thread-block cluster (merged through distributed shared memory):
  // a power of two up to the portable cluster size of 8 that keeps the grid within one block per
  // SM and leaves every block at least two key tiles.
  int splits = 1;
  while (splits * 2 <= 8 && ctas * (splits * 2) <= sm_count() && key_tiles / (splits * 2) >= 2) splits *= 2;
  pl.splits = splits;
  pl.tickets = 0;
  pl.scratch_bytes = 0;  // nothing goes through global memory
  return pl;
}

cudaError_t launch_tree_attn_tc(const AttnPlan& plan, const clv_shape& s, const clv_kv_cache& c,
                                const void* q, const void* k_tree, const void* v_tree,
                                const int32_t* parent, const int32_t* ctx_len, float scale, void* out,
                                float* lse, int32_t* status, unsigned* tickets, void* scratch,
                                cudaStream_t stream) {
  (void)scratch;
  const int G = s.n_q_heads / s.n_kv_heads;
  static OncePerDevice once;
  cudaError_t e0 = run_once_per_device(once, [] {
    return cudaFuncSetAttribute(tree_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)Cfg::kSmem);
  });
  if (e0 != cudaSuccess) return e0;
  alignas(64) CUtensorMap tm_q, tm_kc, tm_vc, tm_kt, tm_vt, tm_kc2, tm_vc2;
  const uint64_t cache_rows = c.paged ? (uint64_t)c.n_pages * CLV_PAGE_SIZE : (uint64_t)s.batch * c.cap_tokens;
  const uint64_t tree_rows = (uint64_t)s.batch * s.n_nodes;
  if (!make_map(&tm_q, q, tree_rows, s.n_q_heads, G, BM / G) ||
      !make_map(&tm_kc, c.k, cache_rows, s.n_kv_heads, 1, PG) ||
      !make_map(&tm_vc, c.v, cache_rows, s.n_kv_heads, 1, PG) ||
      !make_map(&tm_kt, k_tree, tree_rows, s.n_kv_heads, 1, PG) ||
      !make_map(&tm_vt, v_tree, tree_rows, s.n_kv_heads, 1, PG))
    return cudaErrorInvalidValue;
  // whole-tile copies: only if the driver accepts the 4-D view (else the piece-wise copies do it all)
  const bool pair_boxes = make_map_halves(&tm_kc2, c.k, cache_rows, s.n_kv_heads, BN) &&
                          make_map_halves(&tm_vc2, c.v, cache_rows, s.n_kv_heads, BN);
  if (!pair_boxes) { tm_kc2 = tm_kc; tm_vc2 = tm_vc; }

  Params p;
  p.pair_boxes = pair_boxes ? 1 : 0;
  p.block_table = c.block_table;
  p.parent = parent;
  p.ctx_len = ctx_len;
  p.out = static_cast<uint16_t*>(out);
  p.lse = lse;
  p.status = status;
  const int64_t clusters = (int64_t)s.batch * s.n_kv_heads * plan.m_tiles;
  p.B = s.batch; p.N = s.n_nodes; p.Hq = s.n_q_heads; p.Hkv = s.n_kv_heads; p.G = G;
  p.paged = c.paged; p.cap_tokens = c.cap_tokens; p.n_pages = c.n_pages; p.max_pages = c.max_pages_per_seq;
  p.tiles = plan.m_tiles;
  p.splits = plan.splits;
  p.longest_first = (clusters * plan.splits > sm_count() && s.batch > 1 && s.batch <= 256) ? 1 : 0;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.wait_limit = wait_limit_cycles();
  p.tickets = tickets;
  p.blocks_per_seq = s.n_kv_heads * plan.m_tiles * plan.splits;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(clusters * plan.splits), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::kSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;  // the blocks that share one row tile's keys
  attr[0].val.clusterDim.x = (unsigned)plan.splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up overlaps the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel, tm_q, tm_kc, tm_vc, tm_kt, tm_vt, tm_kc2, tm_vc2, p);
}

}  // namespace clv
