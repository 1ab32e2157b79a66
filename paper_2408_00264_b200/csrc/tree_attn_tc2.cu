// Tree attention (Sec. 2.1) for (sequence, kv head) units of many query rows (four or more row
// tiles of 128): one thread block owns TWO row tiles, so that every K/V tile staged in shared
// memory serves 256 rows (half the shared-memory fill per row of the one-tile kernel, and half as
// many blocks).  tcgen05.mma with accumulators in tensor memory, K/V/Q tiles staged by TMA into
// 128-byte-swizzled shared memory; a key tile is 128 keys, loaded as 64-key pieces (the page size
// of a paged cache); K and V travel through separate rings so that a K buffer is refilled as
// soon as its Q K^T is done.
// Roles: warp 0 = TMA producer, warp 1 = MMA issuer (also owns the TMEM allocation), warps 2-5 and
// 6-9 = two softmax groups of 128 threads, one thread per query row; group s works on row tile s
// and both consume every K/V tile.  Tensor memory: one score buffer and one output accumulator
// per row tile.  Per row tile and key tile:  S = Q K^T  ->  the softmax thread reads its row of S,
// masks, exponentiates against a lazily updated reference maximum, writes P (bf16) back over the
// scores  ->  O += P V (A operand from tensor memory).  While one row tile is in its softmax the
// tensor core works for the other.  Split-KV, masking and the bounded waits are those of the
// one-tile kernel: the blocks that share a pair of row tiles form a thread-block cluster and merge
// through distributed shared memory; masked scores are replaced, not added to; a wait that runs
// out makes the block drain, release tensor memory and report CLV_ERR_TIMEOUT.
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
constexpr int BM = 128;                // rows per MMA / per slot
constexpr int kThreads = 320;
constexpr uint32_t kQTile = BM * HD * 2;      // 32 KB: two [128 rows][64 d] swizzled halves
constexpr uint32_t kPiece = PG * 64 * 2;       // 8 KB: [64 keys][64 d] swizzled, one TMA box
constexpr uint32_t kTmemCols = 512;
constexpr float kRowSumLimit = 256.0f;        // a row of P may sum to 2^8 before the reference is replaced

constexpr int MT = 2;                                    // row tiles per block
struct Cfg {
  static constexpr int BN = 128;                         // keys per tile
  static constexpr int kStagesK = 2;                     // depth of the K ring
  static constexpr int kStagesV = 2;                     // depth of the V ring
  static constexpr uint32_t kTile = BN * HD * 2;         // bytes of one K (or V) tile
  static constexpr uint32_t kSmem = MT * kQTile + (kStagesK + kStagesV) * kTile + 1024;
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
  int row_ctas;    // thread blocks along the row axis per (sequence, kv head)
  int splits;      // thread blocks along the key axis = cluster size (1, 2, 4 or 8)
  float scale_log2;
  long long wait_limit;   // SM cycles a bounded wait may last
  unsigned* tickets;      // per sequence: [2b] blocks that have finished, [2b+1] error bits; zero between calls
  int blocks_per_seq;
};

constexpr uint32_t kIdescPV = make_idesc(BM, HD, true);   // O[128 x 128] += P[128 x 16k] V[16k x 128]

// Distributed shared memory: address of the same variable in block `rank` of the cluster, and a
// 16-byte load from it.  The loads are volatile asm so that a batch of them is issued back to back
// (all in flight together) before the first result is used.
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 dsmem_ld16(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(addr));
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

__device__ __forceinline__ uint2 dsmem_ld8u(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared::cluster.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 half2_bits_to_float2(uint32_t u) {
  return __half22float2(*reinterpret_cast<const __half2*>(&u));
}

// Final combination of NSRC accumulators per output row, for the rows [k_begin, k_end) that this
// block finalises.  The staged accumulators are fp16 (each row scaled by a power of two of its
// own, which the weight undoes), 256 bytes per row.  One warp takes 32 / NSRC rows at a time (32
// remote 8-byte loads in flight per lane); lane j owns output columns 4j .. 4j+3.  w[] holds the
// normalised weights divided by the rows' scales.
template <int NSRC>
__device__ __forceinline__ void merge_rows(uint32_t sO_addr, const float* w, int first_row, int per_rank,
                                           int rot, int warp, int lane, int tile_base, int RT, int rows_total, int G,
                                           int64_t seq_row0, int Hq, int head0, uint16_t* out) {
  constexpr int RB = 32 / NSRC;
  for (int k0 = warp * RB; k0 < per_rank; k0 += RB * (kThreads / 32)) {
    uint2 x[RB * NSRC];
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      const int k = min(k0 + u, per_rank - 1);
      const int rr = first_row + k, tile = rr / BM, trow = rr % BM;
      const uint32_t off = (uint32_t)(trow * (HD * 2) + (((lane >> 1) ^ (trow & 15)) << 4) + ((lane & 1) << 3));
#pragma unroll
      for (int j = 0; j < NSRC; ++j) {
        const int q = (j + rot) & (NSRC - 1);  // every block starts at a different peer
        const int qc = q, qs = tile;
        x[u * NSRC + j] = dsmem_ld8u(dsmem_addr(sO_addr + (uint32_t)(qs * BM * HD * 2) + off, qc));
      }
    }
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      if (k0 + u >= per_rank) continue;
      const int k = k0 + u;
      const int rr = first_row + k, tile = rr / BM, trow = rr % BM;
      const int rg = (tile_base + tile) * RT + trow;
      if (trow >= RT || rg >= rows_total) continue;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int j = 0; j < NSRC; ++j) {
        const float wq = w[k * NSRC + ((j + rot) & (NSRC - 1))];
        const float2 lo = half2_bits_to_float2(x[u * NSRC + j].x), hi = half2_bits_to_float2(x[u * NSRC + j].y);
        acc.x += wq * lo.x; acc.y += wq * lo.y; acc.z += wq * hi.x; acc.w += wq * hi.y;
      }
      const int onode = rg / G, ogq = rg - onode * G;
      uint16_t* dst = out + ((seq_row0 + onode) * Hq + head0 + ogq) * HD + lane * 4;
      *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    }
  }
}

// ------------------------------------------------------------------------------------ kernel
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_tc2_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc,
                    const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kt,
                    const __grid_constant__ CUtensorMap tm_vt, const Params p) {
  constexpr int BN = Cfg::BN;          // keys per tile
  constexpr int PPT = BN / PG;             // 64-key pieces per tile
  constexpr int KST = Cfg::kStagesK, VST = Cfg::kStagesV;
  constexpr uint32_t kTile = Cfg::kTile;
  constexpr uint32_t kHalf = kTile / 2;    // one 64-wide half of the head dimension: [BN keys][64 d]
  constexpr uint32_t kIdescQK = make_idesc(BM, BN, false);  // S[128 x BN] = Q[128 x 16k] K[BN x 16k]^T
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t s_anc[CLV_MAX_NODES][4];
  __shared__ int s_parent[CLV_MAX_NODES];
  __shared__ __align__(8) unsigned long long s_bar[2 * KST + 2 * VST + 8];
  __shared__ int s_tile_ok[VST];  // paged cache: every page of the tile in this V stage is valid
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ float4 s_ml[2][BM];   // (reference maximum, row sum, 1 / staging scale, -) of both slots, for the merge
  __shared__ float s_w[2 * BM];    // merge: normalised weight of every (row of this rank, source)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x / p.row_ctas, row_cta = blockIdx.x - unit * p.row_ctas;
  const int split = blockIdx.y;
  int b = unit / p.Hkv;
  const int kvh = unit - b * p.Hkv;
  const int N = p.N, G = p.G, rows_total = G * N;
  // A row tile holds whole nodes: BM / G of them, i.e. RT = (BM / G) * G of its 128 rows (all 128
  // when G divides 128); the remaining rows of the tile are idle.
  const int RT = (BM / G) * G;
  // ---- set-up that reads no global memory: barriers, tensor memory, descriptor prefetch.  The
  //      kernel is launched with programmatic stream serialisation, so this part may run while the
  //      previous kernel of the stream drains; everything after the grid dependency wait sees that
  //      kernel's results.
  constexpr int NRING = 2 * KST + 2 * VST;
  const uint32_t bar0 = smem_u32(&s_bar[0]);
  if (tid == 0) {
    for (int i = 0; i < NRING; ++i) mbar_init(bar0 + 8u * i, 1);                 // K/V rings
    mbar_init(bar0 + 8u * (NRING), 1);                                           // Q
    for (int s2 = 0; s2 < 2; ++s2) {
      mbar_init(bar0 + 8u * (NRING + 1 + s2), 1);                                // S ready
      mbar_init(bar0 + 8u * (NRING + 3 + s2), BM);                               // P ready
      mbar_init(bar0 + 8u * (NRING + 5 + s2), 1);                                // P V done
    }
    mbar_init(bar0 + 8u * (NRING + 7), 1);                                       // drain
    s_abort = 0;
    fence_barrier_init();
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(&s_tmem), kTmemCols);
  if (tid == 64) {
    tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_kc); tma_prefetch_desc(&tm_vc);
    tma_prefetch_desc(&tm_kt); tma_prefetch_desc(&tm_vt);
  }
  cudaGridDependencySynchronize();

  if (p.longest_first) {
    // More blocks than SMs and contexts of different lengths (ragged batch): hand the sequences
    // out longest first, so that the block scheduler packs the short ones into the gaps.  Block
    // group `b` takes the sequence whose length has rank b (ties by index); every thread ranks
    // at most one sequence.
    __shared__ int s_seq;
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

  // ---- per-sequence checks: everybody reads parent[] and the context length; the one block-wide
  //      synchronisation below publishes them together with the set-up above --------------------
  const int L = p.ctx_len[b];
  bool bad = false;
  for (int i = tid; i < N; i += kThreads) {
    const int par = p.parent[(int64_t)b * N + i];
    s_parent[i] = par;
    bad |= (par < -1 || par >= i);
  }
  bad |= (L < 0);
  const int p_cache = L > 0 ? (L + PG - 1) / PG : 0;  // 64-key pieces (pages) of the context
  if (p.paged) bad |= (p_cache > p.max_pages);
  else bad |= (L > p.cap_tokens);
  tc_fence_before();
  const int seq_bad = __syncthreads_or(bad ? 1 : 0);  // same verdict in every block of the sequence
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const bool reporter = (row_cta == 0 && split == 0 && kvh == 0);
  // status[b] is written once, by whichever block of the sequence finishes last: every block adds
  // its error bits (1 malformed input, 2 a wait ran out) to the sequence's word in the workspace
  // and then takes a ticket; the holder of the last ticket turns the bits into the status code and
  // leaves both words zero for the next call.  So no verdict can be overwritten by a later "fine".
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
  if (seq_bad) {  // the whole cluster leaves together; nothing has been issued yet
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    if (tid == 0) publish(report(1u));
    return;
  }

  // ---- tile range and per-slot rounds -------------------------------------------------------
  // The key axis is cut in 64-key pieces: p_cache pieces of context, then the tree's own pieces.
  // A block takes a contiguous range of pieces (so the split balances to one piece) and walks it
  // in tiles of PPT pieces; a tile may end early or mix context and tree pieces.
  const int p_total = p_cache + (N + PG - 1) / PG;
  const int pc_begin = (int)((int64_t)split * p_total / p.splits);
  const int pc_end = (int)((int64_t)(split + 1) * p_total / p.splits);
  const int n_tiles = (pc_end - pc_begin + PPT - 1) / PPT;
  const int rounds0 = n_tiles, rounds1 = n_tiles;   // both row tiles take every key tile

  // ---- shared memory carve-up (1024-byte aligned tiles for the 128-byte swizzle) ------------
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem_base;
  const uint32_t sK = sQ + MT * kQTile;      // ring of KST K tiles
  const uint32_t sV = sK + KST * kTile;      // ring of VST V tiles
  uint8_t* const sV_gen = smem_raw + (sV - smem_u32(smem_raw));

  auto bar_k_full = [&](int st) { return bar0 + 8u * st; };
  auto bar_k_empty = [&](int st) { return bar0 + 8u * (KST + st); };
  auto bar_v_full = [&](int st) { return bar0 + 8u * (2 * KST + st); };
  auto bar_v_empty = [&](int st) { return bar0 + 8u * (2 * KST + VST + st); };
  const uint32_t bar_q = bar0 + 8u * NRING;
  auto bar_s_full = [&](int s) { return bar0 + 8u * (NRING + 1 + s); };
  auto bar_p_full = [&](int s) { return bar0 + 8u * (NRING + 3 + s); };
  auto bar_pv_done = [&](int s) { return bar0 + 8u * (NRING + 5 + s); };
  const uint32_t bar_drain = bar0 + 8u * (NRING + 7);

  volatile int* abort_flag = &s_abort;
  const long long wlim = p.wait_limit;
  // columns: S of slot s at BN s (P, two bf16 per column, overwrites its first BN/2 columns once
  // the scores have been read); O of slot s at 2 BN + 128 s
  auto tmem_S = [&](int s) { return tmem + (uint32_t)(s * BN); };
  auto tmem_P = [&](int s) { return tmem + (uint32_t)(s * BN); };
  auto tmem_O = [&](int s) { return tmem + (uint32_t)(2 * BN + s * HD); };

  int issued_k = 0, issued_v = 0;  // producer bookkeeping for the drain

  // per-thread state of the softmax groups (warps 2..9); declared here because the epilogue runs
  // after block-wide synchronisation points that all roles must reach together
  const int slot = warp >= 2 ? (warp - 2) >> 2 : 0;
  const int quarter = warp & 3;                  // TMEM lanes this warp may touch
  const int row = quarter * 32 + lane;           // row inside the 128-row tile
  const int my_rounds = slot == 0 ? rounds0 : rounds1;
  const int r_glob = (row_cta * MT + slot) * RT + row;
  const bool row_valid = row < RT && r_glob < rows_total;
  const int node = row_valid ? r_glob / G : 0;
  const int gq = row_valid ? r_glob - node * G : 0;
  const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
  float m_ref = -INFINITY, l_run = 0.f;

  if (warp == 0) {
    // =========================== TMA producer ===============================================
    if (n_tiles > 0) {
      int page_cache = 0;   // lane j: pool page of context piece (page_base + j)
      int page_base = -64;
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int ks = i % KST, vs = i % VST;
        const int g0 = pc_begin + i * PPT;  // first piece of this tile
        if (p.paged && g0 < p_cache && g0 + PPT > page_base + 32) {  // warp-uniform refill
          page_base = g0;
          const int pc = g0 + lane;
          page_cache = (pc < p_cache) ? p.block_table[(int64_t)b * p.max_pages + pc] : 0;
        }
        int row0[PPT];          // first source row of each piece, -1: piece not present
        bool is_tree[PPT];
        int tile_ok = 1;
#pragma unroll
        for (int j = 0; j < PPT; ++j) {
          const int g = g0 + j;
          int pg = __shfl_sync(0xFFFFFFFFu, page_cache, (g - page_base) & 31);
          is_tree[j] = g >= p_cache;
          if (g >= pc_end) {
            row0[j] = -1;
          } else if (is_tree[j]) {
            row0[j] = b * N + (g - p_cache) * PG;
          } else if (p.paged) {
            if (pg < 0 || pg >= p.n_pages) { tile_ok = 0; pg = 0; }  // flagged by the reporter; masked
            row0[j] = pg * PG;
          } else {
            row0[j] = b * p.cap_tokens + g * PG;
          }
        }
        if (lane == 0) {
          int n_pieces = 0;
#pragma unroll
          for (int j = 0; j < PPT; ++j) n_pieces += row0[j] >= 0;
          const uint32_t bytes = (uint32_t)n_pieces * 2u * kPiece;  // both halves of the head dim
          if (i >= KST) ok = mbar_wait(bar_k_empty(ks), ((i / KST) - 1) & 1, abort_flag, wlim);
          if (ok) {
            mbar_expect_tx(bar_k_full(ks), bytes);
#pragma unroll
            for (int j = 0; j < PPT; ++j) {
              if (row0[j] < 0) continue;
              const CUtensorMap* mk = is_tree[j] ? &tm_kt : &tm_kc;
              tma_load_3d(sK + ks * kTile + j * kPiece, mk, 0, kvh, row0[j], bar_k_full(ks));
              tma_load_3d(sK + ks * kTile + kHalf + j * kPiece, mk, 64, kvh, row0[j], bar_k_full(ks));
            }
            issued_k = i + 1;
            if (i >= VST) ok = mbar_wait(bar_v_empty(vs), ((i / VST) - 1) & 1, abort_flag, wlim);
          }
          if (ok) {
            s_tile_ok[vs] = tile_ok;  // read by the softmax threads after this V barrier completes
            mbar_expect_tx(bar_v_full(vs), bytes);
#pragma unroll
            for (int j = 0; j < PPT; ++j) {
              if (row0[j] < 0) continue;
              const CUtensorMap* mv = is_tree[j] ? &tm_vt : &tm_vc;
              tma_load_3d(sV + vs * kTile + j * kPiece, mv, 0, kvh, row0[j], bar_v_full(vs));
              tma_load_3d(sV + vs * kTile + kHalf + j * kPiece, mv, 64, kvh, row0[j], bar_v_full(vs));
            }
            issued_v = i + 1;
          }
        }
        ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
      }
    }
  } else if (warp == 1) {
    // =========================== MMA issuer ===================================================
    if (lane == 0 && n_tiles > 0) {
      bool ok = mbar_wait(bar_q, 0, abort_flag, wlim);
      tc_fence_after();
      auto local_tile = [&](int s, int r) { (void)s; return r; };
      // Descriptors are built once; inside the loops an operand's descriptor is a base plus a
      // constant (the address field counts 16-byte units and never carries out of its 14 bits).
      const uint64_t q_desc = smem_desc(sQ, 16, 1024);
      const uint64_t k_desc = smem_desc(sK, 16, 1024);
      const uint64_t v_desc = smem_desc(sV, kHalf, 1024);
      auto issue_qk = [&](int s, int r) -> bool {
        const int i = local_tile(s, r), st = i % KST;
        // with two row tiles, slot 1 uses the K tile that slot 0 has just waited for
        if (s == 0) {
          if (!mbar_wait(bar_k_full(st), (i / KST) & 1, abort_flag, wlim)) return false;
          tc_fence_after();
        }
        const uint64_t qd = q_desc + (uint64_t)((s * kQTile) >> 4);
        const uint64_t kd = k_desc + (uint64_t)((st * kTile) >> 4);
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const uint32_t qo = (ks >> 2) * (kQTile / 2) + (ks & 3) * 32;
          const uint32_t ko = (ks >> 2) * kHalf + (ks & 3) * 32;
          umma_bf16(tmem_S(s), qd + (qo >> 4), kd + (ko >> 4), kIdescQK, ks > 0 ? 1u : 0u);
        }
        umma_commit(bar_s_full(s));
        if (s == 1) umma_commit(bar_k_empty(st));  // last reader of this K buffer
        return true;
      };
      const int rounds[2] = {rounds0, rounds1};
      for (int s = 0; s < 2 && ok; ++s)
        if (rounds[s] > 0) ok = issue_qk(s, 0);
      for (int r = 0; r < rounds0 && ok; ++r) {
        for (int s = 0; s < 2 && ok; ++s) {
          if (r >= rounds[s]) continue;
          ok = mbar_wait(bar_p_full(s), r & 1, abort_flag, wlim);
          if (!ok) break;
          const int i = local_tile(s, r), st = i % VST;
          if (s == 0) {  // likewise the V tile
            ok = mbar_wait(bar_v_full(st), (i / VST) & 1, abort_flag, wlim);
            if (!ok) break;
          }
          tc_fence_after();
          const uint64_t vd = v_desc + (uint64_t)((st * kTile) >> 4);
#pragma unroll
          for (int kk = 0; kk < BN / 16; ++kk) {
            umma_bf16_ts(tmem_O(s), tmem_P(s) + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), kIdescPV,
                         (r > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(bar_pv_done(s));
          if (s == 1) umma_commit(bar_v_empty(st));  // last reader of this V buffer
          if (r + 1 < rounds[s]) ok = issue_qk(s, r + 1);
        }
      }
    }
  } else {
    // =========================== softmax groups ===============================================
    constexpr int NH = BN / 64;   // the row of S is taken in 64-column halves (register budget)
    const int rounds = my_rounds;
    bool ok = true;
    if (warp == 2 && n_tiles > 0) {  // the Q tile(s): issued here so that the producer starts with K/V
      if (lane == 0) {
        mbar_expect_tx(bar_q, (uint32_t)(MT * RT * HD * 2));   // the boxes hold RT rows of a tile
        const int nodes_per_tile = BM / G;
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          const int node0 = b * N + (row_cta * MT + m) * nodes_per_tile;
          tma_load_3d(sQ + m * kQTile, &tm_q, 0, kvh * G, node0, bar_q);
          tma_load_3d(sQ + m * kQTile + kQTile / 2, &tm_q, 64, kvh * G, node0, bar_q);
        }
      }
    }
    // ancestor bitsets (row i of the tree's topology matrix), built by the softmax warps while
    // the first tiles are on their way; the 256 threads meet at a named barrier of their own
    for (int i = tid - 64; i < N; i += 2 * BM) {
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
    asm volatile("bar.sync 1, 256;" ::: "memory");

    for (int r = 0; r < rounds && ok; ++r) {
      const int i = r;
      const int st = i % VST;   // these threads only touch the V ring
      // allowed columns of this row in this tile (64 per piece), and how many rows of each V
      // piece are real keys
      uint32_t allow[BN / 32];
      int valid[PPT];
      bool cache_tile = false, short_tile = false;
#pragma unroll
      for (int j = 0; j < PPT; ++j) {
        const int g = pc_begin + i * PPT + j;
        if (g >= pc_end) {                 // the range ended inside this tile
          valid[j] = 0;
          allow[2 * j] = allow[2 * j + 1] = 0;
        } else if (g < p_cache) {          // context piece: everything up to the context length
          cache_tile = true;
          valid[j] = min(PG, L - g * PG);
          const uint64_t bits = valid[j] >= 64 ? ~0ull : ((1ull << valid[j]) - 1ull);
          allow[2 * j] = (uint32_t)bits; allow[2 * j + 1] = (uint32_t)(bits >> 32);
        } else {                           // tree piece: the node's ancestors (itself included)
          const int tp = g - p_cache;
          valid[j] = min(PG, N - tp * PG);
          allow[2 * j] = s_anc[node][2 * tp]; allow[2 * j + 1] = s_anc[node][2 * tp + 1];
        }
        short_tile |= valid[j] < PG;
      }
      ok = mbar_wait(bar_s_full(slot), r & 1, abort_flag, wlim);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      if (p.paged && cache_tile) {
        // the producer's verdict on this tile's pages, written before it armed the V barrier (the
        // V stage is not reused before this tile's P V, so the flag is stable)
        ok = mbar_wait(bar_v_full(st), (i / VST) & 1, abort_flag, wlim);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        if (!*(volatile int*)&s_tile_ok[st]) {  // sequence is flagged; hide the whole tile
          short_tile = true;
#pragma unroll
          for (int j = 0; j < PPT; ++j) valid[j] = 0;
#pragma unroll
          for (int w = 0; w < BN / 32; ++w) allow[w] = 0;
        }
      }

      bool full = row_valid;
#pragma unroll
      for (int w = 0; w < BN / 32; ++w) {
        if (!row_valid) allow[w] = 0;
        full = full && (allow[w] == 0xFFFFFFFFu);
      }
      const bool all_full = __all_sync(0xFFFFFFFFu, full);

      uint32_t sv[64];
      // loads half h of the row and replaces the scores of columns that are not allowed by -inf
      auto load_half = [&](int h) {
        tmem_ld_x64(tmem_S(slot) + lane_addr + h * 64, sv);
        tmem_wait_ld();
        if (!all_full) {
#pragma unroll
          for (int j = 0; j < 64; ++j) {
            const uint32_t wbits = allow[2 * h + (j >> 5)];
            if (!((wbits >> (j & 31)) & 1u)) sv[j] = 0xFF800000u;  // -inf
          }
        }
      };
      // One pass with the reference maximum as it stands: exponentiate, pack P (kept in registers)
      // and add up the row.  No per-element maximum is tracked (the softmax threads are bound by
      // instruction issue): a row sum of at most 2^8 proves that no probability exceeded 2^8,
      // i.e. that the reference is still good.  Otherwise (rare after the first tile; inf or NaN
      // from an overflow also lands here) the true maximum is taken from the scores - still
      // intact, because P is stored last - the reference replaced, O rescaled and the tile redone.
      uint32_t pk[NH * 32];
      auto row_max = [&]() {
        float m0 = -INFINITY;
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          load_half(h);
#pragma unroll
          for (int j = 0; j < 64; ++j) m0 = fmaxf(m0, __uint_as_float(sv[j]));
        }
        return m0 * p.scale_log2;  // scale > 0; -inf (no allowed key) stays -inf
      };
      if (r == 0) m_ref = row_max();  // no reference yet: a cheap extra pass instead of a redo
      float sum = 0.f;
      float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      auto exp_pass = [&]() {
        sum = 0.f;
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          load_half(h);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float p0 = ex2(fmaf(__uint_as_float(sv[2 * j]), p.scale_log2, neg_m));
            const float p1 = ex2(fmaf(__uint_as_float(sv[2 * j + 1]), p.scale_log2, neg_m));
            sum += p0 + p1;
            pk[h * 32 + j] = pack_bf16(p0, p1);
          }
        }
      };
      exp_pass();
      const bool suspect = !(sum <= kRowSumLimit);  // also catches inf and NaN
      if (__any_sync(0xFFFFFFFFu, suspect)) {
        const float mx = suspect ? row_max() : m_ref;
        const bool need = mx > m_ref;
        if (r > 0) {  // O must be at rest: the previous P V has completed
          ok = mbar_wait(bar_pv_done(slot), (r - 1) & 1, abort_flag, wlim);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          tc_fence_after();
        }
        const float alpha = need ? ex2(m_ref - mx) : 1.0f;  // ex2(-inf) = 0
        if (need) { m_ref = mx; l_run *= alpha; }
        if (r > 0) {
#pragma unroll 1
          for (int c = 0; c < HD; c += 32) {
            uint32_t ov[32];
            tmem_ld_x32(tmem_O(slot) + lane_addr + c, ov);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
            tmem_st_x32(tmem_O(slot) + lane_addr + c, ov);
          }
          tmem_wait_st();
        }
        neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
        exp_pass();
      }
      // P (the A operand of P V) takes the place of score columns that have been consumed.  The
      // previous P V read these columns before this tile's Q K^T, issued after it, wrote them.
#pragma unroll
      for (int h = 0; h < NH; ++h)
        tmem_st_x32(tmem_P(slot) + lane_addr + h * 32, *reinterpret_cast<const uint32_t(*)[32]>(&pk[h * 32]));
      tmem_wait_st();
      l_run += sum;

      if (short_tile) {
        // Rows of a V piece beyond its real keys hold whatever lies behind them in memory (or were
        // never loaded); their probabilities are exactly 0, but 0 * NaN would poison O: clear them.
        ok = mbar_wait(bar_v_full(st), (i / VST) & 1, abort_flag, wlim);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        uint8_t* vt = sV_gen + st * kTile;
        const int me = (warp - 2 - slot * 4) * 32 + lane;   // 0 .. 127 within the softmax group
#pragma unroll
        for (int j = 0; j < PPT; ++j) {
          const int per_half = (PG - valid[j]) * 8;  // 16-byte chunks per half of the head dimension
          for (int c = me; c < 2 * per_half; c += BM) {
            const int half = c / per_half, rem = c - half * per_half;
            const int vr = j * PG + valid[j] + (rem >> 3), ch = rem & 7;
            *reinterpret_cast<uint4*>(vt + half * kHalf + vr * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
          }
        }
        fence_async_smem();   // cleared V rows visible to the tensor core's reads
      }
      tc_fence_before();
      mbar_arrive(bar_p_full(slot));
    }

    if (ok && rounds > 0) {  // the last P V of this slot has landed in O
      ok = mbar_wait(bar_pv_done(slot), (rounds - 1) & 1, abort_flag, wlim);
      ok = __all_sync(0xFFFFFFFFu, ok);
    }
  }

  // ---- every role meets here: all MMAs and copies of this block are complete -----------------
  __syncwarp();
  if (*abort_flag) {
    if (warp == 0 && lane == 0) {
      // TMA copies that were issued land on their own; wait for the newest phase of each stage
      for (int i = max(0, issued_k - KST); i < issued_k; ++i) mbar_drain(bar_k_full(i % KST), (i / KST) & 1);
      for (int i = max(0, issued_v - VST); i < issued_v; ++i) mbar_drain(bar_v_full(i % VST), (i / VST) & 1);
      if (n_tiles > 0) mbar_drain(bar_q, 0);
    }
    if (warp == 1 && lane == 0) {
      umma_commit(bar_drain);  // completes when every MMA issued so far has finished
      mbar_drain(bar_drain, 0);
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
  const int n_src = p.splits;  // accumulators that cover one output row
  const float kLn2 = 0.6931471805599453f;
  // staging area for the merge: O of both slots as fp16 [slot][128 rows][128], every row scaled by
  // a power of two that puts its largest magnitude in [2^13, 2^14) (half the bytes of fp32 through
  // distributed shared memory, at a relative rounding error of 2^-11, far below that of the bf16
  // output; the scale travels with the row's maximum and sum).  The 16-byte chunk c of row r is
  // stored at chunk (c ^ (r & 15)) so that row-per-thread writes and row-per-warp reads are both
  // conflict free.  The area reuses the tile memory, which nothing reads any more.
  uint8_t* const sO = smem_raw + (sQ - smem_u32(smem_raw));

  if (!aborted && warp >= 2) {
    if (n_src == 1) {
      // only accumulator of these rows: normalise and store
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      uint16_t* dst = p.out + (((int64_t)b * N + node) * p.Hq + kvh * G + gq) * HD;
#pragma unroll 1
      for (int c = 0; c < HD; c += 32) {
        uint32_t ov[32];
        tmem_ld_x32(tmem_O(slot) + lane_addr + c, ov);
        tmem_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(ov[q4 * 8 + 0]) * inv, __uint_as_float(ov[q4 * 8 + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(ov[q4 * 8 + 2]) * inv, __uint_as_float(ov[q4 * 8 + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(ov[q4 * 8 + 4]) * inv, __uint_as_float(ov[q4 * 8 + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(ov[q4 * 8 + 6]) * inv, __uint_as_float(ov[q4 * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + c + q4 * 8) = v;
          }
        }
      }
      if (p.lse != nullptr && row_valid)
        p.lse[((int64_t)b * N + node) * p.Hq + kvh * G + gq] = (m_ref + log2f(l_run)) * kLn2;
    } else {
      uint8_t* orow = sO + ((size_t)slot * BM + row) * (HD * 2);
      // first pass: the row's largest magnitude, which fixes its scale
      float amax = 0.f;
      if (my_rounds > 0) {
#pragma unroll 1
        for (int c = 0; c < HD; c += 32) {
          uint32_t ov[32];
          tmem_ld_x32(tmem_O(slot) + lane_addr + c, ov);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(__uint_as_float(ov[j])));
        }
      }
      // scale 2^lc with amax * 2^lc in [2^13, 2^14); lc is clamped so that the scale and its
      // inverse are normal numbers (a zero row keeps zeros, inf or NaN stay what they are)
      const int biased = (int)((__float_as_uint(amax) >> 23) & 255u);
      const int lc = max(-100, min(100, 140 - biased));
      const float cscale = __uint_as_float((uint32_t)(127 + lc) << 23);
      const float cinv = __uint_as_float((uint32_t)(127 - lc) << 23);
#pragma unroll 1
      for (int c = 0; c < HD; c += 32) {
        uint32_t ov[32];
        if (my_rounds > 0) {
          tmem_ld_x32(tmem_O(slot) + lane_addr + c, ov);
          tmem_wait_ld();
        } else {  // a slot without tiles contributes zeros with weight zero
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
          const int chunk = (c >> 3) + q4;
          *reinterpret_cast<uint4*>(orow + ((chunk ^ (row & 15)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
        }
      }
      s_ml[slot][row] = make_float4(my_rounds > 0 ? m_ref : -INFINITY, my_rounds > 0 ? l_run : 0.f, cinv, 0.f);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, kTmemCols);
  if (n_src == 1) {  // such a block is its own cluster
    if (tid == 0) publish(my_ticket);
    return;
  }

  // ---- merge across the cluster (the split-KV blocks of one row tile) through distributed
  //      shared memory: rank j finalises rows [j, j+1) * rows/splits of the tile(s) ------------
  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();  // every block's staging area is complete (also reached by an aborted block)
  if (!aborted) {
    // Every rank finalises per_rank rows; per_rank * n_src is 256 whatever the split count.
    const int per_rank = MT * BM / p.splits;
    const int first_row = split * per_rank;
    // (a) thread (k, q) fetches the (maximum, sum) pair of source q of row k; the n_src lanes of a
    //     row sit side by side in one warp, so the normalised weights come from shuffles.
    //     Source q is the accumulator of row tile `tile` in block q.
    if (tid < 2 * BM) {
      const int k = tid / n_src, q = tid - k * n_src;
      const int rr = first_row + k, tile = rr / BM, trow = rr % BM;
      const int qc = q, qs = tile;
      const float4 ml = dsmem_ld16(dsmem_addr(smem_u32(&s_ml[qs][trow]), qc));
      float mmax = ml.x;
      for (int o = 1; o < n_src; o <<= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xFFFFFFFFu, mmax, o));
      const float mu = (mmax == -INFINITY) ? 0.f : mmax;
      const float wgt = (ml.y > 0.f) ? ex2(ml.x - mu) : 0.f;
      float lsum = wgt * ml.y;
      for (int o = 1; o < n_src; o <<= 1) lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, o);
      s_w[tid] = wgt * (lsum > 0.f ? 1.f / lsum : 0.f) * ml.z;  // the staged row is 1 / ml.z times O
      const int rg = (row_cta * MT + tile) * RT + trow;
      if (q == 0 && p.lse != nullptr && trow < RT && rg < rows_total) {
        const int onode = rg / G, ogq = rg - onode * G;
        p.lse[((int64_t)b * N + onode) * p.Hq + kvh * G + ogq] = (mmax + log2f(lsum)) * kLn2;
      }
    }
    __syncthreads();
    // (b) weighted sums, rows spread over the warps
    const uint32_t sO_addr = smem_u32(sO);
    const int rot = split + 1;  // first source read: the next block's
    uint16_t* outp = p.out;
    const int64_t seq_row0 = (int64_t)b * N;
    switch (n_src) {
      case 2: merge_rows<2>(sO_addr, s_w, first_row, per_rank, rot, warp, lane, row_cta * MT, RT, rows_total, G, seq_row0, p.Hq, kvh * G, outp); break;
      case 4: merge_rows<4>(sO_addr, s_w, first_row, per_rank, rot, warp, lane, row_cta * MT, RT, rows_total, G, seq_row0, p.Hq, kvh * G, outp); break;
      default: merge_rows<8>(sO_addr, s_w, first_row, per_rank, rot, warp, lane, row_cta * MT, RT, rows_total, G, seq_row0, p.Hq, kvh * G, outp); break;
    }
  }
  cluster.sync();  // no block may leave while a peer still reads its shared memory
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

}  // namespace

bool tc2_attn_wanted(const clv_shape& s) {
  const int G = s.n_q_heads / s.n_kv_heads;
  if (G > BM) return false;
  return (s.n_nodes + BM / G - 1) / (BM / G) >= 4;   // four or more row tiles per (sequence, kv head)
}

AttnPlan tc2_attn_plan(const clv_shape& s, int max_ctx_len) {
  AttnPlan pl;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int tiles = (s.n_nodes + BM / G - 1) / (BM / G);   // row tiles of BM / G whole nodes
  const int row_ctas = (tiles + MT - 1) / MT;
  pl.m_tiles = row_ctas;
  const int64_t ctas = (int64_t)s.batch * s.n_kv_heads * row_ctas;
  const int BN = Cfg::BN;
  const int key_tiles = (max_ctx_len > 0 ? (max_ctx_len + BN - 1) / BN : 0) + (s.n_nodes + BN - 1) / BN;
  // The key axis is split over a thread-block cluster (merged through distributed shared memory),
  // so the split count is a power of two up to the portable cluster size; one block per SM.
  int splits = 1;
  while (splits < 8 && ctas * (splits * 2) <= sm_count() && key_tiles / (splits * 2) >= 1) splits *= 2;
  pl.splits = splits;
  pl.tickets = 0;
  pl.scratch_bytes = 0;  // nothing goes through global memory
  return pl;
}

cudaError_t launch_tree_attn_tc2(const AttnPlan& plan, const clv_shape& s, const clv_kv_cache& c,
                                 const void* q, const void* k_tree, const void* v_tree,
                                 const int32_t* parent, const int32_t* ctx_len, float scale, void* out,
                                 float* lse, int32_t* status, unsigned* tickets, void* scratch,
                                 cudaStream_t stream) {
  (void)scratch;
  const int G = s.n_q_heads / s.n_kv_heads;
  static OncePerDevice once;
  cudaError_t e0 = run_once_per_device(once, [] {
    return cudaFuncSetAttribute(tree_attn_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)Cfg::kSmem);
  });
  if (e0 != cudaSuccess) return e0;
  alignas(64) CUtensorMap tm_q, tm_kc, tm_vc, tm_kt, tm_vt;
  const uint64_t cache_rows = c.paged ? (uint64_t)c.n_pages * CLV_PAGE_SIZE : (uint64_t)s.batch * c.cap_tokens;
  const uint64_t tree_rows = (uint64_t)s.batch * s.n_nodes;
  if (!make_map(&tm_q, q, tree_rows, s.n_q_heads, G, BM / G) ||
      !make_map(&tm_kc, c.k, cache_rows, s.n_kv_heads, 1, PG) ||
      !make_map(&tm_vc, c.v, cache_rows, s.n_kv_heads, 1, PG) ||
      !make_map(&tm_kt, k_tree, tree_rows, s.n_kv_heads, 1, PG) ||
      !make_map(&tm_vt, v_tree, tree_rows, s.n_kv_heads, 1, PG))
    return cudaErrorInvalidValue;

  Params p;
  p.block_table = c.block_table;
  p.parent = parent;
  p.ctx_len = ctx_len;
  p.out = static_cast<uint16_t*>(out);
  p.lse = lse;
  p.status = status;
  const int64_t ctas = (int64_t)s.batch * s.n_kv_heads * plan.m_tiles;
  p.B = s.batch; p.N = s.n_nodes; p.Hq = s.n_q_heads; p.Hkv = s.n_kv_heads; p.G = G;
  p.paged = c.paged; p.cap_tokens = c.cap_tokens; p.n_pages = c.n_pages; p.max_pages = c.max_pages_per_seq;
  p.row_ctas = plan.m_tiles;
  p.splits = plan.splits;
  p.longest_first = (ctas > sm_count() && s.batch > 1 && s.batch <= 256) ? 1 : 0;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.wait_limit = wait_limit_cycles();
  p.tickets = tickets;
  p.blocks_per_seq = s.n_kv_heads * plan.m_tiles * plan.splits;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas, (unsigned)plan.splits, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::kSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;  // the blocks that split one pair of row tiles' keys
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = (unsigned)plan.splits;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up overlaps the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, tree_attn_tc2_kernel, tm_q, tm_kc, tm_vc, tm_kt, tm_vt, p);
}

}  // namespace clv
