// Tree attention (Sec. 2.1): split-KV flash-decode over the committed cache plus the tree's own
// K/V, the tree columns masked by ancestor bitsets derived from parent[] on chip (the N x N
// topology matrix of Fig. 2 is never materialised; cf. App. A.1).
//
// Generic tensor-core path (warp-level mma.sync m16n8k16, bf16 in / fp32 accumulate).  One thread
// block owns a tile of 64 query rows of one (sequence, kv head) - rows are (node, head-in-group)
// pairs, so the G query heads of a group and all tree nodes share every K/V byte fetched - and a
// contiguous range of 64-key tiles.  K/V tiles are staged with 16-byte cp.async into XOR-swizzled
// shared memory, double buffered.  When the key axis is split, the partial (m, l, O) triples go
// to the workspace and the last block to arrive for a row tile merges them.
#include <math.h>

#include "clv_internal.cuh"

namespace clv {
namespace {

constexpr int BM = 64;        // query rows per block
constexpr int BN = 64;        // keys per tile (= page size)
constexpr int HD = CLV_HEAD_DIM;
constexpr int kThreads = 128;
constexpr int kTileBytes = BN * HD * 2;
constexpr int kSmemBytes = kTileBytes * 5;  // Q + 2 x (K, V)
constexpr int kMaxSplits = 16;

struct Params {
  const uint16_t* q;
  const uint16_t* k_tree;
  const uint16_t* v_tree;
  const uint16_t* kc;
  const uint16_t* vc;
  const int32_t* block_table;
  const int32_t* parent;
  const int32_t* ctx_len;
  uint16_t* out;
  float* lse;
  int32_t* status;
  unsigned* tickets;
  float* part_o;   // [row tile][split][BM][HD]
  float* part_ml;  // [row tile][split][BM][2]
  int B, N, Hq, Hkv, G;
  int paged, cap_tokens, n_pages, max_pages;
  int m_tiles, splits;
  float scale_log2;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;  // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N_>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N_));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                        uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                          uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
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
// byte offset of 16-byte chunk `ch` of row `row` inside a [64][128] bf16 tile (XOR swizzle)
__device__ __forceinline__ uint32_t tile_off(int row, int ch) {
  return (uint32_t)(row * 256 + ((ch ^ (row & 7)) << 4));
}

__global__ void __launch_bounds__(kThreads) tree_attn_mma_kernel(Params p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint32_t s_anc[CLV_MAX_NODES][4];
  __shared__ int s_parent[CLV_MAX_NODES];
  __shared__ float s_w[kMaxSplits][BM];
  __shared__ int s_last;

  const int unit = blockIdx.x / p.m_tiles, mt = blockIdx.x - unit * p.m_tiles, split = blockIdx.y;
  const int b = unit / p.Hkv, kvh = unit - b * p.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
  const int N = p.N, G = p.G, rows_total = G * N;

  // ---- per-sequence checks and ancestor bitsets (row i of the topology matrix) ------------
  const int L = p.ctx_len[b];
  bool bad = false;
  for (int i = tid; i < N; i += kThreads) {
    const int par = p.parent[(int64_t)b * N + i];
    s_parent[i] = par;
    bad |= (par < -1 || par >= i);
  }
  bad |= (L < 0);
  const int t_cache = L > 0 ? (L + BN - 1) / BN : 0;
  if (p.paged) bad |= (t_cache > p.max_pages);
  else bad |= (L > p.cap_tokens);
  // parent[] and ctx_len give every block of the sequence the same verdict, so they all leave
  // together.  A bad block-table entry does not end a block: that tile is skipped below.
  const int seq_bad = __syncthreads_or(bad ? 1 : 0);
  if (mt == 0 && split == 0 && kvh == 0) {  // one block per sequence reports
    bool pbad = false;
    if (p.paged && !seq_bad) {
      for (int pg = tid; pg < t_cache; pg += kThreads) {
        const int e = p.block_table[(int64_t)b * p.max_pages + pg];
        pbad |= (e < 0 || e >= p.n_pages);
      }
    }
    const int page_bad = __syncthreads_or(pbad ? 1 : 0);
    if (tid == 0) p.status[b] = (seq_bad || page_bad) ? CLV_ERR_TREE : CLV_OK;
  }
  if (seq_bad) return;
  for (int i = tid; i < N; i += kThreads) {
    uint32_t w[4] = {0, 0, 0, 0};
    int j = i;
    for (int hop = 0; hop < N && j >= 0; ++hop) {  // parent[j] < j: ends within N hops
      w[j >> 5] |= 1u << (j & 31);
      j = s_parent[j];
    }
    s_anc[i][0] = w[0]; s_anc[i][1] = w[1]; s_anc[i][2] = w[2]; s_anc[i][3] = w[3];
  }

  // ---- tile range of this block -----------------------------------------------------------
  const int t_tree = (N + BN - 1) / BN;
  const int t_total = t_cache + t_tree;
  const int t_begin = (int)((int64_t)split * t_total / p.splits);
  const int t_end = (int)((int64_t)(split + 1) * t_total / p.splits);
  const int n_tiles = t_end - t_begin;

  uint8_t* sQ = smem;
  const uint32_t sQ_a = smem_u32(sQ);
  const uint32_t sK_a = sQ_a + kTileBytes;       // two stages
  const uint32_t sV_a = sQ_a + 3 * kTileBytes;   // two stages

  auto load_kv = [&](int stage, int t) {
    const bool is_tree = t >= t_cache;
    int64_t row0 = 0;       // first source row (token index in the source tensor)
    int valid_rows;
    const uint16_t *srcK, *srcV;
    if (!is_tree) {
      valid_rows = min(BN, L - t * BN);
      if (p.paged) {
        const int pg = p.block_table[(int64_t)b * p.max_pages + t];
        if (pg < 0 || pg >= p.n_pages) valid_rows = 0;
        row0 = (int64_t)pg * BN;
      } else {
        row0 = (int64_t)b * p.cap_tokens + (int64_t)t * BN;
      }
      srcK = p.kc; srcV = p.vc;
    } else {
      const int j0 = (t - t_cache) * BN;
      valid_rows = min(BN, N - j0);
      row0 = (int64_t)b * N + j0;
      srcK = p.k_tree; srcV = p.v_tree;
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int idx = tid + c * kThreads;
      const int row = idx >> 4, ch = idx & 15;
      const bool ok = row < valid_rows;
      const int64_t off = ok ? (((row0 + row) * p.Hkv + kvh) * HD + ch * 8) : 0;
      const uint32_t d = tile_off(row, ch);
      cp_async16(sK_a + stage * kTileBytes + d, srcK + off, ok);
      cp_async16(sV_a + stage * kTileBytes + d, srcV + off, ok);
    }
  };

  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  // rows of this thread: warp*16 + g and + 8
  const int r_loc0 = warp * 16 + g, r_loc1 = r_loc0 + 8;
  const int r0 = mt * BM + r_loc0, r1 = mt * BM + r_loc1;
  const bool rv0 = r0 < rows_total, rv1 = r1 < rows_total;
  const int node0 = rv0 ? r0 / G : 0, node1 = rv1 ? r1 / G : 0;

  if (n_tiles > 0) {
    // Q tile: row r = node * G + head-in-group
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int idx = tid + c * kThreads;
      const int row = idx >> 4, ch = idx & 15;
      const int r = mt * BM + row;
      const bool ok = r < rows_total;
      const int node = ok ? r / G : 0, gq = ok ? r - node * G : 0;
      const int64_t off = (((int64_t)b * N + node) * p.Hq + kvh * G + gq) * HD + ch * 8;
      cp_async16(sQ_a + tile_off(row, ch), p.q + (ok ? off : 0), ok);
    }
    load_kv(0, t_begin);
    cp_async_commit();
  }

  uint32_t qa[8][4];
  for (int it = 0; it < n_tiles; ++it) {
    const int stage = it & 1;
    if (it + 1 < n_tiles) {
      load_kv(stage ^ 1, t_begin + it + 1);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (it == 0) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ch = 2 * ks + (lane >> 4);
        ldsm_x4(sQ_a + tile_off(row, ch), qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
      }
    }
    const uint32_t kb = sK_a + stage * kTileBytes, vb = sV_a + stage * kTileBytes;

    // ---- S = Q K^T : 16 rows x 64 keys per warp ----
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        const int mi = lane >> 3;
        const int krow = (2 * np + (mi >> 1)) * 8 + (lane & 7);
        const int ch = 2 * ks + (mi & 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4(kb + tile_off(krow, ch), b0, b1, b2, b3);
        mma_bf16(s[2 * np], qa[ks], b0, b1);
        mma_bf16(s[2 * np + 1], qa[ks], b2, b3);
      }
    }

    // ---- scale, mask, online softmax ----
    const int t = t_begin + it;
    uint32_t a0lo, a0hi, a1lo, a1hi;  // allowed-column bits of this thread's two rows
    if (t < t_cache) {
      const int left = L - t * BN;  // >= 1
      const uint64_t bits = left >= 64 ? ~0ull : ((1ull << left) - 1ull);
      a0lo = a1lo = (uint32_t)bits;
      a0hi = a1hi = (uint32_t)(bits >> 32);
      if (p.paged) {  // an invalid page was zero-filled: hide it completely
        const int pg = p.block_table[(int64_t)b * p.max_pages + t];
        if (pg < 0 || pg >= p.n_pages) a0lo = a0hi = a1lo = a1hi = 0;
      }
    } else {
      const int tt = t - t_cache;
      a0lo = s_anc[node0][2 * tt]; a0hi = s_anc[node0][2 * tt + 1];
      a1lo = s_anc[node1][2 * tt]; a1hi = s_anc[node1][2 * tt + 1];
    }
    if (!rv0) a0lo = a0hi = 0;
    if (!rv1) a1lo = a1hi = 0;
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int col = nt * 8 + 2 * t4;  // col and col+1 lie in the same 32-bit word
      const uint32_t w0 = (nt < 4) ? a0lo : a0hi, w1 = (nt < 4) ? a1lo : a1hi;
      const int sh = col & 31;
      s[nt][0] = ((w0 >> sh) & 1u) ? s[nt][0] * p.scale_log2 : -INFINITY;
      s[nt][1] = ((w0 >> (sh + 1)) & 1u) ? s[nt][1] * p.scale_log2 : -INFINITY;
      s[nt][2] = ((w1 >> sh) & 1u) ? s[nt][2] * p.scale_log2 : -INFINITY;
      s[nt][3] = ((w1 >> (sh + 1)) & 1u) ? s[nt][3] * p.scale_log2 : -INFINITY;
      mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
      mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 2));
    const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
    const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
    const float al0 = ex2(m_run[0] - mu0), al1 = ex2(m_run[1] - mu1);  // ex2(-inf) = 0
    m_run[0] = mn0; m_run[1] = mn1;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t pa[4][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p0 = ex2(s[nt][0] - mu0), p1 = ex2(s[nt][1] - mu0);
      const float p2 = ex2(s[nt][2] - mu1), p3 = ex2(s[nt][3] - mu1);
      sum0 += p0 + p1;
      sum1 += p2 + p3;
      pa[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
      pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    l_run[0] = l_run[0] * al0 + sum0;
    l_run[1] = l_run[1] * al1 + sum1;
#pragma unroll
    for (int nd = 0; nd < 16; ++nd) {
      o[nd][0] *= al0; o[nd][1] *= al0; o[nd][2] *= al1; o[nd][3] *= al1;
    }

    // ---- O += P V ----
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {
        const int mi = lane >> 3;
        const int vrow = 16 * kk + (mi & 1) * 8 + (lane & 7);
        const int ch = 2 * dp + (mi >> 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vb + tile_off(vrow, ch), b0, b1, b2, b3);
        mma_bf16(o[2 * dp], pa[kk], b0, b1);
        mma_bf16(o[2 * dp + 1], pa[kk], b2, b3);
      }
    }
    __syncthreads();  // the other stage may be overwritten by the next iteration's loads
  }

  // row sums live spread over the 4 lanes of a quad
  l_run[0] += __shfl_xor_sync(0xFFFFFFFFu, l_run[0], 1);
  l_run[0] += __shfl_xor_sync(0xFFFFFFFFu, l_run[0], 2);
  l_run[1] += __shfl_xor_sync(0xFFFFFFFFu, l_run[1], 1);
  l_run[1] += __shfl_xor_sync(0xFFFFFFFFu, l_run[1], 2);

  const float kLn2 = 0.6931471805599453f;
  if (p.splits == 1) {
    // normalise, stage as bf16 in the (now free) Q tile, then 16-byte coalesced stores
    const float inv0 = l_run[0] > 0.f ? 1.f / l_run[0] : 0.f;
    const float inv1 = l_run[1] > 0.f ? 1.f / l_run[1] : 0.f;
#pragma unroll
    for (int nd = 0; nd < 16; ++nd) {
      // element column nd*8 + 2*t4 -> chunk nd, 4-byte slot t4
      *reinterpret_cast<uint32_t*>(sQ + tile_off(r_loc0, nd) + 4 * t4) =
          pack_bf16(o[nd][0] * inv0, o[nd][1] * inv0);
      *reinterpret_cast<uint32_t*>(sQ + tile_off(r_loc1, nd) + 4 * t4) =
          pack_bf16(o[nd][2] * inv1, o[nd][3] * inv1);
    }
    if (p.lse != nullptr && t4 == 0) {
      if (rv0) p.lse[((int64_t)b * N + node0) * p.Hq + kvh * G + (r0 - node0 * G)] =
          (m_run[0] + log2f(l_run[0])) * kLn2;
      if (rv1) p.lse[((int64_t)b * N + node1) * p.Hq + kvh * G + (r1 - node1 * G)] =
          (m_run[1] + log2f(l_run[1])) * kLn2;
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int idx = tid + c * kThreads;
      const int row = idx >> 4, ch = idx & 15;
      const int r = mt * BM + row;
      if (r < rows_total) {
        const int node = r / G, gq = r - node * G;
        const int64_t off = (((int64_t)b * N + node) * p.Hq + kvh * G + gq) * HD + ch * 8;
        *reinterpret_cast<uint4*>(p.out + off) = *reinterpret_cast<const uint4*>(sQ + tile_off(row, ch));
      }
    }
    return;
  }

  // ---- split: publish the partial, the last block of this row tile merges ------------------
  const int64_t tile_id = (int64_t)blockIdx.x;
  float* po = p.part_o + (tile_id * p.splits + split) * (int64_t)(BM * HD);
  float* pml = p.part_ml + (tile_id * p.splits + split) * (int64_t)(BM * 2);
#pragma unroll
  for (int nd = 0; nd < 16; ++nd) {
    __stcg(reinterpret_cast<float2*>(po + r_loc0 * HD + nd * 8 + 2 * t4), make_float2(o[nd][0], o[nd][1]));
    __stcg(reinterpret_cast<float2*>(po + r_loc1 * HD + nd * 8 + 2 * t4), make_float2(o[nd][2], o[nd][3]));
  }
  if (t4 == 0) {
    __stcg(reinterpret_cast<float2*>(pml + r_loc0 * 2), make_float2(m_run[0], l_run[0]));
    __stcg(reinterpret_cast<float2*>(pml + r_loc1 * 2), make_float2(m_run[1], l_run[1]));
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned arrived = atomicInc(p.tickets + tile_id, (unsigned)p.splits - 1);  // wraps to 0
    s_last = (arrived == (unsigned)p.splits - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  const float* all_o = p.part_o + tile_id * p.splits * (int64_t)(BM * HD);
  const float* all_ml = p.part_ml + tile_id * p.splits * (int64_t)(BM * 2);
  if (tid < BM) {
    float mmax = -INFINITY;
    for (int s_ = 0; s_ < p.splits; ++s_)
      mmax = fmaxf(mmax, __ldcg(all_ml + (int64_t)s_ * BM * 2 + tid * 2));
    const float mu = (mmax == -INFINITY) ? 0.f : mmax;
    float lsum = 0.f;
    for (int s_ = 0; s_ < p.splits; ++s_) {
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(all_ml + (int64_t)s_ * BM * 2 + tid * 2));
      const float w = ex2(ml.x - mu);
      s_w[s_][tid] = w;
      lsum += w * ml.y;
    }
    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
    for (int s_ = 0; s_ < p.splits; ++s_) s_w[s_][tid] *= inv;
    const int r = mt * BM + tid;
    if (p.lse != nullptr && r < rows_total) {
      const int node = r / G, gq = r - node * G;
      p.lse[((int64_t)b * N + node) * p.Hq + kvh * G + gq] = (mmax + log2f(lsum)) * kLn2;
    }
  }
  __syncthreads();
  {
    const int row = tid >> 1, half = tid & 1;
    const int r = mt * BM + row;
    if (r < rows_total) {
      const int node = r / G, gq = r - node * G;
      uint16_t* dst = p.out + (((int64_t)b * N + node) * p.Hq + kvh * G + gq) * HD + half * 64;
#pragma unroll 2
      for (int c = 0; c < 64; c += 8) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int s_ = 0; s_ < p.splits; ++s_) {
          const float w = s_w[s_][row];
          const float4* src = reinterpret_cast<const float4*>(
              all_o + (int64_t)s_ * BM * HD + row * HD + half * 64 + c);
          const float4 x = __ldcg(src), y = __ldcg(src + 1);
          acc[0] += w * x.x; acc[1] += w * x.y; acc[2] += w * x.z; acc[3] += w * x.w;
          acc[4] += w * y.x; acc[5] += w * y.y; acc[6] += w * y.z; acc[7] += w * y.w;
        }
        uint4 v;
        v.x = pack_bf16(acc[0], acc[1]); v.y = pack_bf16(acc[2], acc[3]);
        v.z = pack_bf16(acc[4], acc[5]); v.w = pack_bf16(acc[6], acc[7]);
        *reinterpret_cast<uint4*>(dst + c) = v;
      }
    }
  }
}

}  // namespace

AttnPlan attn_plan(const clv_shape& s, int max_ctx_len) {
  AttnPlan pl;
  const int G = s.n_q_heads / s.n_kv_heads;
  pl.m_tiles = (G * s.n_nodes + BM - 1) / BM;
  const int64_t row_tiles = (int64_t)s.batch * s.n_kv_heads * pl.m_tiles;
  const int key_tiles = (max_ctx_len > 0 ? (max_ctx_len + BN - 1) / BN : 0) + (s.n_nodes + BN - 1) / BN;
  int64_t want = (2LL * sm_count()) / (row_tiles > 0 ? row_tiles : 1);  // two resident blocks per SM
  if (want > kMaxSplits) want = kMaxSplits;
  if (want > key_tiles) want = key_tiles;
  if (want < 1 || row_tiles > kTickets) want = 1;
  pl.splits = (int)want;
  pl.tickets = pl.splits > 1 ? (int)row_tiles : 0;
  pl.scratch_bytes = pl.splits > 1
      ? (size_t)row_tiles * pl.splits * (BM * HD + BM * 2) * sizeof(float) : 0;
  return pl;
}

cudaError_t launch_tree_attn(const AttnPlan& plan, const clv_shape& s, const clv_kv_cache& c,
                             const void* q, const void* k_tree, const void* v_tree,
                             const int32_t* parent, const int32_t* ctx_len, float scale, void* out,
                             float* lse, int32_t* status, unsigned* tickets, void* scratch,
                             cudaStream_t stream) {
  static bool attr_done[kMaxDevices] = {};
  if (first_call_on_device(attr_done)) {
    cudaError_t e = cudaFuncSetAttribute(tree_attn_mma_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
  }
  Params p;
  p.q = static_cast<const uint16_t*>(q);
  p.k_tree = static_cast<const uint16_t*>(k_tree);
  p.v_tree = static_cast<const uint16_t*>(v_tree);
  p.kc = static_cast<const uint16_t*>(c.k);
  p.vc = static_cast<const uint16_t*>(c.v);
  p.block_table = c.block_table;
  p.parent = parent;
  p.ctx_len = ctx_len;
  p.out = static_cast<uint16_t*>(out);
  p.lse = lse;
  p.status = status;
  p.tickets = tickets;
  const int64_t row_tiles = (int64_t)s.batch * s.n_kv_heads * plan.m_tiles;
  p.part_o = static_cast<float*>(scratch);
  p.part_ml = p.part_o + row_tiles * plan.splits * (int64_t)(BM * HD);
  p.B = s.batch; p.N = s.n_nodes; p.Hq = s.n_q_heads; p.Hkv = s.n_kv_heads;
  p.G = s.n_q_heads / s.n_kv_heads;
  p.paged = c.paged; p.cap_tokens = c.cap_tokens; p.n_pages = c.n_pages;
  p.max_pages = c.max_pages_per_seq;
  p.m_tiles = plan.m_tiles; p.splits = plan.splits;
  p.scale_log2 = scale * 1.4426950408889634f;
  dim3 grid((unsigned)row_tiles, (unsigned)plan.splits, 1);
  tree_attn_mma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace clv
