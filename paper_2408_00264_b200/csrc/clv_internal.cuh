// Internal declarations shared by the translation units of libclv (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "clv.h"

namespace clv {

// ---- workspace layout -------------------------------------------------------------------------
// [0, 256)                     header (reserved)
// [256, 256 + 4*kTickets)      arrival counters, zero between calls (self-resetting atomicInc)
// [kWsFixedBytes, ...)         scratch for partial results (contents are garbage between calls)
constexpr size_t kWsHeaderBytes = 256;
constexpr int kTickets = 65536;
constexpr size_t kWsFixedBytes = kWsHeaderBytes + sizeof(unsigned) * (size_t)kTickets;

inline unsigned* ws_tickets(void* ws) {
  return reinterpret_cast<unsigned*>(static_cast<char*>(ws) + kWsHeaderBytes);
}
inline void* ws_scratch(void* ws) { return static_cast<char*>(ws) + kWsFixedBytes; }

// ---- argmax -----------------------------------------------------------------------------------
struct ArgmaxPlan {
  int rows;         // B * N
  int chunks;       // thread blocks per row
  int chunk_elems;  // multiple of 8
  size_t scratch_bytes;
};
ArgmaxPlan argmax_plan(int rows, int vocab);
cudaError_t launch_argmax(const ArgmaxPlan& plan, const void* logits, int64_t ld, int vocab,
                          int32_t* ids, unsigned* tickets, void* scratch, cudaStream_t stream);

// variant with its scratch in a fixed device array of the library (no caller workspace)
bool argmax_static_fits(int rows, int vocab);
cudaError_t launch_argmax_static(const void* logits, int64_t ld, int rows, int vocab, int32_t* ids,
                                 cudaStream_t stream);

// ---- stochastic acceptance (temperature > 0): statistics pass over the logits + per-sequence walk
int sample_max_vocab();
size_t sample_scratch_bytes(int rows, int vocab);
cudaError_t launch_accept_sample(const clv_shape& s, const void* logits, int64_t ld, const int32_t* parent,
                                 const int32_t* tokens, const float* uniforms, float temperature,
                                 int32_t* accept_len, int32_t* accept_idx, int32_t* next_token, int32_t* status,
                                 void* scratch, cudaStream_t stream);

// ---- walk / commit ----------------------------------------------------------------------------
cudaError_t launch_walk(const clv_shape& s, const int32_t* parent, const int32_t* tokens,
                        const int32_t* ids, int32_t* accept_len, int32_t* accept_idx,
                        int32_t* next_token, int32_t* status, cudaStream_t stream);
cudaError_t launch_commit(const clv_shape& s, const clv_kv_cache& c, const void* k_tree,
                          const void* v_tree, const int32_t* accept_idx, const int32_t* accept_len,
                          const int32_t* ctx_len, int32_t* ctx_len_out, int32_t* status,
                          cudaStream_t stream);

cudaError_t launch_walk_commit(const clv_shape& s, const clv_kv_cache& c, const int32_t* parent,
                               const int32_t* tokens, const int32_t* ids, const void* k_tree,
                               const void* v_tree, const int32_t* ctx_len, int32_t* accept_len,
                               int32_t* accept_idx, int32_t* next_token, int32_t* ctx_len_out,
                               int32_t* walk_status, int32_t* commit_status, cudaStream_t stream);

cudaError_t launch_commit_layers(const clv_shape& s, const clv_kv_cache& c, int n_layers, int64_t cache_layer_stride,
                                 const void* k_tree, const void* v_tree, int64_t tree_layer_stride,
                                 const int32_t* accept_idx, const int32_t* accept_len, const int32_t* ctx_len,
                                 int32_t* ctx_len_out, int32_t* status, cudaStream_t stream);

// ---- interval (depth-first label) form of the tree mask
cudaError_t launch_tree_to_intervals(int batch, int n_nodes, const int32_t* parent, int32_t* tin, int32_t* tout,
                                     int32_t* status, cudaStream_t stream);
cudaError_t launch_tree_from_intervals(int batch, int n_nodes, const int32_t* tin, const int32_t* tout,
                                       int32_t* parent, int32_t* status, cudaStream_t stream);

// ---- tree attention (tcgen05 / TMA; a row tile holds whole nodes: any group size G up to 128) -------
struct AttnPlan {
  int m_tiles;   // row tiles per (sequence, kv head)
  int splits;    // thread blocks along the key axis per row tile
  size_t scratch_bytes;
  int tickets;   // counters used
};
bool tc_attn_supported(const clv_shape& s, const clv_kv_cache& c);
AttnPlan tc_attn_plan(const clv_shape& s, int max_ctx_len);
cudaError_t launch_tree_attn_tc(const AttnPlan& plan, const clv_shape& s, const clv_kv_cache& c,
                                const void* q, const void* k_tree, const void* v_tree,
                                const int32_t* parent, const int32_t* ctx_len, float scale, void* out,
                                float* lse, int32_t* status, unsigned* tickets, void* scratch,
                                cudaStream_t stream);
// units of four or more row tiles per (sequence, kv head): blocks of two row tiles that share every
// staged K/V tile (same results, same plan fields; m_tiles counts pairs of row tiles)
bool tc2_attn_wanted(const clv_shape& s);
AttnPlan tc2_attn_plan(const clv_shape& s, int max_ctx_len);
cudaError_t launch_tree_attn_tc2(const AttnPlan& plan, const clv_shape& s, const clv_kv_cache& c,
                                 const void* q, const void* k_tree, const void* v_tree,
                                 const int32_t* parent, const int32_t* ctx_len, float scale, void* out,
                                 float* lse, int32_t* status, unsigned* tickets, void* scratch,
                                 cudaStream_t stream);

// ---- LM head fused with the argmax (tcgen05 GEMM whose logits stay in tensor memory) ---------------
bool lm_head_supported(int rows, int hidden, int vocab);
cudaError_t launch_lm_head_argmax(const void* hidden, int64_t ld_hidden, const void* weight, int64_t ld_weight,
                                  int rows, int hidden_dim, int vocab, int32_t* ids, int32_t* status,
                                  unsigned* tickets, cudaStream_t stream);

int rows_linear_splits(int rows, int in_dim, int out_dim, int n);
cudaError_t launch_rows_linear(int n, const void* const* x, int64_t ld_x, const void* const* weight,
                               int64_t ld_weight, const void* const* bias, int rows, int in_dim, int out_dim,
                               float* const* out, int64_t ld_out, int splits, int64_t split_stride, int32_t* status,
                               unsigned* tickets, cudaStream_t stream);

// ---- one step of a Clover-2 draft head
size_t draft_head_scratch_bytes(int rows, int hidden, int vocab);
cudaError_t launch_draft_head_step(const clv_draft_head& w, int rows, const void* h, const void* e, int k_top,
                                   void* hidden_out, int32_t* top_ids, float* top_logits, int32_t* status,
                                   unsigned* tickets, void* scratch, cudaStream_t stream);

// ---- token tree from speculated sequences -------------------------------------------------------
cudaError_t launch_token_tree(int batch, int n_cand, int max_len, int node_cap, const int32_t* root_token,
                              const int32_t* cand, const int32_t* cand_len, int32_t* tokens, int32_t* parent,
                              int32_t* n_nodes, int32_t* node_of, int32_t* status, cudaStream_t stream);

int sm_count();   // of the current device

// SM cycles a bounded on-chip wait may last before the block gives up (default: about a second;
// clv_test_set_wait_limit shortens it for the tests of the time-out path).
long long wait_limit_cycles();

// Per-device one-time set-up (function attributes belong to the device that is current when they
// are set).  run_once_per_device(state, fn) runs fn() with the current device until it has
// succeeded once on that device; concurrent first calls from several host threads are serialised,
// and a failed set-up is retried by the next call.
constexpr int kMaxDevices = 64;
struct OncePerDevice {
  std::mutex mu;
  bool done[kMaxDevices] = {};
};
template <class Fn>
inline cudaError_t run_once_per_device(OncePerDevice& st, Fn fn) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return fn();   // not remembered: set up at every call
  std::lock_guard<std::mutex> lock(st.mu);
  if (st.done[dev]) return cudaSuccess;
  e = fn();
  if (e == cudaSuccess) st.done[dev] = true;
  return e;
}

}  // namespace clv
