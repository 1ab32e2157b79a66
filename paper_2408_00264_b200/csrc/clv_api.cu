// C ABI of libclv: argument checks and dispatch.  No device memory is allocated here, nothing
// synchronises, every launch goes to the caller's stream.
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "clv_internal.cuh"

namespace clv {

static thread_local int g_last_cuda_error = 0;

int sm_count() {
  static std::mutex mu;
  static int cached[kMaxDevices] = {};
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return 148;  // B200; used for sizing only when no device can be queried
  }
  std::lock_guard<std::mutex> lock(mu);
  if (cached[dev] == 0) {
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      cached[dev] = v;
    else
      return 148;
  }
  return cached[dev];
}

static std::atomic<long long> g_wait_limit{2000000000ll};  // SM cycles: about a second
long long wait_limit_cycles() { return g_wait_limit.load(std::memory_order_relaxed); }

static clv_status cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return CLV_ERR_CUDA;
}
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static clv_status check_shape(const clv_shape* s) {
  if (!s) return CLV_ERR_NULL;
  if (s->batch < 1 || s->n_nodes < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1) return CLV_ERR_SHAPE;
  if (s->n_q_heads % s->n_kv_heads) return CLV_ERR_SHAPE;
  if (s->head_dim != CLV_HEAD_DIM || s->n_nodes > CLV_MAX_NODES) return CLV_ERR_UNSUPPORTED;
  return CLV_OK;
}

static clv_status check_cache(const clv_kv_cache* c) {
  if (!c || !c->k || !c->v) return CLV_ERR_NULL;
  if (!aligned16(c->k) || !aligned16(c->v)) return CLV_ERR_ALIGN;
  if (c->paged) {
    if (!c->block_table) return CLV_ERR_NULL;
    if (c->page_size != CLV_PAGE_SIZE) return CLV_ERR_UNSUPPORTED;
    if (c->n_pages < 1 || c->max_pages_per_seq < 1) return CLV_ERR_SHAPE;
  } else if (c->cap_tokens < 1) {
    return CLV_ERR_SHAPE;
  }
  return CLV_OK;
}

static size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace clv

using namespace clv;

extern "C" {

size_t clv_workspace_bytes(const clv_shape* shape, const clv_kv_cache* cache, int32_t max_ctx_len) {
  (void)cache;
  if (check_shape(shape) != CLV_OK) return 0;
  if (max_ctx_len < 0) max_ctx_len = 0;
  size_t scratch = (tc2_attn_wanted(*shape) ? tc2_attn_plan(*shape, max_ctx_len)
                                            : tc_attn_plan(*shape, max_ctx_len)).scratch_bytes;
  if (shape->vocab > 0) {
    const ArgmaxPlan gp = argmax_plan(shape->batch * shape->n_nodes, shape->vocab);
    if (gp.scratch_bytes > scratch) scratch = gp.scratch_bytes;
    const size_t sb = sample_scratch_bytes(shape->batch * shape->n_nodes, shape->vocab);
    if (sb > scratch) scratch = sb;
  }
  return kWsFixedBytes + round_up(scratch, 256);
}

clv_status clv_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!workspace) return CLV_ERR_NULL;
  if (workspace_bytes < kWsFixedBytes) return CLV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return CLV_ERR_ALIGN;
  cudaError_t e = cudaMemsetAsync(workspace, 0, kWsFixedBytes, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

// Argument checks of clv_tree_attn (nothing is enqueued); fills the plan on success.
static clv_status validate_tree_attn(const clv_shape* shape, const clv_kv_cache* cache, const void* q,
                                     const void* k_tree, const void* v_tree, const int32_t* parent,
                                     const int32_t* ctx_len, int32_t max_ctx_len, const void* out,
                                     const int32_t* status, const void* workspace, size_t workspace_bytes,
                                     AttnPlan* plan) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  st = check_cache(cache);
  if (st != CLV_OK) return st;
  if (!q || !k_tree || !v_tree || !parent || !ctx_len || !out || !status) return CLV_ERR_NULL;
  if (!aligned16(q) || !aligned16(k_tree) || !aligned16(v_tree) || !aligned16(out)) return CLV_ERR_ALIGN;
  if (max_ctx_len < 0) return CLV_ERR_SHAPE;
  if (shape->n_q_heads / shape->n_kv_heads > 128) return CLV_ERR_UNSUPPORTED;
  if (shape->batch > kTickets / 2) return CLV_ERR_UNSUPPORTED;   // two counters per sequence
  *plan = tc2_attn_wanted(*shape) ? tc2_attn_plan(*shape, max_ctx_len) : tc_attn_plan(*shape, max_ctx_len);
  if (!workspace || workspace_bytes < kWsFixedBytes + plan->scratch_bytes) return CLV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return CLV_ERR_ALIGN;
  if (!tc_attn_supported(*shape, *cache)) return CLV_ERR_UNSUPPORTED;   // asks the driver: last
  return CLV_OK;
}

clv_status clv_tree_attn(const clv_shape* shape, const clv_kv_cache* cache, const void* q,
                         const void* k_tree, const void* v_tree, const int32_t* parent,
                         const int32_t* ctx_len, int32_t max_ctx_len, float softmax_scale,
                         void* out, float* lse, int32_t* status, void* workspace,
                         size_t workspace_bytes, void* cuda_stream) {
  AttnPlan plan;
  const clv_status st = validate_tree_attn(shape, cache, q, k_tree, v_tree, parent, ctx_len, max_ctx_len,
                                           out, status, workspace, workspace_bytes, &plan);
  if (st != CLV_OK) return st;
  cudaError_t e = tc2_attn_wanted(*shape)
                      ? launch_tree_attn_tc2(plan, *shape, *cache, q, k_tree, v_tree, parent, ctx_len, softmax_scale,
                                             out, lse, status, ws_tickets(workspace), ws_scratch(workspace),
                                             static_cast<cudaStream_t>(cuda_stream))
                      : launch_tree_attn_tc(plan, *shape, *cache, q, k_tree, v_tree, parent, ctx_len, softmax_scale,
                                            out, lse, status, ws_tickets(workspace), ws_scratch(workspace),
                                            static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

static clv_status validate_accept_argmax(const clv_shape* shape, const void* logits, int64_t ld,
                                         const int32_t* argmax_ids, const void* workspace,
                                         size_t workspace_bytes, ArgmaxPlan* plan) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  if (!logits || !argmax_ids) return CLV_ERR_NULL;
  if (shape->vocab < 1 || ld < shape->vocab) return CLV_ERR_SHAPE;
  if (!aligned16(logits) || (ld % 8) != 0) return CLV_ERR_ALIGN;
  const int64_t rows = (int64_t)shape->batch * shape->n_nodes;
  if (rows > kTickets) return CLV_ERR_UNSUPPORTED;
  *plan = argmax_plan((int)rows, shape->vocab);
  if (plan->chunks > 1) {
    if (!workspace || workspace_bytes < kWsFixedBytes + plan->scratch_bytes) return CLV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return CLV_ERR_ALIGN;
  }
  return CLV_OK;
}

clv_status clv_accept_argmax(const clv_shape* shape, const void* logits, int64_t ld,
                             int32_t* argmax_ids, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
  ArgmaxPlan plan;
  const clv_status st = validate_accept_argmax(shape, logits, ld, argmax_ids, workspace, workspace_bytes, &plan);
  if (st != CLV_OK) return st;
  cudaError_t e = launch_argmax(plan, logits, ld, shape->vocab, argmax_ids,
                                workspace ? ws_tickets(workspace) : nullptr,
                                workspace ? ws_scratch(workspace) : nullptr,
                                static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_accept_argmax_noalloc(const clv_shape* shape, const void* logits, int64_t ld,
                                     int32_t* argmax_ids, void* cuda_stream) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  if (!logits || !argmax_ids) return CLV_ERR_NULL;
  if (shape->vocab < 1 || ld < shape->vocab) return CLV_ERR_SHAPE;
  if (!aligned16(logits) || (ld % 8) != 0) return CLV_ERR_ALIGN;
  const int64_t rows = (int64_t)shape->batch * shape->n_nodes;
  if (rows > INT32_MAX || !argmax_static_fits((int)rows, shape->vocab)) return CLV_ERR_TOO_LARGE;
  cudaError_t e = launch_argmax_static(logits, ld, (int)rows, shape->vocab, argmax_ids,
                                       static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

static bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
  return x < y + nb && y < x + na;
}

static clv_status validate_walk_commit(const clv_shape* shape, const clv_kv_cache* cache,
                                       const int32_t* parent, const int32_t* tokens, const int32_t* argmax_ids,
                                       const void* k_tree, const void* v_tree, const int32_t* ctx_len,
                                       const int32_t* accept_len, const int32_t* accept_idx,
                                       const int32_t* next_token, const int32_t* ctx_len_out,
                                       const int32_t* walk_status, const int32_t* commit_status) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  st = check_cache(cache);
  if (st != CLV_OK) return st;
  if (!parent || !tokens || !argmax_ids || !k_tree || !v_tree || !ctx_len || !accept_len || !accept_idx ||
      !next_token || !ctx_len_out || !walk_status || !commit_status)
    return CLV_ERR_NULL;
  if (!aligned16(k_tree) || !aligned16(v_tree)) return CLV_ERR_ALIGN;
  if (shape->path_cap < 1) return CLV_ERR_SHAPE;
  const size_t row = (size_t)shape->n_kv_heads * CLV_HEAD_DIM * 2;
  const size_t tree_bytes = (size_t)shape->batch * shape->n_nodes * row;
  const size_t cache_bytes = cache->paged ? (size_t)cache->n_pages * CLV_PAGE_SIZE * row
                                          : (size_t)shape->batch * cache->cap_tokens * row;
  if (overlaps(k_tree, tree_bytes, cache->k, cache_bytes) || overlaps(k_tree, tree_bytes, cache->v, cache_bytes) ||
      overlaps(v_tree, tree_bytes, cache->k, cache_bytes) || overlaps(v_tree, tree_bytes, cache->v, cache_bytes))
    return CLV_ERR_UNSUPPORTED;
  return CLV_OK;
}

clv_status clv_accept_walk_commit(const clv_shape* shape, const clv_kv_cache* cache,
                                  const int32_t* parent, const int32_t* tokens, const int32_t* argmax_ids,
                                  const void* k_tree, const void* v_tree, const int32_t* ctx_len,
                                  int32_t* accept_len, int32_t* accept_idx, int32_t* next_token,
                                  int32_t* ctx_len_out, int32_t* walk_status, int32_t* commit_status,
                                  void* cuda_stream) {
  const clv_status st = validate_walk_commit(shape, cache, parent, tokens, argmax_ids, k_tree, v_tree, ctx_len,
                                             accept_len, accept_idx, next_token, ctx_len_out, walk_status,
                                             commit_status);
  if (st != CLV_OK) return st;
  cudaError_t e = launch_walk_commit(*shape, *cache, parent, tokens, argmax_ids, k_tree, v_tree, ctx_len,
                                     accept_len, accept_idx, next_token, ctx_len_out, walk_status,
                                     commit_status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_accept_sample(const clv_shape* shape, const void* logits, int64_t ld, const int32_t* parent,
                             const int32_t* tokens, const float* uniforms, float temperature,
                             int32_t* accept_len, int32_t* accept_idx, int32_t* next_token, int32_t* status,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  if (!logits || !parent || !tokens || !uniforms || !accept_len || !accept_idx || !next_token || !status)
    return CLV_ERR_NULL;
  if (shape->vocab < 1 || ld < shape->vocab || shape->path_cap < 1) return CLV_ERR_SHAPE;
  if (!(temperature > 0.0f) || !(temperature < INFINITY)) return CLV_ERR_SHAPE;
  if (!aligned16(logits) || (ld % 8) != 0) return CLV_ERR_ALIGN;
  const int64_t rows = (int64_t)shape->batch * shape->n_nodes;
  if (rows > INT32_MAX / 64 || shape->vocab > sample_max_vocab()) return CLV_ERR_UNSUPPORTED;
  const size_t need = kWsFixedBytes + sample_scratch_bytes((int)rows, shape->vocab);
  if (!workspace || workspace_bytes < need) return CLV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return CLV_ERR_ALIGN;
  cudaError_t e = launch_accept_sample(*shape, logits, ld, parent, tokens, uniforms, temperature, accept_len,
                                       accept_idx, next_token, status, ws_scratch(workspace),
                                       static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_tree_to_intervals(int32_t batch, int32_t n_nodes, const int32_t* parent, int32_t* tin,
                                 int32_t* tout, int32_t* status, void* cuda_stream) {
  if (!parent || !tin || !tout || !status) return CLV_ERR_NULL;
  if (batch < 1 || n_nodes < 1) return CLV_ERR_SHAPE;
  if (n_nodes > CLV_MAX_NODES) return CLV_ERR_UNSUPPORTED;
  cudaError_t e = launch_tree_to_intervals(batch, n_nodes, parent, tin, tout, status,
                                           static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_tree_from_intervals(int32_t batch, int32_t n_nodes, const int32_t* tin, const int32_t* tout,
                                   int32_t* parent, int32_t* status, void* cuda_stream) {
  if (!parent || !tin || !tout || !status) return CLV_ERR_NULL;
  if (batch < 1 || n_nodes < 1) return CLV_ERR_SHAPE;
  if (n_nodes > CLV_MAX_NODES) return CLV_ERR_UNSUPPORTED;
  cudaError_t e = launch_tree_from_intervals(batch, n_nodes, tin, tout, parent, status,
                                             static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_kv_commit_layers(const clv_shape* shape, const clv_kv_cache* cache, int32_t n_layers,
                                int64_t cache_layer_stride, const void* k_tree, const void* v_tree,
                                int64_t tree_layer_stride, const int32_t* accept_idx, const int32_t* accept_len,
                                const int32_t* ctx_len, int32_t* ctx_len_out, int32_t* status, void* cuda_stream) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  st = check_cache(cache);
  if (st != CLV_OK) return st;
  if (!k_tree || !v_tree || !accept_idx || !accept_len || !ctx_len || !ctx_len_out || !status) return CLV_ERR_NULL;
  if (!aligned16(k_tree) || !aligned16(v_tree)) return CLV_ERR_ALIGN;
  if (shape->path_cap < 1 || n_layers < 1 || n_layers > 65535) return CLV_ERR_SHAPE;
  const int64_t row = (int64_t)shape->n_kv_heads * CLV_HEAD_DIM;   // elements per token row
  const int64_t tree_elems = (int64_t)shape->batch * shape->n_nodes * row;
  const int64_t cache_elems = cache->paged ? (int64_t)cache->n_pages * CLV_PAGE_SIZE * row
                                           : (int64_t)shape->batch * cache->cap_tokens * row;
  if (n_layers > 1 && (cache_layer_stride < cache_elems || tree_layer_stride < tree_elems)) return CLV_ERR_SHAPE;
  if ((cache_layer_stride % 8) != 0 || (tree_layer_stride % 8) != 0) return CLV_ERR_ALIGN;
  if (ctx_len_out == ctx_len) return CLV_ERR_UNSUPPORTED;   // every layer's block reads ctx_len
  const size_t tree_bytes = (size_t)(((int64_t)n_layers - 1) * tree_layer_stride + tree_elems) * 2;
  const size_t cache_bytes = (size_t)(((int64_t)n_layers - 1) * cache_layer_stride + cache_elems) * 2;
  if (overlaps(k_tree, tree_bytes, cache->k, cache_bytes) || overlaps(k_tree, tree_bytes, cache->v, cache_bytes) ||
      overlaps(v_tree, tree_bytes, cache->k, cache_bytes) || overlaps(v_tree, tree_bytes, cache->v, cache_bytes))
    return CLV_ERR_UNSUPPORTED;
  cudaError_t e = launch_commit_layers(*shape, *cache, n_layers, cache_layer_stride, k_tree, v_tree,
                                       tree_layer_stride, accept_idx, accept_len, ctx_len, ctx_len_out, status,
                                       static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

size_t clv_draft_head_workspace_bytes(int32_t rows, int32_t hidden_dim, int32_t vocab) {
  if (rows < 1 || hidden_dim < 1 || vocab < 1) return 0;
  return kWsFixedBytes + draft_head_scratch_bytes(rows, hidden_dim, vocab);
}

clv_status clv_draft_head_step(const clv_draft_head* head, int32_t rows, const void* h, const void* e,
                               int32_t k_top, void* hidden_out, int32_t* top_ids, float* top_logits,
                               int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!head || !h || !e || !hidden_out || !top_ids || !top_logits || !status) return CLV_ERR_NULL;
  if (!head->norm1 || !head->norm2 || !head->wq || !head->wk || !head->wv || !head->bq || !head->bk || !head->bv ||
      !head->wfc || !head->bfc || !head->lm_head)
    return CLV_ERR_NULL;
  const int H = head->hidden_dim;
  if (rows < 1 || H < 1 || head->n_heads < 1 || head->vocab < 1 || k_top < 1 || k_top > head->vocab) return CLV_ERR_SHAPE;
  if (!(head->rms_eps > 0.f)) return CLV_ERR_SHAPE;
  if (rows > 256 || (H % 64) != 0 || (H % head->n_heads) != 0 || ((H / head->n_heads) % 4) != 0 || k_top > 64)
    return CLV_ERR_UNSUPPORTED;
  if (!lm_head_supported(rows, H, head->vocab)) return CLV_ERR_UNSUPPORTED;
  const void* ptrs[] = {h, e, hidden_out, head->wq, head->wk, head->wv, head->wfc, head->lm_head, head->norm1,
                        head->norm2};
  for (const void* q : ptrs) if (!aligned16(q)) return CLV_ERR_ALIGN;
  if (!workspace || workspace_bytes < kWsFixedBytes + draft_head_scratch_bytes(rows, H, head->vocab))
    return CLV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return CLV_ERR_ALIGN;
  cudaError_t err = launch_draft_head_step(*head, rows, h, e, k_top, hidden_out, top_ids, top_logits, status,
                                           ws_tickets(workspace), ws_scratch(workspace),
                                           static_cast<cudaStream_t>(cuda_stream));
  return err == cudaSuccess ? CLV_OK : cuda_fail(err);
}

clv_status clv_build_token_tree(int32_t batch, int32_t n_cand, int32_t max_len, int32_t node_cap,
                                const int32_t* root_token, const int32_t* cand, const int32_t* cand_len,
                                int32_t* tokens, int32_t* parent, int32_t* n_nodes, int32_t* node_of,
                                int32_t* status, void* cuda_stream) {
  if (!root_token || !cand || !cand_len || !tokens || !parent || !n_nodes || !node_of || !status)
    return CLV_ERR_NULL;
  if (batch < 1 || n_cand < 1 || max_len < 1 || node_cap < 1) return CLV_ERR_SHAPE;
  if (n_cand > CLV_TREE_MAX_CAND || max_len > CLV_TREE_MAX_LEN || node_cap > CLV_MAX_NODES)
    return CLV_ERR_UNSUPPORTED;
  cudaError_t e = launch_token_tree(batch, n_cand, max_len, node_cap, root_token, cand, cand_len, tokens,
                                    parent, n_nodes, node_of, status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_lm_head_argmax(const void* hidden, int64_t ld_hidden, const void* weight,
                              int64_t ld_weight, int32_t rows, int32_t hidden_dim, int32_t vocab,
                              int32_t* argmax_ids, int32_t* status, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
  if (!hidden || !weight || !argmax_ids || !status) return CLV_ERR_NULL;
  if (rows < 1 || hidden_dim < 1 || vocab < 1 || ld_hidden < hidden_dim || ld_weight < hidden_dim)
    return CLV_ERR_SHAPE;
  if (!aligned16(hidden) || !aligned16(weight) || (ld_hidden % 8) != 0 || (ld_weight % 8) != 0)
    return CLV_ERR_ALIGN;
  if (!lm_head_supported(rows, hidden_dim, vocab)) return CLV_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < kWsFixedBytes) return CLV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return CLV_ERR_ALIGN;
  cudaError_t e = launch_lm_head_argmax(hidden, ld_hidden, weight, ld_weight, rows, hidden_dim, vocab,
                                        argmax_ids, status, ws_tickets(workspace),
                                        static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_accept_walk(const clv_shape* shape, const int32_t* parent, const int32_t* tokens,
                           const int32_t* argmax_ids, int32_t* accept_len, int32_t* accept_idx,
                           int32_t* next_token, int32_t* status, void* cuda_stream) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  if (!parent || !tokens || !argmax_ids || !accept_len || !accept_idx || !next_token || !status)
    return CLV_ERR_NULL;
  if (shape->path_cap < 1) return CLV_ERR_SHAPE;
  cudaError_t e = launch_walk(*shape, parent, tokens, argmax_ids, accept_len, accept_idx, next_token,
                              status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

clv_status clv_kv_commit(const clv_shape* shape, const clv_kv_cache* cache, const void* k_tree,
                         const void* v_tree, const int32_t* accept_idx, const int32_t* accept_len,
                         const int32_t* ctx_len, int32_t* ctx_len_out, int32_t* status,
                         void* cuda_stream) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  st = check_cache(cache);
  if (st != CLV_OK) return st;
  if (!k_tree || !v_tree || !accept_idx || !accept_len || !ctx_len || !ctx_len_out || !status)
    return CLV_ERR_NULL;
  if (!aligned16(k_tree) || !aligned16(v_tree)) return CLV_ERR_ALIGN;
  if (shape->path_cap < 1) return CLV_ERR_SHAPE;
  const size_t row = (size_t)shape->n_kv_heads * CLV_HEAD_DIM * 2;
  const size_t tree_bytes = (size_t)shape->batch * shape->n_nodes * row;
  const size_t cache_bytes = cache->paged ? (size_t)cache->n_pages * CLV_PAGE_SIZE * row
                                          : (size_t)shape->batch * cache->cap_tokens * row;
  if (overlaps(k_tree, tree_bytes, cache->k, cache_bytes) ||
      overlaps(k_tree, tree_bytes, cache->v, cache_bytes) ||
      overlaps(v_tree, tree_bytes, cache->k, cache_bytes) ||
      overlaps(v_tree, tree_bytes, cache->v, cache_bytes))
    return CLV_ERR_UNSUPPORTED;  // a destination row could be another thread's source row
  cudaError_t e = launch_commit(*shape, *cache, k_tree, v_tree, accept_idx, accept_len, ctx_len,
                                ctx_len_out, status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CLV_OK : cuda_fail(e);
}

// ---- whole step from host buffers ---------------------------------------------------------------
namespace {
struct Staging {
  size_t q, k_tree, v_tree, parent, tokens, logits, out, ids, alen, aidx, next, status, total;
};
Staging staging_layout(const clv_shape& s, int64_t ld) {
  Staging L;
  const size_t B = s.batch, N = s.n_nodes;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += round_up(bytes, 256); return at; };
  L.q = take(B * N * s.n_q_heads * CLV_HEAD_DIM * 2);
  L.k_tree = take(B * N * s.n_kv_heads * CLV_HEAD_DIM * 2);
  L.v_tree = take(B * N * s.n_kv_heads * CLV_HEAD_DIM * 2);
  L.parent = take(B * N * 4);
  L.tokens = take(B * N * 4);
  L.logits = take(B * N * (size_t)ld * 2);
  L.out = take(B * N * s.n_q_heads * CLV_HEAD_DIM * 2);
  L.ids = take(B * N * 4);
  L.alen = take(B * 4);
  L.aidx = take(B * (size_t)s.path_cap * 4);
  L.next = take(B * 4);
  L.status = take(3 * B * 4);
  L.total = o;
  return L;
}
}  // namespace

size_t clv_staging_bytes(const clv_shape* shape, int64_t ld) {
  if (check_shape(shape) != CLV_OK || ld < 1 || shape->path_cap < 1) return 0;
  return staging_layout(*shape, ld).total;
}

clv_status clv_verify_step_host(const clv_shape* shape, const clv_kv_cache* cache,
                                const clv_host_inputs* in, const clv_host_outputs* out,
                                int32_t* ctx_len, int32_t max_ctx_len, float softmax_scale,
                                void* staging, size_t staging_bytes, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
  clv_status st = check_shape(shape);
  if (st != CLV_OK) return st;
  if (!in || !out || !ctx_len || !staging) return CLV_ERR_NULL;
  if (!in->q || !in->k_tree || !in->v_tree || !in->parent || !in->tokens || !in->logits ||
      !out->out || !out->argmax_ids || !out->accept_len || !out->accept_idx || !out->next_token ||
      !out->status)
    return CLV_ERR_NULL;
  if (shape->path_cap < 1 || in->ld < shape->vocab || shape->vocab < 1) return CLV_ERR_SHAPE;
  if (!aligned16(staging)) return CLV_ERR_ALIGN;
  const Staging L = staging_layout(*shape, in->ld);
  if (staging_bytes < L.total) return CLV_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* d = static_cast<char*>(staging);
  const size_t B = shape->batch, N = shape->n_nodes;
  const size_t qb = B * N * shape->n_q_heads * CLV_HEAD_DIM * 2;
  const size_t tb = B * N * shape->n_kv_heads * CLV_HEAD_DIM * 2;
  int32_t* const dstat = reinterpret_cast<int32_t*>(d + L.status);
  // every check of the three calls first: a mistake the host can see must leave the stream empty
  AttnPlan attn_plan_unused;
  ArgmaxPlan argmax_plan_unused;
  st = validate_tree_attn(shape, cache, d + L.q, d + L.k_tree, d + L.v_tree,
                          reinterpret_cast<int32_t*>(d + L.parent), ctx_len, max_ctx_len, d + L.out, dstat,
                          workspace, workspace_bytes, &attn_plan_unused);
  if (st != CLV_OK) return st;
  st = validate_accept_argmax(shape, d + L.logits, in->ld, reinterpret_cast<int32_t*>(d + L.ids), workspace,
                              workspace_bytes, &argmax_plan_unused);
  if (st != CLV_OK) return st;
  st = validate_walk_commit(shape, cache, reinterpret_cast<int32_t*>(d + L.parent),
                            reinterpret_cast<int32_t*>(d + L.tokens), reinterpret_cast<int32_t*>(d + L.ids),
                            d + L.k_tree, d + L.v_tree, ctx_len, reinterpret_cast<int32_t*>(d + L.alen),
                            reinterpret_cast<int32_t*>(d + L.aidx), reinterpret_cast<int32_t*>(d + L.next),
                            ctx_len, dstat + B, dstat + 2 * B);
  if (st != CLV_OK) return st;
  cudaError_t e;
#define CLV_COPY(dst, src, n, kind) \
  if ((e = cudaMemcpyAsync(dst, src, n, kind, s)) != cudaSuccess) return cuda_fail(e)
  CLV_COPY(d + L.q, in->q, qb, cudaMemcpyHostToDevice);
  CLV_COPY(d + L.k_tree, in->k_tree, tb, cudaMemcpyHostToDevice);
  CLV_COPY(d + L.v_tree, in->v_tree, tb, cudaMemcpyHostToDevice);
  CLV_COPY(d + L.parent, in->parent, B * N * 4, cudaMemcpyHostToDevice);
  CLV_COPY(d + L.tokens, in->tokens, B * N * 4, cudaMemcpyHostToDevice);
  CLV_COPY(d + L.logits, in->logits, B * N * (size_t)in->ld * 2, cudaMemcpyHostToDevice);
  st = clv_tree_attn(shape, cache, d + L.q, d + L.k_tree, d + L.v_tree,
                     reinterpret_cast<int32_t*>(d + L.parent), ctx_len, max_ctx_len, softmax_scale,
                     d + L.out, nullptr, dstat, workspace, workspace_bytes, cuda_stream);
  if (st != CLV_OK) return st;
  st = clv_accept_argmax(shape, d + L.logits, in->ld, reinterpret_cast<int32_t*>(d + L.ids),
                         workspace, workspace_bytes, cuda_stream);
  if (st != CLV_OK) return st;
  st = clv_accept_walk_commit(shape, cache, reinterpret_cast<int32_t*>(d + L.parent),
                              reinterpret_cast<int32_t*>(d + L.tokens), reinterpret_cast<int32_t*>(d + L.ids),
                              d + L.k_tree, d + L.v_tree, ctx_len, reinterpret_cast<int32_t*>(d + L.alen),
                              reinterpret_cast<int32_t*>(d + L.aidx), reinterpret_cast<int32_t*>(d + L.next),
                              ctx_len, dstat + B, dstat + 2 * B, cuda_stream);
  if (st != CLV_OK) return st;
  CLV_COPY(out->out, d + L.out, qb, cudaMemcpyDeviceToHost);
  CLV_COPY(out->argmax_ids, d + L.ids, B * N * 4, cudaMemcpyDeviceToHost);
  CLV_COPY(out->accept_len, d + L.alen, B * 4, cudaMemcpyDeviceToHost);
  CLV_COPY(out->accept_idx, d + L.aidx, B * (size_t)shape->path_cap * 4, cudaMemcpyDeviceToHost);
  CLV_COPY(out->next_token, d + L.next, B * 4, cudaMemcpyDeviceToHost);
  CLV_COPY(out->status, d + L.status, 3 * B * 4, cudaMemcpyDeviceToHost);
#undef CLV_COPY
  return CLV_OK;
}

const char* clv_status_string(clv_status s) {
  switch (s) {
    case CLV_OK: return "ok";
    case CLV_ERR_NULL: return "a required pointer is NULL";
    case CLV_ERR_SHAPE: return "invalid shape";
    case CLV_ERR_UNSUPPORTED: return "unsupported configuration";
    case CLV_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case CLV_ERR_WORKSPACE: return "workspace missing or too small";
    case CLV_ERR_CUDA: return "CUDA runtime error";
    case CLV_ERR_TREE: return "malformed tree or capacity exceeded";
    case CLV_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case CLV_ERR_TOO_LARGE: return "problem exceeds the fixed built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

int clv_last_cuda_error(void) { return g_last_cuda_error; }

void clv_test_set_wait_limit(int64_t sm_cycles) {
  g_wait_limit.store(sm_cycles > 0 ? (long long)sm_cycles : 2000000000ll, std::memory_order_relaxed);
}
int clv_version(void) { return 111; }

}  // extern "C"
