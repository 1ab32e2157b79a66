/*
 * clv - tree verification for Clover-2-style speculative decoding on one B200 (sm_100a).
 *
 * The library implements the target model's verification step that the paper describes in
 * Sec. 2.1 ("Speculative Decoding and Tree Attention"): the target ingests all N tokens of a draft
 * token tree at once, attention uses the tree's topology matrix as its causal mask, wrong drafts
 * are filtered out, and the result equals plain decoding.  Four stream-ordered calls cover it:
 *
 *   clv_tree_attn      tree-masked attention of the N tree tokens against the committed KV cache
 *                      and against their own ancestors            (Sec. 2.1, Fig. 2 caption;
 *                      the mask is derived from parent[] on chip, cf. App. A.1 "compressed tree
 *                      mask": the N x N matrix never exists in memory)
 *   clv_accept_argmax  the target's greedy choice per tree node   (Sec. 4.2: temperature 0 is
 *                      greedy decoding of the target)
 *   clv_accept_walk    longest root-to-node path the target agrees with (Sec. 2.1 verification
 *                      phase; greedy rule of the tree-sampling algorithm adopted in Sec. 4.1)
 *   clv_kv_commit      append the accepted nodes' K/V rows to the cache (implied by the
 *                      equivalence requirement of Sec. 2.1: afterwards the cache holds what plain
 *                      decoding of the accepted tokens would hold)
 *
 * Conventions
 *   - Plain C ABI.  Every pointer is a DEVICE pointer unless the comment says "host".
 *     The two descriptor structs live in host memory and are read during the call only.
 *   - The caller owns every buffer, including the workspace.  The library allocates no device
 *     memory, never synchronises, and only enqueues work on the given stream (a cudaStream_t
 *     passed as void*; NULL = the legacy default stream).
 *   - Inputs are const.  Only the documented outputs are written; clv_kv_commit writes cache
 *     rows [ctx_len[b], ctx_len[b] + accept_len[b]) of each sequence and nothing else.
 *   - bf16 tensors are dense, innermost dimension contiguous, base 16-byte aligned.
 *   - Host-detectable mistakes return an error code and enqueue nothing.  Mistakes only the
 *     device can see (a malformed parent[], a context that does not fit its capacity, an invalid
 *     block-table entry) never trap: the sequence is skipped and CLV_ERR_TREE is written to its
 *     slot of the caller's int32 status[batch] array (0 = fine).
 *   - Notation: B sequences, N tree nodes per sequence (node 0 = root = the last token the target
 *     emitted; parent[b][0] = -1, parent[b][i] in [0, i)), Hq query heads, Hkv KV heads,
 *     G = Hq / Hkv, D = 128, L_b = ctx_len[b] committed tokens.
 */
#ifndef CLV_H_
#define CLV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t clv_status;
enum {
  CLV_OK = 0,
  CLV_ERR_NULL = 1,        /* a required pointer is NULL                                        */
  CLV_ERR_SHAPE = 2,       /* non-positive size, Hq not a multiple of Hkv, ld < vocab, ...      */
  CLV_ERR_UNSUPPORTED = 3, /* head_dim != 128, n_nodes > 128, page_size != 64, forbidden alias  */
  CLV_ERR_ALIGN = 4,       /* a tensor base (or logits row stride) is not 16-byte aligned       */
  CLV_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than clv_workspace_bytes()              */
  CLV_ERR_CUDA = 6,        /* a CUDA runtime call failed; see clv_last_cuda_error()             */
  CLV_ERR_TREE = 7,        /* device status[] only: malformed tree or capacity exceeded         */
  CLV_ERR_TIMEOUT = 8,     /* device status[] only: a bounded on-chip wait gave up              */
  CLV_ERR_TOO_LARGE = 9    /* clv_accept_argmax_noalloc: the problem exceeds its built-in scratch */
};

#define CLV_MAX_NODES 128
#define CLV_TREE_MAX_CAND 128 /* clv_build_token_tree: speculated sequences per tree */
#define CLV_TREE_MAX_LEN 16   /* clv_build_token_tree: tokens per speculated sequence */
#define CLV_HEAD_DIM 128
#define CLV_PAGE_SIZE 64

/* Shape of one verify step (host memory). */
typedef struct {
  int32_t batch;      /* B >= 1                                                    */
  int32_t n_nodes;    /* N in [1, 128]                                             */
  int32_t n_q_heads;  /* Hq, a multiple of n_kv_heads                              */
  int32_t n_kv_heads; /* Hkv                                                       */
  int32_t head_dim;   /* must be 128                                               */
  int32_t vocab;      /* V, used by clv_accept_argmax only                         */
  int32_t path_cap;   /* columns of accept_idx; >= (maximum tree depth + 1)        */
} clv_shape;

/* KV cache descriptor (host memory; k, v and block_table are device pointers). */
typedef struct {
  void* k;            /* contiguous: [B, cap_tokens, Hkv, 128] bf16                          */
  void* v;            /* paged:      [n_pages, 64, Hkv, 128] bf16                            */
  int32_t paged;      /* 0 contiguous, 1 paged                                               */
  int32_t cap_tokens; /* contiguous: rows per sequence                                       */
  int32_t page_size;  /* paged: must be 64                                                   */
  int32_t n_pages;    /* paged: pages in the pool                                            */
  int32_t max_pages_per_seq;  /* paged: columns of block_table                               */
  const int32_t* block_table; /* paged: [B, max_pages_per_seq], logical page -> pool page    */
} clv_kv_cache;

/*
 * Workspace.  clv_tree_attn and clv_accept_argmax split their work over more thread blocks than
 * there are independent outputs and combine the pieces through the workspace.
 * clv_workspace_bytes: bytes needed for this shape with contexts up to max_ctx_len (host call).
 * clv_workspace_init : must be enqueued ONCE on a fresh workspace before its first use (it clears
 *                      the arrival counters; every call leaves them cleared again).  One workspace
 *                      serves both calls and any shape it is large enough for, but calls that
 *                      share a workspace must not overlap on the device.
 */
size_t clv_workspace_bytes(const clv_shape* shape, const clv_kv_cache* cache, int32_t max_ctx_len);
clv_status clv_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Tree attention (Sec. 2.1; Fig. 2 caption).  For every sequence b, node i and query head h:
 *   keys   = cache rows 0 .. L_b-1 of kv head h / G, then the tree rows j that are i itself or an
 *            ancestor of i (row i of the tree's topology matrix),
 *   out    = softmax(softmax_scale * q . k) . v   over those keys, fp32 accumulation, rounded to
 *            bf16 (nearest even);   lse = natural-log sum-exp of the scaled scores (optional).
 * q/k are taken as given (rotary positions L_b + depth(i) are the caller's business).
 * Several roots (extra -1 parents) are accepted here.  L_b = 0 is allowed.
 * status[b] = CLV_ERR_TREE if parent[b] is malformed, L_b < 0, L_b exceeds the cache capacity or
 * a needed block-table entry is outside [0, n_pages); CLV_ERR_TIMEOUT if a bounded on-chip wait of
 * one of the sequence's thread blocks ran out (about a second; never seen on a healthy device);
 * CLV_OK otherwise.  With a non-zero status that sequence's outputs are unspecified; the word is
 * written once per call, by the last thread block of the sequence to finish.
 * max_ctx_len (host): an upper bound of ctx_len[], used only to choose the split count; the
 * result does not depend on it.
 * workspace: required (CLV_ERR_WORKSPACE), at least clv_workspace_bytes(); batch <= 32768.
 * Group sizes G above 128 are refused with CLV_ERR_UNSUPPORTED.
 */
clv_status clv_tree_attn(const clv_shape* shape, const clv_kv_cache* cache,
                         const void* q,        /* bf16 [B, N, Hq, 128]            */
                         const void* k_tree,   /* bf16 [B, N, Hkv, 128]           */
                         const void* v_tree,   /* bf16 [B, N, Hkv, 128]           */
                         const int32_t* parent,  /* [B, N]                        */
                         const int32_t* ctx_len, /* [B]                           */
                         int32_t max_ctx_len, float softmax_scale,
                         void* out,            /* bf16 [B, N, Hq, 128]            */
                         float* lse,           /* fp32 [B, N, Hq] or NULL         */
                         int32_t* status,      /* [B]                             */
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Greedy target choice (Sec. 4.2, temperature 0): argmax_ids[b][i] = the lowest v that maximises
 * logits[b][i][v], v < vocab.  +0 and -0 compare equal; NaN entries are ignored (treated as
 * -infinity); a row of only -infinity/NaN gives 0.  ld = row stride in elements, a multiple of 8.
 */
clv_status clv_accept_argmax(const clv_shape* shape,
                             const void* logits, /* bf16 [B*N, ld]               */
                             int64_t ld,
                             int32_t* argmax_ids, /* [B, N]                      */
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * clv_accept_argmax without any caller-provided scratch.  The paper has no counterpart to this
 * entry point; it exists for integration reasons only.  Some hosts of this library may not
 * allocate device memory when they call it: code running inside a serving engine that handed all
 * of the GPU's memory to its own pool at start-up, a plug-in that is only ever given input and
 * output tensors, or a caller on a latency path where cudaMalloc's implicit synchronisation is
 * not acceptable.  For them the arrival counters and per-chunk partial results live in a fixed
 * array inside the library's device image instead of a workspace.
 *   - Same inputs, outputs and result as clv_accept_argmax (bit-identical ids).
 *   - Limit: B * N <= 4096 rows and rows * (thread blocks per row) <= 131072, where a row is cut
 *     into at most ceil(vocab / 2048) thread blocks: B * N * ceil(vocab / 2048) <= 131072 always
 *     fits.  Anything larger is refused with CLV_ERR_TOO_LARGE and nothing is enqueued.  The
 *     array is about 1.04 MB and stays resident on every GPU that loads the library until the
 *     process exits.
 *   - The call allocates and frees nothing (no cudaMalloc / cudaFree, no allocating library
 *     routine).  The first call on a device looks up the array's device address (with that device
 *     current) and remembers it; make that first call outside of any stream capture.
 *   - All calls on one GPU share the array, and it keeps the previous call's contents; each call
 *     clears the counters it needs on the given stream first.  Two calls that overlap on the GPU
 *     (different streams, or different host threads without ordering) race on it: serialise them.
 */
clv_status clv_accept_argmax_noalloc(const clv_shape* shape,
                                     const void* logits, /* bf16 [B*N, ld]       */
                                     int64_t ld,
                                     int32_t* argmax_ids, /* [B, N]              */
                                     void* cuda_stream);

/*
 * clv_accept_walk followed by clv_kv_commit in one launch (Sec. 2.1: the verification keeps the
 * drafts the target agrees with, and the cache must afterwards equal plain decoding's): a thread
 * block per sequence walks the tree and then copies the accepted rows.  Arguments, results, error
 * codes and per-sequence statuses are those of the two calls (walk_status as clv_accept_walk's
 * status, commit_status as clv_kv_commit's); the result is identical to calling them in turn.
 */
clv_status clv_accept_walk_commit(const clv_shape* shape, const clv_kv_cache* cache,
                                  const int32_t* parent, const int32_t* tokens,
                                  const int32_t* argmax_ids,
                                  const void* k_tree, const void* v_tree, const int32_t* ctx_len,
                                  int32_t* accept_len, int32_t* accept_idx, int32_t* next_token,
                                  int32_t* ctx_len_out, int32_t* walk_status, int32_t* commit_status,
                                  void* cuda_stream);

/*
 * Stochastic acceptance at temperature T > 0 (Sec. 4.1 / 4.2, Table 1 "Temperature = 1": the paper
 * uses its baseline's tree sampling algorithm and prints no formula; the reading taken is
 * speculative sampling for drafts that are proposed deterministically, one token per child).
 * For every sequence, starting at the root (always accepted): p = softmax(logits[cur] / T); the
 * children of the current node are tried in increasing node index, child c with token x being
 * accepted if  uniforms[b][c] < p(x) / (1 - mass of the tokens rejected at this node so far);
 * an accepted child becomes current, a rejected token is struck from p.  When every child is
 * rejected (or there is none), next_token = the first v, in vocabulary order and not struck, whose
 * running sum of p exceeds uniforms[b][N] * (mass left).  The tokens emitted this way follow the
 * target's distribution exactly, whatever the drafts.  Use clv_kv_commit on the result as after
 * clv_accept_walk.
 * logits: device, bf16 [B*N, ld] as for clv_accept_argmax (no NaN: a precondition; the kernels
 * give such an entry no probability);
 * uniforms: device, fp32 [B, N + 1], every value in [0, 1), supplied by the caller (the library
 * draws no random numbers); temperature: host, finite and > 0.
 * accept_len / accept_idx / next_token / status: as clv_accept_walk (status CLV_ERR_TREE for a
 * malformed parent[] or a path longer than path_cap; next_token -1 then, and also for a row
 * without any probability mass).  Arithmetic: fp32 with hardware exp2; a decision whose uniform
 * lies within rounding distance of its threshold (relative 1e-5) may fall either way.
 * workspace: as returned by clv_workspace_bytes for this shape (with vocab set), initialised.
 * Errors: CLV_ERR_NULL, CLV_ERR_SHAPE (also temperature <= 0), CLV_ERR_ALIGN, CLV_ERR_WORKSPACE,
 * CLV_ERR_UNSUPPORTED (vocab above 1048576, or too many rows).
 */
clv_status clv_accept_sample(const clv_shape* shape,
                             const void* logits, /* bf16 [B*N, ld] */
                             int64_t ld,
                             const int32_t* parent, const int32_t* tokens, /* [B, N] */
                             const float* uniforms,                        /* [B, N + 1] */
                             float temperature,
                             int32_t* accept_len, int32_t* accept_idx, int32_t* next_token,
                             int32_t* status,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The compressed, linear form of the tree mask (App. A.1: a mask that is a numerical comparison
 * instead of an N x N matrix; the figure is missing, the encoding taken is depth-first entry/exit
 * labels).  tin[b][i] = position of node i in a depth-first walk of the tree that visits children
 * in increasing node index (several roots one after the other), tout = tin + size of the node's
 * subtree; node j is an ancestor of node i, or i itself, exactly if tin[j] <= tin[i] < tout[j].
 * clv_tree_to_intervals writes the labels of parent[]; clv_tree_from_intervals gives parent[]
 * back from any labels that nest properly (parent of i = the node with the narrowest interval
 * around tin[i]), so that a caller holding labels can feed clv_tree_attn, the walk and the commit.
 * All arrays: device, int32 [B, N], N <= 128.  status[b] = CLV_ERR_TREE (outputs of that sequence
 * all -1) for a malformed parent[] (parent[i] >= i or < -1), or for labels that are not those of a
 * forest in topological node order: an empty interval, two equal tin, intervals that overlap
 * without nesting, a parent that would not come before its child.
 */
clv_status clv_tree_to_intervals(int32_t batch, int32_t n_nodes, const int32_t* parent,
                                 int32_t* tin, int32_t* tout, int32_t* status, void* cuda_stream);
clv_status clv_tree_from_intervals(int32_t batch, int32_t n_nodes, const int32_t* tin, const int32_t* tout,
                                   int32_t* parent, int32_t* status, void* cuda_stream);

/*
 * clv_kv_commit for all layers of a model in one launch (Sec. 2.1: attention is the only block
 * with a sequence dependency, so a verify step runs clv_tree_attn once per layer and can defer the
 * commit of every layer's accepted rows to the end of the step).  Layer l's cache buffers start
 * cache_layer_stride elements (bf16) after layer l-1's - `cache` describes layer 0 -, its tree
 * K/V tree_layer_stride elements after layer l-1's; all layers share accept_idx / accept_len,
 * ctx_len and, for a paged cache, the block table.  Results per layer are those of clv_kv_commit;
 * status and ctx_len_out are written once per sequence (the same for every layer).  Both strides
 * must be multiples of 8 and at least the size of one layer's buffer; ctx_len_out must not alias
 * ctx_len here (CLV_ERR_UNSUPPORTED), nor may tree and cache buffers overlap.
 */
clv_status clv_kv_commit_layers(const clv_shape* shape, const clv_kv_cache* cache, int32_t n_layers,
                                int64_t cache_layer_stride,
                                const void* k_tree, const void* v_tree, int64_t tree_layer_stride,
                                const int32_t* accept_idx, const int32_t* accept_len,
                                const int32_t* ctx_len, int32_t* ctx_len_out, int32_t* status,
                                void* cuda_stream);

/*
 * One step of a Clover-2 draft head (Sec. 3.1 "Attention Decoder output projector", "Other
 * Details"; App. A.3 prints the Attention Decoder) for `rows` rows, one per sequence and candidate:
 *   x = RMSNorm(h; norm1);  q = x wq^T + bq;  k = e wk^T + bk;  v = e wv^T + bv;
 *   per head j (hidden_dim / n_heads consecutive features):
 *       gate_j = <q_j, k_j> / max(|q_j| |k_j|, 1e-8);      a = h + v * gate   (no activation)
 *   p = [a, e] wfc^T + bfc             (the fully connected output projector over the decoder's
 *                                       output and the token embedding)
 *   logits = RMSNorm(p; norm2) lm_head^T;   top_ids / top_logits = the k_top largest logits of each
 *   row, highest first, lower index first among equals;   hidden_out = p (bf16), the hidden state
 *   the next head regresses on.
 * h: the target's last hidden state (first head) or the previous head's hidden_out; e: embedding
 * of the previously emitted token (the paper takes it from the transposed LM head).  The paper's
 * listing names its norm inconsistently and cuts one line short; the reading taken is RMSNorm
 * (eps = rms_eps) before the q projection and before the LM head, linear layers with bias.
 * Arithmetic: the operands of every product are bf16 (x, a, RMSNorm(p) are rounded once), sums,
 * gates and logits fp32 (tensor cores).  All pointers device; h, e, hidden_out bf16 [rows,
 * hidden_dim]; top_ids int32 and top_logits fp32 [rows, k_top]; status int32 [5] (one word per
 * product: CLV_OK or CLV_ERR_TIMEOUT).  rows <= 256, hidden_dim a multiple of 64 and of n_heads,
 * the head size hidden_dim / n_heads a multiple of 4, 1 <= k_top <= 64 (up to 32 the selection
 * is one pass over the logits; beyond, k_top passes).  h, e, hidden_out, the weight matrices and
 * the two norm gains start on 16-byte boundaries (CLV_ERR_ALIGN otherwise); biases may start
 * anywhere (16-byte aligned ones are read faster).  workspace: at least
 * clv_draft_head_workspace_bytes(), initialised with clv_workspace_init; it holds every
 * intermediate (the caller owns it and must not share it between calls that may overlap).  A
 * NaN logit ranks after every number; if a row has fewer than k_top entries (vocab < k_top is
 * rejected, so this never happens) the missing ids would read -1.  The step streams every weight
 * once (1.22 GB at hidden 4096, vocabulary 128256) and is bound by that.
 * Errors: CLV_ERR_NULL, CLV_ERR_SHAPE (a size below 1, k_top > vocab, rms_eps <= 0),
 * CLV_ERR_UNSUPPORTED (the limits above, no tensor-map support in the driver), CLV_ERR_ALIGN,
 * CLV_ERR_WORKSPACE, CLV_ERR_CUDA.  Nothing is launched on an error.
 */
typedef struct {
  int32_t hidden_dim, n_heads, vocab;
  float rms_eps;
  const void* norm1; const void* norm2;                 /* bf16 [hidden_dim]                  */
  const void* wq; const void* wk; const void* wv;       /* bf16 [hidden_dim, hidden_dim]      */
  const void* bq; const void* bk; const void* bv;       /* bf16 [hidden_dim]                  */
  const void* wfc;                                      /* bf16 [hidden_dim, 2 * hidden_dim]  */
  const void* bfc;                                      /* bf16 [hidden_dim]                  */
  const void* lm_head;                                  /* bf16 [vocab, hidden_dim]           */
} clv_draft_head;

size_t clv_draft_head_workspace_bytes(int32_t rows, int32_t hidden_dim, int32_t vocab);
clv_status clv_draft_head_step(const clv_draft_head* head, int32_t rows,
                               const void* h, const void* e, int32_t k_top,
                               void* hidden_out, int32_t* top_ids, float* top_logits, int32_t* status,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * LM head fused with the greedy choice (Sec. 3.1: the target's final norm and LM head produce the
 * logits of every tree node; Sec. 4.2: greedy decoding at temperature 0):
 *   argmax_ids[r] = the lowest v that maximises round_bf16(sum_k hidden[r][k] * weight[v][k]),
 * the products accumulated in fp32 and the logit rounded to bf16 (round to nearest even) before
 * the comparison, as a bf16 logits tensor would hold it.  The logits are never written to memory.
 * hidden: device, bf16 [rows, ld_hidden], already normalised; weight: device, bf16
 * [vocab, ld_weight] (one row per vocabulary entry); hidden_dim must be a multiple of 64, both
 * row strides multiples of 8 elements, both bases 16-byte aligned.  rows <= 32767.
 * status: device, one int32: CLV_OK, or CLV_ERR_TIMEOUT if a bounded wait inside the kernel ran
 * out (argmax_ids is then unspecified).  workspace: as returned by clv_workspace_bytes for any
 * shape, initialised with clv_workspace_init; the caller owns every buffer.  NaN logits are
 * ignored; a row without any finite or infinite logit gives 0.
 * Errors: CLV_ERR_NULL, CLV_ERR_SHAPE, CLV_ERR_ALIGN, CLV_ERR_UNSUPPORTED (hidden_dim not a
 * multiple of 64, too many rows, no tensor-map support in the driver), CLV_ERR_WORKSPACE,
 * CLV_ERR_CUDA.  Nothing is launched on an error.
 */
clv_status clv_lm_head_argmax(const void* hidden, int64_t ld_hidden,
                              const void* weight, int64_t ld_weight,
                              int32_t rows, int32_t hidden_dim, int32_t vocab,
                              int32_t* argmax_ids,   /* [rows] */
                              int32_t* status,       /* [1]    */
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Token tree from speculated sequences (Sec. 2.1 and the caption of Fig. 2: the speculations are
 * merged by prefix matching into a tree).  For every sequence b, n_cand candidate continuations
 * cand[b][c][0 .. cand_len[b][c]) of the root token are merged: a node is a distinct non-empty
 * prefix of some candidate; node 0 is the root and carries root_token[b] with parent -1.  Nodes
 * are numbered by depth first and, within a depth, by the lowest candidate index that contains the
 * prefix, so parent[i] < i and the result is unique.  Siblings carry distinct tokens by
 * construction.  Slots n_nodes[b] .. node_cap-1 are padding: parent 0, token -1 (no target token
 * matches them), so tokens/parent can be given to clv_tree_attn / clv_accept_walk with
 * n_nodes = node_cap unchanged.  node_of[b][c][d] = the node of candidate c's prefix of length
 * d+1, or -1 where d >= cand_len[b][c].
 * All pointers are device pointers; int32; layouts [B], [B, n_cand, max_len], [B, n_cand],
 * [B, node_cap], [B, node_cap], [B], [B, n_cand, max_len], [B].
 * status[b] = CLV_ERR_TREE if a cand_len is outside [0, max_len] or the tree needs more than
 * node_cap nodes: then n_nodes[b] = 1, the tree is the root plus padding, node_of is all -1.
 * Limits: 1 <= n_cand <= CLV_TREE_MAX_CAND, 1 <= max_len <= CLV_TREE_MAX_LEN,
 * 1 <= node_cap <= CLV_MAX_NODES (CLV_ERR_UNSUPPORTED beyond).  Nothing is launched on an error.
 */
clv_status clv_build_token_tree(int32_t batch, int32_t n_cand, int32_t max_len, int32_t node_cap,
                                const int32_t* root_token, const int32_t* cand,
                                const int32_t* cand_len,
                                int32_t* tokens, int32_t* parent, int32_t* n_nodes,
                                int32_t* node_of, int32_t* status, void* cuda_stream);

/*
 * Greedy acceptance walk (Sec. 2.1 verification phase; Sec. 4.1).  Start at the root; at node cur
 * the target wants argmax_ids[cur]; the child of cur whose drafted token equals it (the lowest
 * index if siblings repeat a token) is accepted and becomes cur; otherwise stop.
 *   accept_len[b]  nodes on the accepted path, root included (>= 1)
 *   accept_idx[b]  their node indices in path order, padded with -1 to path_cap columns
 *   next_token[b]  argmax_ids of the last accepted node (the token the target emits next)
 * status[b] = CLV_ERR_TREE when parent[b] is malformed (node 0 must be the only root) or the path
 * does not fit path_cap; then accept_len = 0, next_token = -1, accept_idx = -1.
 */
clv_status clv_accept_walk(const clv_shape* shape, const int32_t* parent /* [B,N] */,
                           const int32_t* tokens /* [B,N] */, const int32_t* argmax_ids /* [B,N] */,
                           int32_t* accept_len /* [B] */, int32_t* accept_idx /* [B,path_cap] */,
                           int32_t* next_token /* [B] */, int32_t* status /* [B] */,
                           void* cuda_stream);

/*
 * KV commit (from the equivalence requirement of Sec. 2.1).  For j < accept_len[b]:
 *   cache row (L_b + j)  <-  tree row accept_idx[b][j], K and V, all Hkv heads;
 *   ctx_len_out[b] = L_b + accept_len[b]   (ctx_len_out may be the same array as ctx_len).
 * k_tree / v_tree must not overlap the cache buffers (CLV_ERR_UNSUPPORTED if they do).
 * status[b] = CLV_ERR_TREE and the sequence is left untouched (ctx_len_out[b] = L_b) if the rows
 * do not fit (contiguous: cap_tokens; paged: block-table entry missing or invalid) or accept_len /
 * accept_idx are out of range.
 */
clv_status clv_kv_commit(const clv_shape* shape, const clv_kv_cache* cache,
                         const void* k_tree, const void* v_tree, /* bf16 [B, N, Hkv, 128] */
                         const int32_t* accept_idx /* [B,path_cap] */,
                         const int32_t* accept_len /* [B] */, const int32_t* ctx_len /* [B] */,
                         int32_t* ctx_len_out /* [B] */, int32_t* status /* [B] */,
                         void* cuda_stream);

/*
 * One whole verify step from HOST buffers (Sec. 2.1: attention, greedy choice, walk, commit in
 * that order).  The per-step inputs are copied from (preferably pinned) host memory to the
 * caller's device staging buffer, the four calls above run, and the results are copied back; all
 * on the given stream, without a synchronisation (results are valid once the stream has drained).
 * The KV cache and ctx_len stay on the device; ctx_len is advanced in place.
 */
typedef struct {          /* host memory; every pointer is a HOST pointer */
  const void* q;          /* bf16 [B, N, Hq, 128]   */
  const void* k_tree;     /* bf16 [B, N, Hkv, 128]  */
  const void* v_tree;     /* bf16 [B, N, Hkv, 128]  */
  const int32_t* parent;  /* [B, N]                 */
  const int32_t* tokens;  /* [B, N]                 */
  const void* logits;     /* bf16 [B*N, ld]         */
  int64_t ld;
} clv_host_inputs;

typedef struct {          /* host memory; every pointer is a HOST pointer, written asynchronously */
  void* out;              /* bf16 [B, N, Hq, 128]   */
  int32_t* argmax_ids;    /* [B, N]                 */
  int32_t* accept_len;    /* [B]                    */
  int32_t* accept_idx;    /* [B, path_cap]          */
  int32_t* next_token;    /* [B]                    */
  int32_t* status;        /* [3, B]: attention, walk, commit */
} clv_host_outputs;

size_t clv_staging_bytes(const clv_shape* shape, int64_t ld);
clv_status clv_verify_step_host(const clv_shape* shape, const clv_kv_cache* cache,
                                const clv_host_inputs* in, const clv_host_outputs* out,
                                int32_t* ctx_len /* device [B], updated in place */,
                                int32_t max_ctx_len, float softmax_scale,
                                void* staging, size_t staging_bytes, /* device */
                                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * For tests only (the paper has no counterpart): the number of SM clock cycles after which a
 * bounded on-chip wait of clv_tree_attn / clv_lm_head_argmax gives up and the call reports
 * CLV_ERR_TIMEOUT in its device status.  The default is about a second; a test passes a few dozen
 * cycles to make a wait for the first tile run out, which exercises the abort path without any
 * fault (copies and tensor-core work in flight are still waited for with the long bound).
 * sm_cycles <= 0 restores the default.  Process-wide; applies to launches made afterwards.
 */
void clv_test_set_wait_limit(int64_t sm_cycles);

const char* clv_status_string(clv_status s);
int clv_last_cuda_error(void); /* cudaError_t of the most recent CLV_ERR_CUDA on this thread */
int clv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CLV_H_ */
