/*
 * CPU checker for the tree-verification step of Clover-2-style speculative decoding.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the verification
 * step computes, written from the paper's prose; the GPU library is compared against it.  It
 * shares no code with the GPU library and must never be called from the product path.
 *
 * All floating point is IEEE double.  bf16 inputs arrive as uint16 bit patterns and are widened
 * exactly.  There is no blocking, tiling or reordering: every function is the definition itself
 * written as nested loops (OpenMP only distributes independent outer iterations).
 *
 * What each function follows:
 *   orc_tree_attn     - Sec. 2.1 "Speculative Decoding and Tree Attention" and the caption of
 *                       Fig. 2: ordinary softmax attention whose causal mask is the token
 *                       tree's topology matrix (a node sees the committed context and its own
 *                       ancestors, itself included).
 *   orc_argmax        - Sec. 4.2 (Table 1 note): temperature 0 is greedy decoding of the target.
 *   orc_lm_head_argmax - Sec. 3.1 (final norm + LM head give the logits) followed by Sec. 4.2's
 *                       greedy choice, the logit held in bf16 like a logits tensor.
 *   build_token_tree (in the Python wrapper, plain loops over a dictionary) - Sec. 2.1 and the
 *                       caption of Fig. 2: speculations merged by prefix matching into a tree.
 *   tree_to_intervals / tree_from_intervals (in the Python wrapper, a recursive walk and plain
 *                       loops) - App. A.1: the compressed, linear form of the tree mask, taken
 *                       as depth-first entry/exit labels.
 *   draft_head_step (in the Python wrapper, float64 numpy) - Sec. 3.1 and App. A.3: the Attention
 *                       Decoder (RMSNorm, q/k/v projections, per-head cosine gate, residual), the
 *                       fully connected output projector over its output and the token
 *                       embedding, then norm + LM head and the head's top-k proposals.
 *   orc_accept_walk   - Sec. 2.1 verification phase (the target filters out wrong drafted
 *                       tokens; the output equals plain decoding) with the greedy rule of the
 *                       tree-sampling algorithm Sec. 4.1 adopts.
 *   orc_accept_sample - Sec. 4.1 / 4.2 (Table 1, temperature 1): the paper adopts the tree sampling
 *                       algorithm of its baseline system and prints no formula; this is the
 *                       speculative-sampling rule for drafts that are proposed deterministically
 *                       (each child of a node is one proposed token): a child is accepted with its
 *                       probability under what is left of the target's distribution, a rejected
 *                       token is struck from it, and when every child is rejected the next token
 *                       is drawn from the remainder.  The emitted tokens then follow the target's
 *                       distribution exactly.
 *   orc_kv_commit     - derived from the equivalence requirement of Sec. 2.1: after a step the
 *                       cache holds exactly what plain decoding of the accepted tokens would.
 *
 * Pins (tests/test_oracle_*.py): path linearisation, chain == causal prefill, star == independent
 * decodes, a float64 library attention with an explicit boolean mask, convex-hull and
 * log-sum-exp identities, mask exactness under perturbation, brute-force path enumeration,
 * numpy's first-occurrence argmax, the commit/append equivalence, and for the LM head a float64
 * library matrix product, a one-hot weight matrix and planted rounding ties; for the stochastic
 * acceptance the exact outcome probabilities of small trees (computed by a separate recursive
 * enumeration) against frequencies over many draws, the emitted token's distribution against the
 * target's softmax, the low-temperature limit against the greedy walk, and certain / impossible
 * drafts.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_TREE 7   /* same numeric meaning as the status values the library documents */

static double bf16_to_f64(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* Round a double to the nearest bf16 (ties to even), one rounding step, result as bits. */
static uint16_t f64_to_bf16(double d) {
  if (d != d) return 0x7FC0;
  uint16_t sign = signbit(d) ? 0x8000 : 0;
  double a = fabs(d);
  if (a == 0.0) return sign;
  if (isinf(a)) return sign | 0x7F80;
  int e;
  (void)frexp(a, &e); /* a = m * 2^e, m in [0.5,1)  ->  floor(log2 a) = e-1 */
  int p = e - 1;
  if (p < -126) p = -126;                /* subnormal range keeps a fixed quantum */
  double quantum = ldexp(1.0, p - 7);    /* spacing of bf16 values in this binade */
  double r = nearbyint(a / quantum) * quantum; /* default rounding mode: ties to even */
  if (r >= ldexp(1.0, 128)) return sign | 0x7F80;
  float f = (float)r; /* exact: r has at most 8 significant bits */
  uint32_t u;
  memcpy(&u, &f, 4);
  return sign | (uint16_t)(u >> 16);
}

/* Address of cache row `t` (token position) of sequence b, kv head g. */
typedef struct {
  const uint16_t *k, *v;
  int paged, cap_tokens, page_size, max_pages, n_kv_heads, head_dim;
  const int32_t *block_table;
} orc_cache;

static int64_t cache_row_offset(const orc_cache *c, int b, int64_t t, int g) {
  int64_t row;
  if (c->paged) {
    int64_t page = c->block_table[(int64_t)b * c->max_pages + t / c->page_size];
    row = page * c->page_size + t % c->page_size;
  } else {
    row = (int64_t)b * c->cap_tokens + t;
  }
  return (row * c->n_kv_heads + g) * c->head_dim;
}

static int tree_ok(const int32_t *parent, int n, int allow_forest) {
  for (int i = 0; i < n; ++i) {
    int p = parent[i];
    if (i == 0) {
      if (p != -1) return 0;
    } else if (p == -1) {
      if (!allow_forest) return 0;
    } else if (p < 0 || p >= i) {
      return 0;
    }
  }
  return 1;
}

/*
 * Tree attention.  rows == NULL: every (b, i, h) in that order, n_rows = B*N*Hq.
 * Otherwise rows holds n_rows triples (b, i, h).  Row r of the outputs belongs to rows[r].
 * out_f64 [n_rows, D] double; out_bf16 [n_rows, D] bits (may be NULL); lse [n_rows] natural log
 * (may be NULL).  status [B]: ORC_ERR_TREE if parent[] of that sequence is malformed (its rows
 * are then filled with zeros).  Forests (several -1 parents) are allowed here.
 */
int orc_tree_attn(int B, int N, int Hq, int Hkv, int D, const uint16_t *q, const uint16_t *kc,
                  const uint16_t *vc, int paged, int cap_tokens, int page_size, int max_pages,
                  const int32_t *block_table, const uint16_t *k_tree, const uint16_t *v_tree,
                  const int32_t *parent, const int32_t *ctx_len, double scale, int64_t n_rows,
                  const int32_t *rows, double *out_f64, uint16_t *out_bf16, double *lse,
                  int32_t *status) {
  orc_cache c = {kc, vc, paged, cap_tokens, page_size, max_pages, Hkv, D, block_table};
  int G = Hq / Hkv;
  for (int b = 0; b < B; ++b)
    status[b] = tree_ok(parent + (int64_t)b * N, N, 1) ? ORC_OK : ORC_ERR_TREE;

#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t r = 0; r < n_rows; ++r) {
    int b, i, h;
    if (rows) {
      b = rows[3 * r]; i = rows[3 * r + 1]; h = rows[3 * r + 2];
    } else {
      b = (int)(r / ((int64_t)N * Hq)); i = (int)((r / Hq) % N); h = (int)(r % Hq);
    }
    double *o = out_f64 + r * D;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (status[b] != ORC_OK) {
      if (out_bf16) for (int d = 0; d < D; ++d) out_bf16[r * D + d] = 0;
      if (lse) lse[r] = 0.0;
      continue;
    }
    int g = h / G;
    int64_t L = ctx_len[b];
    const int32_t *par = parent + (int64_t)b * N;
    /* row i of the topology matrix: allowed[j] = 1 iff j is i or an ancestor of i */
    char *allowed = (char *)calloc((size_t)N, 1);
    for (int j = i; j >= 0; j = par[j]) allowed[j] = 1;
    int64_t n_keys = L + N;
    double *s = (double *)malloc(sizeof(double) * (size_t)n_keys);
    const uint16_t *qrow = q + (((int64_t)b * N + i) * Hq + h) * D;
    double m = -INFINITY;
    for (int64_t t = 0; t < n_keys; ++t) {
      const uint16_t *krow;
      if (t < L) {
        krow = c.k + cache_row_offset(&c, b, t, g);
      } else {
        int j = (int)(t - L);
        if (!allowed[j]) { s[t] = -INFINITY; continue; }
        krow = k_tree + (((int64_t)b * N + j) * Hkv + g) * D;
      }
      double acc = 0.0;
      for (int d = 0; d < D; ++d) acc += bf16_to_f64(qrow[d]) * bf16_to_f64(krow[d]);
      s[t] = scale * acc;
      if (s[t] > m) m = s[t];
    }
    double denom = 0.0;
    for (int64_t t = 0; t < n_keys; ++t) {
      if (s[t] == -INFINITY) continue;
      double w = exp(s[t] - m);
      denom += w;
      const uint16_t *vrow = (t < L) ? c.v + cache_row_offset(&c, b, t, g)
                                     : v_tree + (((int64_t)b * N + (t - L)) * Hkv + g) * D;
      for (int d = 0; d < D; ++d) o[d] += w * bf16_to_f64(vrow[d]);
    }
    for (int d = 0; d < D; ++d) o[d] /= denom;
    if (out_bf16) for (int d = 0; d < D; ++d) out_bf16[r * D + d] = f64_to_bf16(o[d]);
    if (lse) lse[r] = m + log(denom);
    free(s);
    free(allowed);
  }
  return 0;
}

/* ids[r] = index of the first strict maximum of row r (rows of `vocab` bf16 values, stride ld). */
int orc_argmax(int64_t n_rows, int vocab, int64_t ld, const uint16_t *logits, int32_t *ids) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < n_rows; ++r) {
    const uint16_t *row = logits + r * ld;
    double best = bf16_to_f64(row[0]);
    int32_t arg = 0;
    for (int v = 1; v < vocab; ++v) {
      double x = bf16_to_f64(row[v]);
      if (x > best) { best = x; arg = v; }
    }
    ids[r] = arg;
  }
  return 0;
}

/*
 * LM head followed by the greedy choice (Sec. 3.1: the logits of a node are the LM head applied
 * to its normalised hidden state; Sec. 4.2: temperature 0).  For each selected row r:
 *   logit[v] = sum_k hidden[r][k] * weight[v][k]   in double, then rounded to bf16 (the precision
 *   the logits tensor has), ids = the first strict maximum of the rounded values.
 * logits64 (optional, [n_sel][vocab]) receives the unrounded doubles so that a test can see how
 * close the runners-up are.  rows == NULL selects rows 0 .. n_sel-1.
 */
int orc_lm_head_argmax(int n_sel, const int32_t *rows, int hidden_dim, int vocab, int64_t ld_hidden,
                       int64_t ld_weight, const uint16_t *hidden, const uint16_t *weight,
                       double *logits64, int32_t *ids) {
  for (int i = 0; i < n_sel; ++i) {
    const uint16_t *h = hidden + (int64_t)(rows ? rows[i] : i) * ld_hidden;
    double *z = (double *)malloc(sizeof(double) * (size_t)vocab);
    if (!z) return -1;
#pragma omp parallel for schedule(static)
    for (int v = 0; v < vocab; ++v) {
      const uint16_t *w = weight + (int64_t)v * ld_weight;
      double acc = 0.0;
      for (int k = 0; k < hidden_dim; ++k) acc += bf16_to_f64(h[k]) * bf16_to_f64(w[k]);
      z[v] = acc;
    }
    double best = bf16_to_f64(f64_to_bf16(z[0]));
    int32_t arg = 0;
    for (int v = 1; v < vocab; ++v) {
      double x = bf16_to_f64(f64_to_bf16(z[v]));
      if (x > best) { best = x; arg = v; }
    }
    ids[i] = arg;
    if (logits64) memcpy(logits64 + (size_t)i * vocab, z, sizeof(double) * (size_t)vocab);
    free(z);
  }
  return 0;
}

/*
 * Greedy acceptance walk.  Node 0 is the root (the token the target emitted last; always
 * accepted).  From the current node, the target's choice is ids[cur]; the drafted child carrying
 * exactly that token (lowest index if the precondition of distinct siblings is broken) is
 * accepted and becomes current; otherwise the walk ends.  next_token = ids[last accepted].
 * Malformed parent[] (node 0 not the only root, parent[i] >= i or < -1) or a path longer than
 * path_cap: status = ORC_ERR_TREE, accept_len = 0, next_token = -1, accept_idx all -1.
 */
int orc_accept_walk(int B, int N, int path_cap, const int32_t *parent, const int32_t *tokens,
                    const int32_t *ids, int32_t *accept_len, int32_t *accept_idx,
                    int32_t *next_token, int32_t *status) {
  for (int b = 0; b < B; ++b) {
    const int32_t *par = parent + (int64_t)b * N, *tok = tokens + (int64_t)b * N;
    const int32_t *id = ids + (int64_t)b * N;
    int32_t *path = accept_idx + (int64_t)b * path_cap;
    for (int j = 0; j < path_cap; ++j) path[j] = -1;
    status[b] = ORC_OK;
    int ok = tree_ok(par, N, 0) && path_cap >= 1;
    int len = 0, cur = 0;
    if (ok) {
      path[len++] = 0;
      for (;;) {
        int t = id[cur], found = -1;
        for (int cnode = cur + 1; cnode < N; ++cnode)
          if (par[cnode] == cur && tok[cnode] == t) { found = cnode; break; }
        if (found < 0) break;
        if (len == path_cap) { ok = 0; break; }
        path[len++] = found;
        cur = found;
      }
    }
    if (!ok) {
      for (int j = 0; j < path_cap; ++j) path[j] = -1;
      status[b] = ORC_ERR_TREE;
      accept_len[b] = 0;
      next_token[b] = -1;
    } else {
      accept_len[b] = len;
      next_token[b] = id[cur];
    }
  }
  return 0;
}

/*
 * Commit: cache rows ctx_len[b] + j  <-  tree rows accept_idx[b][j], j < accept_len[b], K and V,
 * every kv head.  ctx_len_out[b] = ctx_len[b] + accept_len[b].  The cache buffers are modified in
 * place (the caller passes copies).  A sequence whose accepted rows would not fit its capacity
 * (contiguous: cap_tokens; paged: its block-table entries must exist and be valid), or whose
 * accept_len / accept_idx are out of range, is left untouched: status = ORC_ERR_TREE and
 * ctx_len_out[b] = ctx_len[b].
 */
int orc_kv_commit(int B, int N, int Hkv, int D, int path_cap, uint16_t *kc, uint16_t *vc, int paged,
                  int cap_tokens, int page_size, int n_pages, int max_pages,
                  const int32_t *block_table, const uint16_t *k_tree, const uint16_t *v_tree,
                  const int32_t *accept_idx, const int32_t *accept_len, const int32_t *ctx_len,
                  int32_t *ctx_len_out, int32_t *status) {
  orc_cache c = {kc, vc, paged, cap_tokens, page_size, max_pages, Hkv, D, block_table};
  for (int b = 0; b < B; ++b) {
    int64_t L = ctx_len[b];
    int len = accept_len[b];
    int ok = (L >= 0) && (len >= 0) && (len <= path_cap);
    for (int j = 0; ok && j < len; ++j) {
      int a = accept_idx[(int64_t)b * path_cap + j];
      if (a < 0 || a >= N) ok = 0;
      int64_t t = L + j;
      if (paged) {
        if (t / page_size >= max_pages) ok = 0;
        else {
          int pg = block_table[(int64_t)b * max_pages + t / page_size];
          if (pg < 0 || pg >= n_pages) ok = 0;
        }
      } else if (t >= cap_tokens) ok = 0;
    }
    if (!ok) { status[b] = ORC_ERR_TREE; ctx_len_out[b] = (int32_t)L; continue; }
    status[b] = ORC_OK;
    for (int j = 0; j < len; ++j) {
      int a = accept_idx[(int64_t)b * path_cap + j];
      for (int g = 0; g < Hkv; ++g) {
        int64_t dst = cache_row_offset(&c, b, L + j, g);
        int64_t src = (((int64_t)b * N + a) * Hkv + g) * D;
        memcpy(kc + dst, k_tree + src, sizeof(uint16_t) * (size_t)D);
        memcpy(vc + dst, v_tree + src, sizeof(uint16_t) * (size_t)D);
      }
    }
    ctx_len_out[b] = (int32_t)(L + len);
  }
  return 0;
}

/* Exposed so a test can pin the rounding helper against an independent bf16 conversion. */
/*
 * Stochastic acceptance at temperature T > 0.  Node 0 is the root (always accepted).  At the current
 * node the target's distribution is p = softmax(logits[cur] / T) over the vocabulary.  Its
 * children are looked at in increasing node index; child c carries token x = tokens[c] and is
 * accepted if  u[c] < p(x) / (1 - mass of the tokens rejected at this node so far);  an accepted
 * child becomes the current node (with a fresh distribution).  A rejected token is struck from the
 * distribution.  When no child is accepted (or there is none), the next token is drawn from what
 * is left: the first v, in vocabulary order and not struck, whose running sum of p exceeds
 * u[N] * (1 - rejected mass).  u: [B, N + 1] uniforms in [0, 1) supplied by the caller (u[b][c]
 * decides child c, u[b][N] draws the next token).  A struck token cannot be proposed again at the
 * same node (siblings carry distinct tokens; if they do not, the repeat is rejected).
 * margin[b][0] receives the smallest |u - threshold| over the accept tests of the sequence (in
 * probability units), margin[b][1] the distance of the final draw's target to the nearer of the
 * two running sums that bracket it, divided by the remaining mass, so that a caller can tell
 * results that rounding cannot change from those it can.  Malformed trees are reported like
 * orc_accept_walk does.
 */
int orc_accept_sample(int B, int N, int vocab, int64_t ld, int path_cap, const uint16_t *logits,
                      const int32_t *parent, const int32_t *tokens, const float *u, double temperature,
                      int32_t *accept_len, int32_t *accept_idx, int32_t *next_token, int32_t *status,
                      double *margin) {
  double *p = (double *)malloc(sizeof(double) * (size_t)vocab);
  if (!p) return 1;
  for (int b = 0; b < B; ++b) {
    const int32_t *par = parent + (int64_t)b * N, *tok = tokens + (int64_t)b * N;
    const float *ub = u + (int64_t)b * (N + 1);
    int32_t *path = accept_idx + (int64_t)b * path_cap;
    for (int j = 0; j < path_cap; ++j) path[j] = -1;
    status[b] = ORC_OK;
    margin[2 * b] = 1.0;
    margin[2 * b + 1] = 1.0;
    int ok = tree_ok(par, N, 0) && path_cap >= 1 && temperature > 0.0;
    int len = 0, cur = 0, nxt = -1;
    if (ok) {
      path[len++] = 0;
      for (;;) {
        /* the target's distribution at the current node */
        const uint16_t *row = logits + ((int64_t)b * N + cur) * ld;
        double m = -INFINITY, z = 0.0;
        for (int v = 0; v < vocab; ++v) { double l = bf16_to_f64(row[v]) / temperature; if (l > m) m = l; }
        for (int v = 0; v < vocab; ++v) { p[v] = exp(bf16_to_f64(row[v]) / temperature - m); z += p[v]; }
        for (int v = 0; v < vocab; ++v) p[v] /= z;
        double rejected = 0.0;
        int found = -1;
        for (int c = cur + 1; c < N && found < 0; ++c) {
          if (par[c] != cur) continue;
          const int x = tok[c];
          double a = 0.0;
          if (x >= 0 && x < vocab && rejected < 1.0) a = p[x] / (1.0 - rejected);
          const double d = fabs((double)ub[c] - a);
          if (d < margin[2 * b]) margin[2 * b] = d;
          if ((double)ub[c] < a) {
            found = c;
          } else if (x >= 0 && x < vocab) {
            rejected += p[x];
            p[x] = 0.0;
          }
        }
        if (found >= 0) {
          if (len == path_cap) { ok = 0; break; }
          path[len++] = found;
          cur = found;
          continue;
        }
        /* every child rejected (or no child): draw from what is left */
        double left = 0.0;
        for (int v = 0; v < vocab; ++v) left += p[v];
        const double target = (double)ub[N] * left;
        double run = 0.0;
        nxt = -1;
        int last = -1;
        for (int v = 0; v < vocab; ++v) {
          if (p[v] <= 0.0) continue;
          last = v;
          const double before = run;
          run += p[v];
          if (run > target) {
            nxt = v;
            double d = (target - before < run - target ? target - before : run - target) / left;
            if (before == 0.0) d = (run - target) / left;   /* nothing below the first candidate */
            if (d < margin[2 * b + 1]) margin[2 * b + 1] = d;
            break;
          }
        }
        if (nxt < 0) nxt = last;   /* rounding left the running sum a hair short of the target */
        break;
      }
    }
    if (!ok) {
      for (int j = 0; j < path_cap; ++j) path[j] = -1;
      len = 0;
      nxt = -1;
      status[b] = ORC_ERR_TREE;
    }
    accept_len[b] = len;
    next_token[b] = nxt;
  }
  free(p);
  return 0;
}

uint16_t orc_f64_to_bf16(double d) { return f64_to_bf16(d); }
