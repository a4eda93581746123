/*
 * CPU oracle for the tree-verification step of EAGLE speculative decoding.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the CUDA library is
 * checked against.  It shares no code with the CUDA path, and nothing in the product path may
 * call it.  Everything is fp64 and written as the definition / the algorithm's steps, with no
 * blocking, fusion or reordering.  OpenMP only distributes independent (sequence, head) units.
 *
 * What each function follows:
 *   oracle_tree_ancestors    - "tree attention" (Sec. 3.1, Sec. 3.3, App. A.1): a draft token sees the
 *                              tokens on its own root path.  The set is found by walking parent links.
 *   oracle_tree_verify_attn  - Sec. 3.3 / App. A.1: one target forward pass scores every tree token;
 *                              for one attention layer that is softmax attention over the committed
 *                              prefix plus the node's ancestors and itself (plain definition).
 *   oracle_tree_verify_attn_paged - the same over a cache stored in pages addressed through a block table.
 *   oracle_tree_verify_attn_fp8 - the same over a cache stored as fp8 (e4m3) codes with one scale per (sequence, KV head).
 *   oracle_tree_verify_attn_fp8_paged - the fp8 cache kept in pages behind a block table.
 *   oracle_tree_accept       - Algorithm 1 (multi-round speculative sampling, App. A.2) applied
 *                              recursively at every node from the root (Sec. 3.3); the greedy setting
 *                              (Preliminaries) is the same rule with a one-hot target distribution.
 *   oracle_tree_accept_logits - the same with the distributions given as logits (softmax at a temperature, fp64).
 *   oracle_tree_expand       - App. A.1 (tree structure): the children of a draft-tree node are the k most probable
 *                              tokens of its draft distribution in the greedy setting, k sampled tokens otherwise.
 *   oracle_tree_commit       - Sec. 3.3, last sentence: the accepted tokens and their features are recorded
 *                              for the next drafting phase.  For the target's KV cache that means: the
 *                              keys and values of the accepted tree nodes become the next slots of the
 *                              committed prefix, in path order; the accepted nodes' feature vectors are
 *                              gathered in the same order (plain definition: a simultaneous assignment).
 *   oracle_tree_commit_paged - the same on a cache stored in pages.
 *
 * Readings taken where the paper is silent or garbled are listed next to the code that uses them.
 * Pins: see tests/test_oracle_*.py.  The sibling order, the lowest-index tie-break of argmax and the
 * assignment of uniforms to decisions are conventions of this library, not fixed by the paper:
 * "parity unpinned" for those three conventions (they are pinned only by this file's own statement).
 */
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_TREE (-2)
#define ORACLE_ERR_NOMEM (-3)

/* kinds of decision in the acceptance walk's trace */
#define ORACLE_DEC_ACCEPT 0
#define ORACLE_DEC_REJECT 1
#define ORACLE_DEC_BONUS 2
#define ORACLE_DEC_ARGMAX 3

static double bf16_to_f64(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

static int tree_size_of(const int32_t* tree_sizes, int b, int max_tree) {
  return tree_sizes ? tree_sizes[b] : max_tree;
}

/* A parent array is valid when -1 <= parent[i] < i (topological order; -1 = child of the context). */
static int tree_valid(const int32_t* parent, int n) {
  for (int i = 0; i < n; ++i)
    if (parent[i] < -1 || parent[i] >= i) return 0;
  return 1;
}

/*
 * Ancestor-or-self set of every node, as a bit set, and the node's depth (top-level nodes have
 * depth 1).  Found by following parent links up to the context; no recurrence over earlier results.
 * parent: int32 [batch, max_tree]; tree_sizes: int32 [batch] or NULL; anc: uint64 [batch, max_tree];
 * depth: int32 [batch, max_tree].  Entries of nodes >= tree size are set to 0.
 */
int oracle_tree_ancestors(const int32_t* parent, const int32_t* tree_sizes, int batch, int max_tree,
                          uint64_t* anc, int32_t* depth) {
  if (!parent || !anc || batch < 0 || max_tree < 0 || max_tree > 64) return ORACLE_ERR_ARG;
  for (int b = 0; b < batch; ++b) {
    const int n = tree_size_of(tree_sizes, b, max_tree);
    if (n < 0 || n > max_tree) return ORACLE_ERR_ARG;
    const int32_t* par = parent + (size_t)b * max_tree;
    if (!tree_valid(par, n)) return ORACLE_ERR_TREE;
    for (int i = 0; i < max_tree; ++i) {
      uint64_t set = 0;
      int d = 0;
      if (i < n) {
        for (int c = i; c >= 0; c = par[c]) {
          set |= (uint64_t)1 << c;
          ++d;
        }
      }
      anc[(size_t)b * max_tree + i] = set;
      if (depth) depth[(size_t)b * max_tree + i] = d;
    }
  }
  return ORACLE_OK;
}

/*
 * Tree-masked attention of one layer, by definition.
 *
 *   q        bf16 bits [batch, max_tree, num_q_heads, head_dim]
 *   k_cache  bf16 bits [batch, num_kv_heads, kv_capacity, head_dim]   (v_cache alike)
 *   seq_lens int32 [batch]   committed prefix length L_b; tree node m's key/value sit at slot L_b + m
 *   out      fp64  [batch, max_tree, num_q_heads, head_dim]; rows of nodes >= tree size are 0
 *
 * Node i of sequence b, query head h (KV head h / G, G = num_q_heads / num_kv_heads) sees slot j iff
 * j < L_b, or j = L_b + m with m on the path from i up to the context (i itself included).
 * s_j = sm_scale * <q, k_j>;  out = sum_j softmax(s)_j v_j.   Slots that are not visible are never
 * read, so they may hold anything (NaN included).
 */
int oracle_tree_verify_attn(int batch, int num_q_heads, int num_kv_heads, int head_dim, int max_tree,
                            int kv_capacity, const int32_t* tree_sizes, double sm_scale,
                            const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                            const int32_t* seq_lens, const int32_t* tree_parent, double* out) {
  if (batch < 0 || num_q_heads <= 0 || num_kv_heads <= 0 || head_dim <= 0 || max_tree < 0 ||
      max_tree > 64 || num_q_heads % num_kv_heads != 0 || !seq_lens || !tree_parent || !out)
    return ORACLE_ERR_ARG;
  const int G = num_q_heads / num_kv_heads;
  const int D = head_dim;
  if (sm_scale == 0.0) sm_scale = 1.0 / sqrt((double)D);
  for (int b = 0; b < batch; ++b) {
    const int n = tree_size_of(tree_sizes, b, max_tree);
    if (n < 0 || n > max_tree || seq_lens[b] < 0 || seq_lens[b] + n > kv_capacity) return ORACLE_ERR_ARG;
    if (!tree_valid(tree_parent + (size_t)b * max_tree, n)) return ORACLE_ERR_TREE;
  }
  memset(out, 0, sizeof(double) * (size_t)batch * max_tree * num_q_heads * D);
  int failed = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < batch; ++b) {
    for (int h = 0; h < num_q_heads; ++h) {
      const int n = tree_size_of(tree_sizes, b, max_tree);
      const int L = seq_lens[b];
      const int g = h / G;
      const int32_t* par = tree_parent + (size_t)b * max_tree;
      const uint16_t* kb = k_cache + ((size_t)b * num_kv_heads + g) * (size_t)kv_capacity * D;
      const uint16_t* vb = v_cache + ((size_t)b * num_kv_heads + g) * (size_t)kv_capacity * D;
      int* slots = (int*)malloc(sizeof(int) * (size_t)(L + max_tree + 1));
      double* s = (double*)malloc(sizeof(double) * (size_t)(L + max_tree + 1));
      if (!slots || !s) {
        failed = 1;
        free(slots);
        free(s);
        continue;
      }
      for (int i = 0; i < n; ++i) {
        const uint16_t* qi = q + (((size_t)b * max_tree + i) * num_q_heads + h) * D;
        double* oi = out + (((size_t)b * max_tree + i) * num_q_heads + h) * D;
        /* visible slots: the whole prefix, then the root path of node i */
        int cnt = 0;
        for (int j = 0; j < L; ++j) slots[cnt++] = j;
        for (int c = i; c >= 0; c = par[c]) slots[cnt++] = L + c;
        double smax = -INFINITY;
        for (int t = 0; t < cnt; ++t) {
          const uint16_t* kj = kb + (size_t)slots[t] * D;
          double acc = 0.0;
          for (int d = 0; d < D; ++d) acc += bf16_to_f64(qi[d]) * bf16_to_f64(kj[d]);
          s[t] = sm_scale * acc;
          if (s[t] > smax) smax = s[t];
        }
        double denom = 0.0;
        for (int t = 0; t < cnt; ++t) {
          s[t] = exp(s[t] - smax);
          denom += s[t];
        }
        for (int d = 0; d < D; ++d) {
          double acc = 0.0;
          for (int t = 0; t < cnt; ++t) acc += s[t] * bf16_to_f64(vb[(size_t)slots[t] * D + d]);
          oi[d] = acc / denom;
        }
      }
      free(slots);
      free(s);
    }
  }
  return failed ? ORACLE_ERR_NOMEM : ORACLE_OK;
}

/*
 * The same attention when the cache is kept in pages (a cache layout, not a change of the method: Sec. 3.3's
 * verification pass reads the same keys and values wherever they are stored).
 *
 *   k_pages     bf16 bits [num_pages, num_kv_heads, page_size, head_dim]   (v_pages alike)
 *   block_table int32 [batch, max_pages_per_seq]: logical slot j of sequence b is row j % page_size of page
 *               block_table[b, j / page_size]
 *
 * By definition: the slots a sequence can see (j < L_b + tree size) are copied out of their pages into a contiguous
 * cache of capacity max_pages_per_seq * page_size, and the contiguous definition above is applied.  Table entries
 * of pages that hold no visible slot are never read.  A visible slot whose page is outside [0, num_pages) is an
 * argument error.
 */
int oracle_tree_verify_attn_paged(int batch, int num_q_heads, int num_kv_heads, int head_dim, int max_tree,
                                  int num_pages, int page_size, int max_pages_per_seq, const int32_t* tree_sizes,
                                  double sm_scale, const uint16_t* q, const uint16_t* k_pages, const uint16_t* v_pages,
                                  const int32_t* block_table, const int32_t* seq_lens, const int32_t* tree_parent,
                                  double* out) {
  if (batch < 0 || num_kv_heads <= 0 || head_dim <= 0 || num_pages < 0 || page_size <= 0 || max_pages_per_seq < 0 ||
      !block_table || !seq_lens)
    return ORACLE_ERR_ARG;
  const size_t cap = (size_t)max_pages_per_seq * page_size, D = (size_t)head_dim;
  if (cap > 0x7fffffffu) return ORACLE_ERR_ARG;
  const size_t elems = (size_t)batch * num_kv_heads * cap * D;
  uint16_t* kc = (uint16_t*)calloc(elems ? elems : 1, sizeof(uint16_t));
  uint16_t* vc = (uint16_t*)calloc(elems ? elems : 1, sizeof(uint16_t));
  int rc = (kc && vc) ? ORACLE_OK : ORACLE_ERR_NOMEM;
  for (int b = 0; b < batch && rc == ORACLE_OK; ++b) {
    const int n = tree_size_of(tree_sizes, b, max_tree);
    if (n < 0 || n > max_tree || seq_lens[b] < 0 || (size_t)seq_lens[b] + n > cap) {
      rc = ORACLE_ERR_ARG;
      break;
    }
    const int visible = n > 0 ? seq_lens[b] + n : 0;
    for (int j = 0; j < visible && rc == ORACLE_OK; ++j) {
      const int page = block_table[(size_t)b * max_pages_per_seq + j / page_size], row = j % page_size;
      if (page < 0 || page >= num_pages) {
        rc = ORACLE_ERR_ARG;
        break;
      }
      for (int g = 0; g < num_kv_heads; ++g) {
        const size_t src = (((size_t)page * num_kv_heads + g) * page_size + row) * D;
        const size_t dst = (((size_t)b * num_kv_heads + g) * cap + j) * D;
        memcpy(kc + dst, k_pages + src, D * sizeof(uint16_t));
        memcpy(vc + dst, v_pages + src, D * sizeof(uint16_t));
      }
    }
  }
  if (rc == ORACLE_OK)
    rc = oracle_tree_verify_attn(batch, num_q_heads, num_kv_heads, head_dim, max_tree, (int)cap, tree_sizes, sm_scale, q, kc,
                                 vc, seq_lens, tree_parent, out);
  free(kc);
  free(vc);
  return rc;
}

/*
 * Value of an fp8 "e4m3" code (the 8-bit float with 1 sign, 4 exponent and 3 mantissa bits, exponent bias 7, no
 * infinities; the two codes with all exponent and mantissa bits set are NaN), written from that definition:
 * exponent field 0 -> (mantissa / 8) * 2^-6 (zero and the subnormals), else (1 + mantissa / 8) * 2^(exponent - 7).
 */
static double e4m3_to_f64(uint8_t c) {
  const int sign = c >> 7, e = (c >> 3) & 15, m = c & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0) v = ldexp((double)m / 8.0, -6);
  else v = ldexp(1.0 + (double)m / 8.0, e - 7);
  return sign ? -v : v;
}

/* The 256 values of the code above (for the test that pins the table against a library's conversion). */
void oracle_e4m3_table(double* out256) {
  for (int c = 0; c < 256; ++c) out256[c] = e4m3_to_f64((uint8_t)c);
}

/*
 * The same attention when the cache is STORED in fp8 (a storage format of the same cache: Sec. 4.4 notes that the
 * decoding being sped up is bound by memory traffic, and Sec. 4.2 reports the method on a quantised deployment; the
 * paper gives no quantisation scheme, so the convention is this library's): k_cache / v_cache hold e4m3 codes
 * [batch, num_kv_heads, kv_capacity, head_dim] and every (sequence, KV head) has one fp32 scale for its keys and one
 * for its values, k_scale / v_scale [batch, num_kv_heads]: key = code value * k_scale, value = code value * v_scale,
 * exactly (fp64).  Everything after that is the definition of oracle_tree_verify_attn, written out again on those
 * values: queries stay bf16, scores / softmax / sums are fp64.  Slots that are not visible are never read.
 */
int oracle_tree_verify_attn_fp8(int batch, int num_q_heads, int num_kv_heads, int head_dim, int max_tree,
                                int kv_capacity, const int32_t* tree_sizes, double sm_scale, const uint16_t* q,
                                const uint8_t* k_cache, const uint8_t* v_cache, const float* k_scale, const float* v_scale,
                                const int32_t* seq_lens, const int32_t* tree_parent, double* out) {
  if (batch < 0 || num_q_heads <= 0 || num_kv_heads <= 0 || head_dim <= 0 || max_tree < 0 || max_tree > 64 ||
      num_q_heads % num_kv_heads != 0 || !seq_lens || !tree_parent || !out || !k_scale || !v_scale)
    return ORACLE_ERR_ARG;
  const int G = num_q_heads / num_kv_heads;
  const int D = head_dim;
  if (sm_scale == 0.0) sm_scale = 1.0 / sqrt((double)D);
  for (int b = 0; b < batch; ++b) {
    const int n = tree_size_of(tree_sizes, b, max_tree);
    if (n < 0 || n > max_tree || seq_lens[b] < 0 || seq_lens[b] + n > kv_capacity) return ORACLE_ERR_ARG;
    if (!tree_valid(tree_parent + (size_t)b * max_tree, n)) return ORACLE_ERR_TREE;
  }
  memset(out, 0, sizeof(double) * (size_t)batch * max_tree * num_q_heads * D);
  int failed = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < batch; ++b) {
    for (int h = 0; h < num_q_heads; ++h) {
      const int n = tree_size_of(tree_sizes, b, max_tree);
      const int L = seq_lens[b];
      const int g = h / G;
      const int32_t* par = tree_parent + (size_t)b * max_tree;
      const uint8_t* kb = k_cache + ((size_t)b * num_kv_heads + g) * (size_t)kv_capacity * D;
      const uint8_t* vb = v_cache + ((size_t)b * num_kv_heads + g) * (size_t)kv_capacity * D;
      const double ks = (double)k_scale[(size_t)b * num_kv_heads + g], vs = (double)v_scale[(size_t)b * num_kv_heads + g];
      int* slots = (int*)malloc(sizeof(int) * (size_t)(L + max_tree + 1));
      double* s = (double*)malloc(sizeof(double) * (size_t)(L + max_tree + 1));
      if (!slots || !s) {
        failed = 1;
        free(slots);
        free(s);
        continue;
      }
      for (int i = 0; i < n; ++i) {
        const uint16_t* qi = q + (((size_t)b * max_tree + i) * num_q_heads + h) * D;
        double* oi = out + (((size_t)b * max_tree + i) * num_q_heads + h) * D;
        int cnt = 0;
        for (int j = 0; j < L; ++j) slots[cnt++] = j;                      /* the whole prefix */
        for (int c = i; c >= 0; c = par[c]) slots[cnt++] = L + c;          /* then the root path of node i */
        double smax = -INFINITY;
        for (int t = 0; t < cnt; ++t) {
          const uint8_t* kj = kb + (size_t)slots[t] * D;
          double acc = 0.0;
          for (int d = 0; d < D; ++d) acc += bf16_to_f64(qi[d]) * (e4m3_to_f64(kj[d]) * ks);
          s[t] = sm_scale * acc;
          if (s[t] > smax) smax = s[t];
        }
        double denom = 0.0;
        for (int t = 0; t < cnt; ++t) {
          s[t] = exp(s[t] - smax);
          denom += s[t];
        }
        for (int d = 0; d < D; ++d) {
          double acc = 0.0;
          for (int t = 0; t < cnt; ++t) acc += s[t] * (e4m3_to_f64(vb[(size_t)slots[t] * D + d]) * vs);
          oi[d] = acc / denom;
        }
      }
      free(slots);
      free(s);
    }
  }
  return failed ? ORACLE_ERR_NOMEM : ORACLE_OK;
}

/*
 * The fp8 cache kept in pages: both storage choices at once (reading as for the two functions above; the scales
 * stay per (sequence, KV head), pages belong to one sequence).
 *
 *   k_pages     e4m3 codes [num_pages, num_kv_heads, page_size, head_dim]   (v_pages alike)
 *   block_table int32 [batch, max_pages_per_seq]: logical slot j of sequence b is row j % page_size of page
 *               block_table[b, j / page_size]
 *
 * By definition: the slots a sequence can see (j < L_b + tree size) are copied out of their pages into a contiguous
 * cache of codes of capacity max_pages_per_seq * page_size, and the contiguous fp8 definition is applied.
 */
int oracle_tree_verify_attn_fp8_paged(int batch, int num_q_heads, int num_kv_heads, int head_dim, int max_tree,
                                      int num_pages, int page_size, int max_pages_per_seq, const int32_t* tree_sizes,
                                      double sm_scale, const uint16_t* q, const uint8_t* k_pages, const uint8_t* v_pages,
                                      const float* k_scale, const float* v_scale, const int32_t* block_table,
                                      const int32_t* seq_lens, const int32_t* tree_parent, double* out) {
  if (batch < 0 || num_kv_heads <= 0 || head_dim <= 0 || num_pages < 0 || page_size <= 0 || max_pages_per_seq < 0 ||
      !block_table || !seq_lens)
    return ORACLE_ERR_ARG;
  const size_t cap = (size_t)max_pages_per_seq * page_size, D = (size_t)head_dim;
  if (cap > 0x7fffffffu) return ORACLE_ERR_ARG;
  const size_t elems = (size_t)batch * num_kv_heads * cap * D;
  uint8_t* kc = (uint8_t*)calloc(elems ? elems : 1, 1);
  uint8_t* vc = (uint8_t*)calloc(elems ? elems : 1, 1);
  int rc = (kc && vc) ? ORACLE_OK : ORACLE_ERR_NOMEM;
  for (int b = 0; b < batch && rc == ORACLE_OK; ++b) {
    const int n = tree_size_of(tree_sizes, b, max_tree);
    if (n < 0 || n > max_tree || seq_lens[b] < 0 || (size_t)seq_lens[b] + n > cap) {
      rc = ORACLE_ERR_ARG;
      break;
    }
    const int visible = n > 0 ? seq_lens[b] + n : 0;
    for (int j = 0; j < visible && rc == ORACLE_OK; ++j) {
      const int page = block_table[(size_t)b * max_pages_per_seq + j / page_size], row = j % page_size;
      if (page < 0 || page >= num_pages) {
        rc = ORACLE_ERR_ARG;
        break;
      }
      for (int g = 0; g < num_kv_heads; ++g) {
        const size_t src = (((size_t)page * num_kv_heads + g) * page_size + row) * D;
        const size_t dst = (((size_t)b * num_kv_heads + g) * cap + j) * D;
        memcpy(kc + dst, k_pages + src, D);
        memcpy(vc + dst, v_pages + src, D);
      }
    }
  }
  if (rc == ORACLE_OK)
    rc = oracle_tree_verify_attn_fp8(batch, num_q_heads, num_kv_heads, head_dim, max_tree, (int)cap, tree_sizes, sm_scale, q,
                                     kc, vc, k_scale, v_scale, seq_lens, tree_parent, out);
  free(kc);
  free(vc);
  return rc;
}

/*
 * Acceptance along the tree.
 *
 *   target_probs fp32 [batch, max_tree + 1, vocab]  row 0: distribution after the committed context;
 *                                                    row i + 1: distribution after tree node i
 *   draft_probs  fp32 [batch, max_tree, vocab]       row i: the distribution node i's token was drawn from
 *   draft_tokens int32 [batch, max_tree]
 *   tree_parent  int32 [batch, max_tree]
 *   uniforms     fp32 [batch, max_tree + 1]          entry i: the r of node i's accept test;
 *                                                    entry max_tree: the final draw
 *   greedy       uint8 [batch] or NULL               1: temperature-0 rule for that sequence
 *   accepted_path int32 [batch, path_cap] (-1 padded), bonus_token int32 [batch], accept_len int32 [batch]
 *   min_margin   fp64 [batch] or NULL: smallest distance to a decision boundary met on the walk
 *                (accept test: |r - p(t)/p^(t)|; final draw: distance of u to the nearer edge of the
 *                chosen cell of the normalised CDF; greedy: gap between the two largest probabilities)
 *   n_sweeps     int32 [batch] or NULL: vocabulary-wide passes the walk needed (rejections + final draw,
 *                or one argmax per visited node)
 *   n_zero_mass  int32 [batch] or NULL: rejections whose residual had zero mass (distribution kept)
 *   n_dec, dec_kind, dec_node, dec_margin (all or none; int32 [batch], int32 / int32 / fp64 [batch, max_tree + 1]):
 *                the walk's decisions one by one, in the order they were taken, so that a differing result can be
 *                traced to the first decision that differs.  kind ORACLE_DEC_ACCEPT / ORACLE_DEC_REJECT: the accept
 *                test of candidate `node` and its outcome, margin |r - p(t)/p^(t)| (+inf when p^(t) = 0);
 *                ORACLE_DEC_BONUS: the final draw at `node` (-1 = the context), margin = distance of u to the nearer
 *                edge of the chosen cell of the normalised CDF; ORACLE_DEC_ARGMAX: the greedy argmax at `node`,
 *                margin = gap between the two largest probabilities.  A walk takes at most max_tree + 1 decisions
 *                (every node is tested at most once, then one draw; or one argmax per visited node).
 *
 * Walk (Sec. 3.3: Algorithm 1 applied at every node, starting from the root):
 *   cur = context.  p = target row of cur (used as given, each node starts from its own row).
 *   Candidates = children of cur, ascending node index (Algorithm 1's i = 1..k).
 *   Stochastic (Algorithm 1): for each candidate i with token t: r = uniforms[i]; accept iff
 *   r < p(t)/p^_i(t), evaluated as r * p^_i(t) < p(t) so that p^_i(t) = 0 needs no division;
 *   on rejection p <- norm(max(0, p - p^_i)) over the whole vocabulary (the Preliminaries' vector
 *   form of the update; Algorithm 1 prints it with scalar arguments); zero residual mass keeps p.
 *   After the candidates are exhausted (k = 0 at a leaf included) draw x ~ p by inverse CDF in
 *   ascending token id with u = uniforms[max_tree]: smallest x with cumsum(x) > u * total.
 *   Greedy: a = argmax p (lowest id on ties); move to the lowest-index child whose token is a,
 *   else emit a.  Exactly one extra token is emitted per call.
 */
/* One row of a distribution as fp64: the fp32 probabilities as given, or (logits != 0) the softmax of the fp32
 * logits at the given temperature, p(v) = exp((z_v - max z) / T) / sum, every operation in fp64. */
static void load_row(double* dst, const float* row, int vocab, int logits, double temperature) {
  if (!logits) {
    for (int v = 0; v < vocab; ++v) dst[v] = (double)row[v];
    return;
  }
  double zmax = -INFINITY;
  for (int v = 0; v < vocab; ++v)
    if ((double)row[v] > zmax) zmax = (double)row[v];
  double sum = 0.0;
  for (int v = 0; v < vocab; ++v) {
    dst[v] = exp(((double)row[v] - zmax) / temperature);
    sum += dst[v];
  }
  for (int v = 0; v < vocab; ++v) dst[v] /= sum;
}

static int accept_walk(int batch, int max_tree, int vocab, int path_cap, const int32_t* tree_sizes,
                       const uint8_t* greedy, const float* target_probs, const float* draft_probs,
                       const int32_t* draft_tokens, const int32_t* tree_parent, const float* uniforms,
                       int32_t* accepted_path, int32_t* bonus_token, int32_t* accept_len,
                       double* min_margin, int32_t* n_sweeps, int32_t* n_zero_mass, int32_t* n_dec, int32_t* dec_kind,
                       int32_t* dec_node, double* dec_margin, int logits, double temperature) {
  if (batch < 0 || max_tree < 0 || max_tree > 64 || vocab <= 0 || path_cap < 0 || !target_probs ||
      !tree_parent || !draft_tokens || !accepted_path || !bonus_token)
    return ORACLE_ERR_ARG;
  if (n_dec && (!dec_kind || !dec_node || !dec_margin)) return ORACLE_ERR_ARG;
  for (int b = 0; b < batch; ++b) {
    const int n = tree_size_of(tree_sizes, b, max_tree);
    if (n < 0 || n > max_tree) return ORACLE_ERR_ARG;
    if (!tree_valid(tree_parent + (size_t)b * max_tree, n)) return ORACLE_ERR_TREE;
    for (int i = 0; i < n; ++i) {
      const int t = draft_tokens[(size_t)b * max_tree + i];
      if (t < 0 || t >= vocab) return ORACLE_ERR_ARG;
    }
    const int is_greedy = greedy ? greedy[b] != 0 : 0;
    if (!is_greedy && (!draft_probs || !uniforms)) return ORACLE_ERR_ARG;
  }
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < batch; ++b) {
    const int n = tree_size_of(tree_sizes, b, max_tree);
    const int is_greedy = greedy ? greedy[b] != 0 : 0;
    const int32_t* par = tree_parent + (size_t)b * max_tree;
    const int32_t* tok = draft_tokens + (size_t)b * max_tree;
    int32_t* path = accepted_path + (size_t)b * path_cap;
    for (int j = 0; j < path_cap; ++j) path[j] = -1;
    double* p = (double*)malloc(sizeof(double) * 2 * (size_t)vocab);
    if (!p) {
      failed = 1;
      continue;
    }
    double* q = p + vocab;   /* the draft row of the candidate under test */
    int cur = -1, len = 0, sweeps = 0, zero_mass = 0, bonus = -1, decisions = 0;
    double margin = INFINITY;
    const size_t dec0 = (size_t)b * (max_tree + 1);
    for (;;) {
      const float* prow = target_probs + ((size_t)b * (max_tree + 1) + (size_t)(cur + 1)) * vocab;
      load_row(p, prow, vocab, logits, temperature);
      int next = -1;
      if (is_greedy) {
        int a = 0;
        for (int v = 1; v < vocab; ++v)
          if (p[v] > p[a]) a = v;
        double second = -INFINITY;
        for (int v = 0; v < vocab; ++v)
          if (v != a && p[v] > second) second = p[v];
        if (vocab > 1 && p[a] - second < margin) margin = p[a] - second;
        if (n_dec) {
          dec_kind[dec0 + decisions] = ORACLE_DEC_ARGMAX;
          dec_node[dec0 + decisions] = cur;
          dec_margin[dec0 + decisions] = vocab > 1 ? p[a] - second : INFINITY;
          ++decisions;
        }
        ++sweeps;
        for (int i = 0; i < n && next < 0; ++i)
          if (par[i] == cur && tok[i] == a) next = i;
        if (next < 0) bonus = a;
      } else {
        for (int i = 0; i < n && next < 0; ++i) {
          if (par[i] != cur) continue;
          const float* qrow = draft_probs + ((size_t)b * max_tree + i) * vocab;
          const int t = tok[i];
          const double r = (double)uniforms[(size_t)b * (max_tree + 1) + i];
          load_row(q, qrow, vocab, logits, temperature);
          const double pt = p[t], qt = q[t];
          const double m_test = qt > 0.0 ? fabs(r - pt / qt) : INFINITY;
          if (m_test < margin) margin = m_test;
          if (n_dec) {
            dec_kind[dec0 + decisions] = r * qt < pt ? ORACLE_DEC_ACCEPT : ORACLE_DEC_REJECT;
            dec_node[dec0 + decisions] = i;
            dec_margin[dec0 + decisions] = m_test;
            ++decisions;
          }
          if (r * qt < pt) {
            next = i;
          } else {
            double Z = 0.0;
            for (int v = 0; v < vocab; ++v) {
              const double d = p[v] - q[v];
              Z += d > 0.0 ? d : 0.0;
            }
            ++sweeps;
            if (Z > 0.0) {
              for (int v = 0; v < vocab; ++v) {
                const double d = p[v] - q[v];
                p[v] = (d > 0.0 ? d : 0.0) / Z;
              }
            } else {
              ++zero_mass;
            }
          }
        }
        if (next < 0) {
          const double u = (double)uniforms[(size_t)b * (max_tree + 1) + max_tree];
          double total = 0.0;
          for (int v = 0; v < vocab; ++v) total += p[v];
          const double thr = u * total;
          double c = 0.0, c_prev = 0.0;
          int x = -1, last_pos = -1;
          double m_draw = 0.0;   /* rounding left no cell above the threshold: the draw sits on the last edge */
          for (int v = 0; v < vocab; ++v) {
            if (p[v] > 0.0) last_pos = v;
            c_prev = c;
            c += p[v];
            if (c > thr) {
              x = v;
              break;
            }
          }
          if (x < 0) {
            x = last_pos >= 0 ? last_pos : vocab - 1;
          } else if (total > 0.0) {
            const double lo = (thr - c_prev) / total, hi = (c - thr) / total;
            m_draw = lo < hi ? lo : hi;
            if (m_draw < margin) margin = m_draw;
          }
          if (n_dec) {
            dec_kind[dec0 + decisions] = ORACLE_DEC_BONUS;
            dec_node[dec0 + decisions] = cur;
            dec_margin[dec0 + decisions] = m_draw;
            ++decisions;
          }
          ++sweeps;
          bonus = x;
        }
      }
      if (next < 0) break;
      if (len < path_cap) path[len] = next;
      ++len;
      cur = next;
    }
    bonus_token[b] = bonus;
    if (accept_len) accept_len[b] = len;
    if (min_margin) min_margin[b] = margin;
    if (n_sweeps) n_sweeps[b] = sweeps;
    if (n_zero_mass) n_zero_mass[b] = zero_mass;
    if (n_dec) n_dec[b] = decisions;
    free(p);
  }
  return failed ? ORACLE_ERR_NOMEM : ORACLE_OK;
}

int oracle_tree_accept(int batch, int max_tree, int vocab, int path_cap, const int32_t* tree_sizes,
                       const uint8_t* greedy, const float* target_probs, const float* draft_probs,
                       const int32_t* draft_tokens, const int32_t* tree_parent, const float* uniforms,
                       int32_t* accepted_path, int32_t* bonus_token, int32_t* accept_len,
                       double* min_margin, int32_t* n_sweeps, int32_t* n_zero_mass, int32_t* n_dec, int32_t* dec_kind,
                       int32_t* dec_node, double* dec_margin) {
  return accept_walk(batch, max_tree, vocab, path_cap, tree_sizes, greedy, target_probs, draft_probs, draft_tokens,
                     tree_parent, uniforms, accepted_path, bonus_token, accept_len, min_margin, n_sweeps, n_zero_mass, n_dec,
                     dec_kind, dec_node, dec_margin, 0, 1.0);
}

/*
 * The same walk on LOGITS: every target / draft row is the softmax of the given fp32 logits at `temperature` > 0
 * (Sec. 4: the experiments sample at temperature 1; temperature 0 is the greedy flag), taken in fp64.  Greedy
 * sequences use the argmax, which the softmax does not move.
 */
int oracle_tree_accept_logits(int batch, int max_tree, int vocab, int path_cap, const int32_t* tree_sizes,
                              const uint8_t* greedy, const float* target_logits, const float* draft_logits,
                              const int32_t* draft_tokens, const int32_t* tree_parent, const float* uniforms,
                              double temperature, int32_t* accepted_path, int32_t* bonus_token, int32_t* accept_len,
                              double* min_margin, int32_t* n_sweeps, int32_t* n_zero_mass, int32_t* n_dec, int32_t* dec_kind,
                              int32_t* dec_node, double* dec_margin) {
  if (!(temperature > 0.0)) return ORACLE_ERR_ARG;
  return accept_walk(batch, max_tree, vocab, path_cap, tree_sizes, greedy, target_logits, draft_logits, draft_tokens,
                     tree_parent, uniforms, accepted_path, bonus_token, accept_len, min_margin, n_sweeps, n_zero_mass, n_dec,
                     dec_kind, dec_node, dec_margin, 1, temperature);
}

/*
 * Commit of the accepted path (Sec. 3.3: accepted tokens and their features are kept for the next drafting phase).
 *
 * Readings (the paper does not say where anything is stored): tree node m's key / value rows sit at cache slot
 * L + m (as in oracle_tree_verify_attn); after the step the accepted nodes path[0..a-1] are part of the committed
 * prefix, so slot L + j must hold what slot L + path[j] held, for every j < a at once, and the new prefix length
 * is L + a.  Slots below L and from L + a on are left as they are.  features_out[b, j] = features_in[b, path[j]]
 * for j < a and zeros for j >= a.  accepted_path rows hold node indices from the top of the tree down, then -1.
 * A row that is not strictly increasing, leaves [0, max_tree) or points past the cache marks the sequence invalid:
 * nothing of it is moved, its length stays L, its feature rows are zeros, valid[b] = 0.
 *
 * k_cache, v_cache: bf16 bit patterns [B, Hkv, S_cap, D], modified in place (either may be NULL).
 * features_in [B, max_tree, F], features_out [B, path_cap, F]: bf16 bit patterns (both NULL when F = 0).
 */
int oracle_tree_commit(int batch, int num_kv_heads, int head_dim, int kv_capacity, int max_tree, int path_cap,
                       const int32_t* seq_lens, const int32_t* accepted_path, uint16_t* k_cache, uint16_t* v_cache,
                       int feature_dim, const uint16_t* features_in, uint16_t* features_out, int32_t* new_seq_lens,
                       int32_t* valid) {
  if (batch < 0 || num_kv_heads < 0 || head_dim < 0 || kv_capacity < 0 || max_tree < 0 || path_cap < 0 || feature_dim < 0)
    return ORACLE_ERR_ARG;
  if (!seq_lens || !accepted_path) return ORACLE_ERR_ARG;
  const size_t row = (size_t)head_dim;
  uint16_t* tmp = (uint16_t*)malloc(sizeof(uint16_t) * row * (size_t)(path_cap > 0 ? path_cap : 1));
  if (!tmp) return ORACLE_ERR_NOMEM;
  for (int b = 0; b < batch; ++b) {
    const int32_t* path = accepted_path + (size_t)b * path_cap;
    const int L = seq_lens[b];
    int a = 0, ok = L >= 0;
    while (a < path_cap && path[a] != -1) ++a;                       /* accepted length: entries before the first -1 */
    for (int j = 0; j < a && ok; ++j) {
      if (path[j] < 0 || path[j] >= max_tree) ok = 0;                /* a tree node */
      else if (j > 0 && path[j] <= path[j - 1]) ok = 0;              /* a child comes after its parent */
      else if ((long long)L + path[j] >= kv_capacity) ok = 0;        /* its slot exists */
    }
    if (valid) valid[b] = ok;
    if (new_seq_lens) new_seq_lens[b] = ok ? L + a : L;
    if (features_out)
      memset(features_out + (size_t)b * path_cap * feature_dim, 0, sizeof(uint16_t) * (size_t)path_cap * feature_dim);
    if (!ok) continue;
    for (int t = 0; t < 2; ++t) {
      uint16_t* cache = t == 0 ? k_cache : v_cache;
      if (!cache) continue;
      for (int g = 0; g < num_kv_heads; ++g) {
        uint16_t* base = cache + ((size_t)b * num_kv_heads + g) * (size_t)kv_capacity * row;
        /* simultaneous assignment: read every source row, then write every destination row */
        for (int j = 0; j < a; ++j) memcpy(tmp + (size_t)j * row, base + (size_t)(L + path[j]) * row, sizeof(uint16_t) * row);
        for (int j = 0; j < a; ++j) memcpy(base + (size_t)(L + j) * row, tmp + (size_t)j * row, sizeof(uint16_t) * row);
      }
    }
    if (features_in && features_out)
      for (int j = 0; j < a; ++j)
        memcpy(features_out + ((size_t)b * path_cap + j) * feature_dim, features_in + ((size_t)b * max_tree + path[j]) * feature_dim,
               sizeof(uint16_t) * (size_t)feature_dim);
  }
  free(tmp);
  return ORACLE_OK;
}

/*
 * The same commit when the cache is kept in pages: slot j of sequence b is row j % page_size of page
 * block_table[b, j / page_size] of k_pages / v_pages [num_pages, Hkv, page_size, D] (modified in place).  The rule is
 * the one above with that address map; the capacity is max_pages_per_seq * page_size, and a path one of whose
 * source or destination slots lies on a page outside [0, num_pages) is invalid as well.  Pages are not moved or
 * allocated: the accepted rows are copied between (or within) the pages the sequence already owns.
 */
int oracle_tree_commit_paged(int batch, int num_kv_heads, int head_dim, int num_pages, int page_size, int max_pages_per_seq,
                             int max_tree, int path_cap, const int32_t* seq_lens, const int32_t* accepted_path,
                             const int32_t* block_table, uint16_t* k_pages, uint16_t* v_pages, int32_t* new_seq_lens,
                             int32_t* valid) {
  if (batch < 0 || num_kv_heads < 0 || head_dim < 0 || num_pages < 0 || page_size <= 0 || max_pages_per_seq < 0 || max_tree < 0 ||
      path_cap < 0 || !seq_lens || !accepted_path || !block_table)
    return ORACLE_ERR_ARG;
  const size_t row = (size_t)head_dim;
  const long long capacity = (long long)max_pages_per_seq * page_size;
  uint16_t* tmp = (uint16_t*)malloc(sizeof(uint16_t) * row * (size_t)(path_cap > 0 ? path_cap : 1));
  if (!tmp) return ORACLE_ERR_NOMEM;
  for (int b = 0; b < batch; ++b) {
    const int32_t* path = accepted_path + (size_t)b * path_cap;
    const int32_t* table = block_table + (size_t)b * max_pages_per_seq;
    const int L = seq_lens[b];
    int a = 0, ok = L >= 0;
    while (a < path_cap && path[a] != -1) ++a;
    for (int j = 0; j < a && ok; ++j) {
      if (path[j] < 0 || path[j] >= max_tree) ok = 0;
      else if (j > 0 && path[j] <= path[j - 1]) ok = 0;
      else if ((long long)L + path[j] >= capacity) ok = 0;
      else {
        const int src = table[(L + path[j]) / page_size], dst = table[(L + j) / page_size];
        if (src < 0 || src >= num_pages || dst < 0 || dst >= num_pages) ok = 0;
      }
    }
    if (valid) valid[b] = ok;
    if (new_seq_lens) new_seq_lens[b] = ok ? L + a : L;
    if (!ok) continue;
    for (int t = 0; t < 2; ++t) {
      uint16_t* pages = t == 0 ? k_pages : v_pages;
      if (!pages) continue;
      for (int g = 0; g < num_kv_heads; ++g) {
        /* simultaneous assignment: read every source row, then write every destination row */
        for (int j = 0; j < a; ++j) {
          const int s = L + path[j];
          memcpy(tmp + (size_t)j * row, pages + (((size_t)table[s / page_size] * num_kv_heads + g) * page_size + s % page_size) * row,
                 sizeof(uint16_t) * row);
        }
        for (int j = 0; j < a; ++j) {
          const int d = L + j;
          memcpy(pages + (((size_t)table[d / page_size] * num_kv_heads + g) * page_size + d % page_size) * row, tmp + (size_t)j * row,
                 sizeof(uint16_t) * row);
        }
      }
    }
  }
  free(tmp);
  return ORACLE_OK;
}

/*
 * Child tokens of draft-tree nodes (App. A.1: in the greedy setting the k most probable tokens become the children,
 * otherwise k tokens are sampled; k differs from node to node).
 *
 * probs [B, R, V] fp32: the draft distribution at each of R nodes per sequence (used as given, not renormalised);
 * num_children [B, R]: k of each node, 0 <= k <= max_children; greedy [B] or NULL; uniforms [B, R, max_children]
 * (needed by stochastic sequences).  Outputs: tokens [B, R, max_children] (-1 past k), token_probs (0 past k).
 * Readings (the paper gives neither a tie rule nor a sampling scheme): top-k is by descending probability with the
 * lower token id first among equal values; the k samples are independent draws with replacement, draw j being the
 * smallest x with sum_{v<=x} p(v) > uniforms[j] * sum_v p(v) (the inverse CDF in ascending token id, as in
 * oracle_tree_accept; the last token with positive mass if rounding leaves none).  min_margin [B, R] (optional):
 * the smallest distance, as a fraction of the row's mass, between a draw's threshold and the edges of the cell it
 * fell into; +inf for greedy rows.
 */
int oracle_tree_expand(int batch, int rows, int vocab, int max_children, const int32_t* num_children,
                       const uint8_t* greedy, const float* probs, const float* uniforms, int32_t* tokens,
                       float* token_probs, double* min_margin) {
  if (batch < 0 || rows < 0 || vocab <= 0 || max_children < 0 || !num_children || !probs || !tokens) return ORACLE_ERR_ARG;
  for (long long i = 0; i < (long long)batch * rows; ++i) {
    const int g = greedy && greedy[i / rows];
    if (num_children[i] < 0 || num_children[i] > max_children) return ORACLE_ERR_ARG;
    if (g && num_children[i] > vocab) return ORACLE_ERR_ARG;       /* k distinct tokens */
    if (!g && !uniforms) return ORACLE_ERR_ARG;
  }
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long long i = 0; i < (long long)batch * rows; ++i) {
    const int b = (int)(i / rows), k = num_children[i];
    const float* p = probs + (size_t)i * vocab;
    int32_t* out = tokens + (size_t)i * max_children;
    float* outp = token_probs ? token_probs + (size_t)i * max_children : NULL;
    for (int j = 0; j < max_children; ++j) {
      out[j] = -1;
      if (outp) outp[j] = 0.f;
    }
    double margin = INFINITY;
    if (greedy && greedy[b]) {
      /* k rounds: the most probable token not taken yet, lowest id among equals */
      unsigned char* taken = (unsigned char*)calloc((size_t)vocab, 1);
      if (!taken) {
        failed = 1;
        continue;
      }
      for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int v = 0; v < vocab; ++v)
          if (!taken[v] && (best < 0 || p[v] > p[best])) best = v;
        taken[best] = 1;
        out[j] = best;
        if (outp) outp[j] = p[best];
      }
      free(taken);
    } else {
      double total = 0.0;
      for (int v = 0; v < vocab; ++v) total += (double)p[v];
      for (int j = 0; j < k; ++j) {
        const double thr = (double)uniforms[(size_t)i * max_children + j] * total;
        double c = 0.0, c_prev = 0.0;
        int x = -1, last_pos = -1;
        for (int v = 0; v < vocab; ++v) {
          if (p[v] > 0.f) last_pos = v;
          c_prev = c;
          c += (double)p[v];
          if (c > thr) {
            x = v;
            break;
          }
        }
        if (x < 0) {
          x = last_pos >= 0 ? last_pos : vocab - 1;
        } else if (total > 0.0) {
          const double lo = (thr - c_prev) / total, hi = (c - thr) / total;
          const double m = lo < hi ? lo : hi;
          if (m < margin) margin = m;
        }
        out[j] = x;
        if (outp) outp[j] = p[x];
      }
    }
    if (min_margin) min_margin[i] = margin;
  }
  return failed ? ORACLE_ERR_NOMEM : ORACLE_OK;
}

/* Threads the OpenMP loops above use (reported next to the oracle's timing). */
int oracle_num_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
#endif
  return n;
}

/* Number of threads the OpenMP loops above use from now on (0 or less: the OpenMP default).  Timing aid only: the
 * results do not depend on it (every unit is computed by one thread, in the same order of operations). */
void oracle_set_num_threads(int n) {
#ifdef _OPENMP
  omp_set_num_threads(n > 0 ? n : omp_get_num_procs());
#else
  (void)n;
#endif
}
