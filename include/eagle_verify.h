/*
 * eagle_verify.h - C ABI of the B200 (sm_100a) tree-verification library for EAGLE speculative decoding.
 *
 * The verification phase (Sec. 3.3, App. A.1 and A.2 of the EAGLE paper) scores every token of a
 * tree-structured draft in one target forward pass with tree attention, then walks the tree applying
 * multi-round speculative sampling (Algorithm 1) at every node.  This library implements, for one
 * attention layer and for the acceptance walk, exactly those two operations:
 *
 *   eagle_tree_verify_attn  tree-masked attention of the T draft-tree tokens against the committed
 *                           KV prefix plus the tree's own keys (a node sees the prefix, its ancestors
 *                           and itself)
 *   eagle_tree_accept       acceptance along the tree: greedy, or Algorithm 1 at every node
 *
 * Conventions shared by every call
 *   - Every pointer marked "device" is a device pointer owned by the caller; the library keeps none of
 *     them after the call returns, allocates no memory and never synchronises: work is enqueued on
 *     `stream` and the call returns.  Pointers marked "host" are ordinary host pointers.
 *   - Return value: EAGLE_OK, or a negative EAGLE_ERR_* when the host-side check of the arguments fails
 *     (nothing is launched) or a launch fails.  Problems only the device can see (a parent entry out of
 *     range, a prefix that does not fit the cache, a wait that ran out) are written to `*status`
 *     (device int32, first error wins, 0 = none); the affected sequence's rows are zeroed (attention)
 *     or its outputs set to "nothing accepted, bonus -1" (acceptance).  No trap is ever raised.
 *   - Tree: node i of sequence b has parent tree_parent[b, i] in [-1, i-1]; -1 means "child of the
 *     committed context".  At most 64 nodes per tree.  Entries at i >= tree size are ignored.
 */
#ifndef EAGLE_VERIFY_H_
#define EAGLE_VERIFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque CUDA handles: a cudaStream_t / cudaEvent_t passed as a pointer-sized value. */
typedef void* eagle_stream_t;
typedef void* eagle_event_t;

enum {
  EAGLE_OK = 0,
  EAGLE_ERR_NULL = -1,       /* a required pointer is NULL */
  EAGLE_ERR_SHAPE = -2,      /* batch / heads / head_dim / max_tree / vocab out of the supported range */
  EAGLE_ERR_WORKSPACE = -3,  /* workspace missing, misaligned (256 B) or too small */
  EAGLE_ERR_LAUNCH = -4,     /* CUDA reported an error when launching */
  EAGLE_ERR_TREE = -5,       /* device-detected: parent entry outside [-1, i-1], or tree size out of range */
  EAGLE_ERR_SEQ = -6,        /* device-detected: seq_lens[b] < 0 or seq_lens[b] + tree size > kv_capacity */
  EAGLE_ERR_TOKEN = -7,      /* device-detected: draft token outside [0, vocab) */
  EAGLE_ERR_TIMEOUT = -8,    /* device-detected: a bounded wait inside a kernel ran out */
  EAGLE_ERR_DEVICE = -9,     /* the GPU is not an sm_100 device, or it lacks a required limit */
  EAGLE_ERR_PATH = -10,      /* device-detected: an accepted path that is not an increasing list of tree nodes whose slots exist */
  EAGLE_ERR_PAGE = -11       /* device-detected: a block-table entry of a page in use outside [0, num_pages) */
};

#define EAGLE_MAX_TREE 64

/*
 * Descriptor of one attention call.  Plain data, read during the call only.
 */
typedef struct eagle_attn_desc {
  int32_t batch;               /* B >= 0 */
  int32_t num_q_heads;         /* Hq; Hq % Hkv == 0, group size G = Hq / Hkv <= 16 */
  int32_t num_kv_heads;        /* Hkv */
  int32_t head_dim;            /* D: 64 or 128 */
  int32_t max_tree;            /* T_max <= 64: row stride of tree_parent, q and out */
  int32_t kv_capacity;         /* S_cap: slots per (sequence, KV head) of k_cache / v_cache */
  const int32_t* tree_sizes;   /* device int32 [B], or NULL: every tree has T_max nodes */
  float sm_scale;              /* softmax scale, > 0; 0 means 1/sqrt(D); negative or NaN is EAGLE_ERR_SHAPE */
  int32_t num_splits;          /* KV splits per sequence; 0 lets the device-side planner choose */
  void* workspace;             /* device, 256-byte aligned, >= eagle_tree_verify_attn_workspace() bytes */
  size_t workspace_bytes;
  int32_t* status;             /* device int32 or NULL */
  eagle_event_t ev_attn_begin; /* optional: recorded on `stream` right before / after the split-KV   */
  eagle_event_t ev_attn_end;   /* attention kernel (the dominant kernel), for timing it alone; or NULL */
  int32_t shared_tree;         /* nonzero: one tree for every sequence (the paper's experiments use one fixed tree shape,
                                  App. A.1): tree_parent is int32 [T_max] and tree_sizes NULL or int32 [1] */
} eagle_attn_desc;

/* Bytes of scratch one call with this descriptor needs (host function, no CUDA work).
 * Depends on batch, heads, head_dim, max_tree and num_splits only.  Returns 0 if the shape is unsupported.
 * With num_splits = 0 it is about 35 MB whatever the batch (plus some 100 bytes per (sequence, KV head, 256 query rows)). */
size_t eagle_tree_verify_attn_workspace(const eagle_attn_desc* desc);

/*
 * Tree-masked attention of one layer (tree attention of the verification pass: Sec. 3.3, App. A.1).
 *
 *   q        device bf16 [B, T_max, Hq, D]        queries of the tree tokens (already position-encoded)
 *   k_cache  device bf16 [B, Hkv, S_cap, D]       keys; slots [0, L_b) hold the committed prefix, slot
 *   v_cache  device bf16 [B, Hkv, S_cap, D]       L_b + m holds tree node m; later slots are never used
 *                                                 in the result, whatever they contain (NaN included)
 *   seq_lens device int32 [B]                     L_b, the committed prefix length (tree not included)
 *   tree_parent device int32 [B, T_max]           ([T_max] when desc->shared_tree is set)
 *   out      device bf16 [B, T_max, Hq, D]        out[b,i,h,:] = sum_j softmax_j(scale * q[b,i,h]·k[b,h/G,j]) v[b,h/G,j]
 *                                                 over j < L_b and j = L_b + m, m an ancestor of i or i itself;
 *                                                 rows of nodes i >= tree size are written as zeros
 *
 * Arithmetic: bf16 inputs, fp32 scores / softmax / accumulation, bf16 output (round to nearest even).
 * q, k_cache and v_cache must be 16-byte aligned, out 32-byte aligned (else EAGLE_ERR_SHAPE).  Launches, in order on `stream`: the planner (tree masks +
 * work list), the split-KV attention kernel, the combine kernel.  The workspace must not be shared by
 * calls that can overlap on the GPU.
 */
int eagle_tree_verify_attn(const eagle_attn_desc* desc, const void* q, const void* k_cache, const void* v_cache,
                           const int32_t* seq_lens, const int32_t* tree_parent, void* out, eagle_stream_t stream);

/*
 * The same attention, for callers that cannot provide a workspace.  (The paper has no counterpart to this entry
 * point: it exists for the way the library is embedded, not for the method.)
 *
 * Who needs it: code that receives device pointers for its tensors but may not allocate device memory when it
 * runs - a serving backend whose memory pool is fixed at start-up, a plug-in living inside another engine's
 * execution context, a decode loop that must never call cudaMalloc because that call stalls the whole device.
 * Here the planner tables and the split partials live in a fixed array inside the library's device image,
 * eagle_tree_verify_attn_static_capacity() bytes (24 MiB) per GPU that loads the library, held until the
 * process ends.  `desc->workspace` and `desc->workspace_bytes` are ignored; everything else is as for
 * eagle_tree_verify_attn, and so are the results.
 *
 *   - No cudaMalloc, cudaFree or other allocating call is made, on any call.
 *   - Shapes whose tables and partials do not fit the array are refused with EAGLE_ERR_WORKSPACE and nothing is
 *     launched.  The need grows with batch * num_kv_heads * ceil(max_tree * G / 128), and steeply with a
 *     forced num_splits > 1; with num_splits = 0 the partials take (2 * (number of SMs) + 2 * batch if num_kv_heads is
 *     odd) * 128 * (D + 2) * 4 bytes (19.7 MB on a 148-SM B200 at D = 128), which leaves room for the tables of some 30 000
 *     (sequence, KV head, 256 query rows) units.
 *   - The first call on a device looks up the array's device address (once per device, with that device
 *     current).  Make that first call outside any stream capture.
 *   - All calls on one GPU share the one array, and it keeps the previous call's contents.  Nothing in it needs
 *     to start at zero (the planner kernel rewrites every table that is read, and each partial is written
 *     before it is merged), but two calls that can overlap on the GPU - different streams, or graphs replayed
 *     concurrently - would overwrite each other's plan: issue them on one stream, or order them yourself.
 */
int eagle_tree_verify_attn_static(const eagle_attn_desc* desc, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* seq_lens, const int32_t* tree_parent, void* out, eagle_stream_t stream);

/* Size in bytes of the fixed array used by eagle_tree_verify_attn_static (host function). */
size_t eagle_tree_verify_attn_static_capacity(void);

/*
 * A KV cache kept in pages (a storage layout of the same cache: the verification pass of Sec. 3.3 reads the same keys
 * and values wherever a serving engine stores them).
 */
typedef struct eagle_paged_kv {
  const void* k_pages;          /* device bf16 [num_pages, Hkv, page_size, D], 16-byte aligned (uint8 codes for the _fp8 calls) */
  const void* v_pages;          /* device bf16 [num_pages, Hkv, page_size, D], 16-byte aligned */
  const int32_t* block_table;   /* device int32 [B, max_pages_per_seq]: slot j of sequence b is row j % page_size of page
                                   block_table[b, j / page_size]; entries of pages that hold no slot below
                                   seq_lens[b] + tree size are never read */
  int32_t num_pages;            /* pages in the pool, >= 1 */
  int32_t page_size;            /* slots per page: a power of two, >= 16 */
  int32_t max_pages_per_seq;    /* row length of block_table; a sequence holds at most max_pages_per_seq * page_size slots */
} eagle_paged_kv;

/*
 * eagle_tree_verify_attn over a paged cache.  Everything is as for that call (same planner, same kernels, same
 * arithmetic and results, same workspace size) except where the keys and values are read from: each 128-slot tile
 * is fetched page by page through the block table (one TMA box per page, or one box out of a page of 128 slots or
 * more).  desc->kv_capacity is ignored: the capacity is max_pages_per_seq * page_size.  A sequence whose prefix + tree
 * does not fit it reports EAGLE_ERR_SEQ, one with a block-table entry in use outside [0, num_pages) reports
 * EAGLE_ERR_PAGE; its output rows are zeros and no page is read for it.
 */
int eagle_tree_verify_attn_paged(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* kv,
                                 const int32_t* seq_lens, const int32_t* tree_parent, void* out, eagle_stream_t stream);

/*
 * The same call in two halves, for a verification pass over many layers.  The verification phase is one target
 * forward pass over every layer with the same draft tree and the same prefix lengths (Sec. 3.3, App. A.1); the tree
 * masks and the work split depend on nothing else, so they are made once per pass and reused by every layer:
 *
 *   eagle_tree_verify_plan          the planner alone: masks + work list into desc->workspace (one launch).
 *                                   `paged` is NULL for a contiguous cache; for a paged cache it names the block table
 *                                   (its page pointers are not read), so that the pages in use are validated.
 *   eagle_tree_verify_attn_planned  attention + combine of one layer over the plan in desc->workspace (two launches).
 *   eagle_tree_verify_attn_planned_paged   the same over a paged cache.
 *
 * The descriptor of the planned calls must equal the one the plan was made with (shape fields, num_splits, workspace),
 * on the same GPU; sm_scale, status and the events may differ.  Plan followed by planned gives bit for bit what
 * eagle_tree_verify_attn gives.  The plan stays valid until the workspace is written by another plan; the split
 * partials in the workspace are reused by every planned call, so planned calls that share a workspace must not overlap
 * on the GPU.  Arguments, results and errors as for eagle_tree_verify_attn (device-detected errors of the trees and
 * lengths are reported by the plan call; the planned calls then write zeros for the affected sequences).
 */
int eagle_tree_verify_plan(const eagle_attn_desc* desc, const int32_t* seq_lens, const int32_t* tree_parent,
                           const eagle_paged_kv* paged, eagle_stream_t stream);
int eagle_tree_verify_attn_planned(const eagle_attn_desc* desc, const void* q, const void* k_cache, const void* v_cache,
                                   void* out, eagle_stream_t stream);
int eagle_tree_verify_attn_planned_paged(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* kv, void* out,
                                         eagle_stream_t stream);

/*
 * The same attention over a cache STORED in fp8.  The decoding this method speeds up is bound by memory traffic (Sec. 4.4)
 * and the paper reports the method on a quantised deployment (Sec. 4.2); it fixes no quantisation scheme, so the
 * convention here is this library's: k_codes / v_codes are device uint8 [B, Hkv, S_cap, D] holding fp8 "e4m3" codes (1
 * sign, 4 exponent, 3 mantissa bits, bias 7, no infinities), and every (sequence, KV head) has one fp32 scale for its keys
 * and one for its values, k_scale / v_scale device fp32 [B, Hkv]:  key = value(code) * k_scale[b, h],  value =
 * value(code) * v_scale[b, h].  Only the storage changes: the codes are widened exactly (every e4m3 number is an fp16
 * number) on their way to the tensor cores, the keys' scale is folded into the softmax scale and the values' scale into
 * the output.  A tensor-core instruction takes one 16-bit type for both operands, so this form multiplies in fp16: the
 * bf16 queries are converted to fp16 (exact for magnitudes from 2^-14 to 65504; smaller ones are rounded to multiples of
 * 2^-24, larger ones become infinite) and the probabilities are rounded to fp16 instead of bf16.  Everything else (fp32
 * scores / softmax / accumulation, bf16 output, planner, work split, errors) is as for eagle_tree_verify_attn.  What it
 * saves is half of the cache bytes held and read.  head_dim must be 128 (else EAGLE_ERR_SHAPE).
 * Slots that are not visible may hold any code; one of the two NaN codes (0x7f, 0xff) in a VISIBLE slot makes the output
 * rows that see it NaN.
 * eagle_tree_verify_attn_planned_fp8 is the per-layer half over a plan made by eagle_tree_verify_plan (paged = NULL).
 */
int eagle_tree_verify_attn_fp8(const eagle_attn_desc* desc, const void* q, const void* k_codes, const void* v_codes,
                               const float* k_scale, const float* v_scale, const int32_t* seq_lens, const int32_t* tree_parent,
                               void* out, eagle_stream_t stream);
int eagle_tree_verify_attn_planned_fp8(const eagle_attn_desc* desc, const void* q, const void* k_codes, const void* v_codes,
                                       const float* k_scale, const float* v_scale, void* out, eagle_stream_t stream);

/*
 * The fp8 cache kept in pages: both storage choices of the same cache at once (Sec. 3.3 reads the same keys and values
 * wherever and however a serving engine stores them).  kv->k_pages / kv->v_pages are device uint8
 * [num_pages, Hkv, page_size, D] holding e4m3 codes, addressed through kv->block_table as for
 * eagle_tree_verify_attn_paged; k_scale / v_scale are device fp32 [B, Hkv] as for eagle_tree_verify_attn_fp8 (a page
 * belongs to one sequence, so the scales stay per (sequence, KV head)).  Arithmetic, errors and limits are those of the
 * two calls it combines: head_dim 128 (else EAGLE_ERR_SHAPE), fp16 x fp16 products, EAGLE_ERR_SEQ / EAGLE_ERR_PAGE per
 * sequence.  The planned form runs over a plan made by eagle_tree_verify_plan with the same `paged` description.
 */
int eagle_tree_verify_attn_paged_fp8(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* kv, const float* k_scale,
                                     const float* v_scale, const int32_t* seq_lens, const int32_t* tree_parent, void* out,
                                     eagle_stream_t stream);
int eagle_tree_verify_attn_planned_paged_fp8(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* kv,
                                             const float* k_scale, const float* v_scale, void* out, eagle_stream_t stream);


/*
 * Where a plan keeps its tree masks (host function, no CUDA work): device uint64 [B, T_max] inside desc->workspace,
 * bit m of entry [b, i] set iff node m is node i or one of its ancestors (the mask tree attention implies, Sec. 3.1 /
 * 3.3); entries of nodes >= tree size and of invalid sequences are 0.  Valid after eagle_tree_verify_plan or
 * eagle_tree_verify_attn on that workspace has run.  NULL if the descriptor is unusable.
 */
const uint64_t* eagle_tree_verify_plan_masks(const eagle_attn_desc* desc);

/*
 * How long a wait inside the attention kernel may go without progress before the kernel gives up, in nanoseconds
 * (host function; process-wide; applies to launches made after the call; 0 restores the default of two seconds).
 * Every wait in the kernels is bounded: when one runs out the kernel sets *status to EAGLE_ERR_TIMEOUT, releases what
 * it holds and returns, and the context stays usable.  Keep the limit far above the time a copy takes (milliseconds
 * are safe): a kernel that gives up while its own copies are still in flight would leave them writing into shared
 * memory it no longer owns.
 */
void eagle_set_wait_limit_ns(uint64_t ns);

/*
 * Test hook (fault injection for the time-out path; not for production use): attention launches made after this call
 * have their K/V producer stop issuing copies after `after_tiles` tiles per CTA, so the consumers' waits run out and
 * the kernel reports EAGLE_ERR_TIMEOUT.  Nothing is in flight when it returns.  A negative value switches it off.
 */
void eagle_test_stall_kv_producer(int32_t after_tiles);

/*
 * Descriptor of one acceptance call.
 */
typedef struct eagle_accept_desc {
  int32_t batch;               /* B >= 0 */
  int32_t max_tree;            /* T_max <= 64: row stride of the per-node arrays */
  int32_t vocab;               /* V >= 1 */
  int32_t path_cap;            /* entries per row of accepted_path; >= the deepest tree (T_max is always enough) */
  const int32_t* tree_sizes;   /* device int32 [B] or NULL */
  const uint8_t* greedy;       /* device uint8 [B] or NULL (= every sequence stochastic); 1: temperature-0 rule */
  int32_t* accept_len;         /* device int32 [B] or NULL: number of accepted nodes */
  int32_t* status;             /* device int32 or NULL */
  int32_t shared_tree;         /* nonzero: one tree for every sequence: tree_parent is int32 [T_max], tree_sizes NULL or int32 [1]
                                  (draft_tokens, the probability rows and the uniforms stay per sequence) */
} eagle_accept_desc;

/*
 * Acceptance along the draft tree: Algorithm 1 (multi-round speculative sampling, App. A.2) applied at
 * every node starting from the committed context (Sec. 3.3), or the greedy rule (Preliminaries).
 *
 *   target_probs device fp32 [B, T_max+1, V]   row 0: target distribution after the context;
 *                                              row i+1: target distribution after tree node i
 *   draft_probs  device fp32 [B, T_max, V]     row i: the distribution node i's token was drawn from
 *                                              (may be NULL when every sequence is greedy)
 *   draft_tokens device int32 [B, T_max]
 *   tree_parent  device int32 [B, T_max]      ([T_max] when desc->shared_tree is set)
 *   uniforms     device fp32 [B, T_max+1]      entry i: the uniform of node i's accept test; entry T_max:
 *                                              the uniform of the final draw (may be NULL when all greedy)
 *   accepted_path device int32 [B, path_cap]   accepted node indices from the top of the tree down, then -1
 *   bonus_token  device int32 [B]              the one extra token every step emits
 *
 * Per sequence: cur = context.  The children of cur, in ascending index, are Algorithm 1's candidates
 * against p = target row of cur: candidate i with token t is accepted iff r_i * p^_i(t) < p(t) (that is
 * r_i < p(t)/p^_i(t)); on rejection p <- norm(max(0, p - p^_i)) over the vocabulary (kept if its mass is
 * zero).  An accepted child becomes cur and starts again from its own target row.  When no child is
 * accepted (a leaf included) the bonus token is drawn from p by inverse CDF in ascending token id: the
 * smallest x with sum_{v<=x} p(v) > u * sum_v p(v).  Greedy sequences move to the lowest-index child whose
 * token equals argmax p (lowest id on ties), else emit that argmax.  Rows are used as given (not
 * renormalised).  Scalars and sums are fp64, so decisions agree with an fp64 reference except within
 * rounding of a boundary.
 */
int eagle_tree_accept(const eagle_accept_desc* desc, const float* target_probs, const float* draft_probs,
                      const int32_t* draft_tokens, const int32_t* tree_parent, const float* uniforms,
                      int32_t* accepted_path, int32_t* bonus_token, eagle_stream_t stream);

/*
 * How an acceptance call of this batch size and vocabulary is laid out on the current GPU (host function, launches
 * nothing): 0 when one warp walks each tree (vocabularies up to 4096), else the number of 512-thread CTAs, 1, 2, 4 or
 * 8, that form the thread-block cluster walking one tree (the fewer trees, the wider the cluster).  The result of
 * eagle_tree_accept does not depend on it; it is reported so that every variant can be told apart and exercised.
 * Negative EAGLE_ERR_* on a bad argument or when no sm_100 device is current.
 */
int eagle_tree_accept_cluster_width(int32_t batch, int32_t vocab);
/* The same for a call that passes draft_probs == NULL or uniforms == NULL, i.e. one whose sequences are all greedy (the
 * setting of most of the paper's tables, temperature 0): its walk is argmax sweeps only, and where eight CTAs per tree
 * would not fit the GPU at once it takes four. */
int eagle_tree_accept_cluster_width_greedy(int32_t batch, int32_t vocab);

/*
 * One whole verification step driven from HOST buffers (the two calls above, with the copies around them).
 *
 * Every input pointer below is a host pointer (pinned memory makes the copies asynchronous); the call enqueues on
 * `stream`: host->device copies of the inputs into `arena` (see eagle_tree_verify_step_host_bytes for what is copied),
 * eagle_tree_verify_attn, eagle_tree_accept, and
 * device->host copies of out, accepted_path, bonus_token and accept_len.  It allocates nothing: `arena` is device
 * memory provided by the caller, 256-byte aligned, at least eagle_tree_verify_step_host_arena() bytes (device copies
 * of all tensors plus the attention workspace).  The results are in the host buffers once `stream` has drained.
 * Verification phase: Sec. 3.3; acceptance: App. A.2, Algorithm 1.  Shapes and meanings as for the device calls.
 */
typedef struct eagle_host_step {
  int32_t batch, num_q_heads, num_kv_heads, head_dim, max_tree, kv_capacity, vocab, path_cap;
  float sm_scale;
  const void* q;                 /* host bf16 [B, T_max, Hq, D] */
  const void* k_cache;           /* host bf16 [B, Hkv, S_cap, D] */
  const void* v_cache;
  const int32_t* seq_lens;       /* host int32 [B] */
  const int32_t* tree_sizes;     /* host int32 [B] or NULL */
  const int32_t* tree_parent;    /* host int32 [B, T_max] */
  const float* target_probs;     /* host fp32 [B, T_max+1, V] */
  const float* draft_probs;      /* host fp32 [B, T_max, V] */
  const int32_t* draft_tokens;   /* host int32 [B, T_max] */
  const float* uniforms;         /* host fp32 [B, T_max+1] */
  const uint8_t* greedy;         /* host uint8 [B] or NULL */
  void* out;                     /* host bf16 [B, T_max, Hq, D] */
  int32_t* accepted_path;        /* host int32 [B, path_cap] */
  int32_t* bonus_token;          /* host int32 [B] */
  int32_t* accept_len;           /* host int32 [B] */
  int32_t* status;               /* host int32[1]: device-detected status of the step (0 = ok) */
  void* arena;                   /* device */
  size_t arena_bytes;
} eagle_host_step;

size_t eagle_tree_verify_step_host_arena(const eagle_host_step* step);
int eagle_tree_verify_step_host(const eagle_host_step* step, eagle_stream_t stream);

/*
 * Bytes one eagle_tree_verify_step_host call with these arguments copies host->device and device->host (host function,
 * no CUDA work; reads the host arrays seq_lens and tree_sizes).  Of k_cache / v_cache only the slots a sequence can see
 * (seq_lens[b] + tree size, clamped to the capacity; none for an empty tree) and of target_probs / draft_probs only the
 * rows of existing nodes are ever read by the kernels, so when that saves more than the extra copy calls cost the step
 * copies exactly those, sequence by sequence (2-D copies), and leaves the rest of the arena as it is; otherwise every
 * tensor is copied whole.  This function reports which of the two the call does.
 */
int eagle_tree_verify_step_host_bytes(const eagle_host_step* step, size_t* h2d_bytes, size_t* d2h_bytes);

/*
 * The same acceptance walk with the distributions given as LOGITS: every row the walk touches is taken as
 * softmax(logits / temperature) without being materialised (the target and draft probability tensors, [B, T_max+1, V]
 * and [B, T_max, V], are never written or read as a whole; only the rows on the walk are swept).  Sec. 4 runs the
 * method at temperature 1 (and at temperature 0, which is the per-sequence `greedy` flag of the descriptor: greedy
 * sequences use the argmax of the logits and ignore `temperature`).
 *
 *   target_logits device fp32 [B, T_max+1, V], draft_logits device fp32 [B, T_max, V]; temperature > 0 (else
 *   EAGLE_ERR_SHAPE); everything else as for eagle_tree_accept.
 *
 * Each row costs one more sweep (its maximum and its mass).  Exponentials are taken in fp32 (2^((z - max) * log2(e) /
 * temperature)), sums and scalars in fp64, so a decision can differ from an fp64 softmax only when it sits within
 * about 1e-6 of its boundary.
 */
int eagle_tree_accept_logits(const eagle_accept_desc* desc, const float* target_logits, const float* draft_logits,
                             const int32_t* draft_tokens, const int32_t* tree_parent, const float* uniforms,
                             float temperature, int32_t* accepted_path, int32_t* bonus_token, eagle_stream_t stream);

#define EAGLE_MAX_CHILDREN 16

typedef struct eagle_expand_desc {
  int32_t batch;               /* B >= 0 (at most 65535) */
  int32_t rows;                /* R >= 0: draft-tree nodes expanded per sequence in this call */
  int32_t vocab;               /* V >= 1 */
  int32_t max_children;        /* K <= EAGLE_MAX_CHILDREN: row stride of the per-child arrays */
  const uint8_t* greedy;       /* device uint8 [B] or NULL (= every sequence stochastic) */
  int32_t* status;             /* device int32 or NULL */
} eagle_expand_desc;

/*
 * Child tokens of draft-tree nodes (App. A.1, tree structure: in the greedy setting the k most probable tokens of a
 * node's draft distribution become its children, otherwise k tokens are sampled; k varies from node to node).
 *
 *   draft_probs  device fp32 [B, R, V]   the draft distribution at each node (used as given, not renormalised)
 *   num_children device int32 [B, R]     k of each node, 0 <= k <= K (greedy: also k <= V)
 *   uniforms     device fp32 [B, R, K]   one uniform in [0, 1) per draw (may be NULL when every sequence is greedy)
 *   child_tokens device int32 [B, R, K]  the k tokens, then -1
 *   child_probs  device fp32 [B, R, K] or NULL   draft_probs at those tokens, then 0
 *
 * Greedy sequences: descending probability, the lower token id first among equal values (exact).  Other sequences: k
 * independent draws (with replacement; the paper does not say), draw j = the smallest x with
 * sum_{v<=x} p(v) > uniforms[j] * sum_v p(v), prefix sums in fp64 (the last token with positive mass if rounding
 * leaves none).  A node whose k is out of range sets *status to EAGLE_ERR_SHAPE and gets no children.
 * One launch, asynchronous on `stream`; no workspace.
 */
int eagle_tree_expand(const eagle_expand_desc* desc, const float* draft_probs, const int32_t* num_children,
                      const float* uniforms, int32_t* child_tokens, float* child_probs, eagle_stream_t stream);

typedef struct eagle_commit_desc {
  int32_t batch;               /* B >= 0 (at most 65535) */
  int32_t num_kv_heads;        /* Hkv >= 0 */
  int32_t head_dim;            /* D: 64 or 128 */
  int32_t kv_capacity;         /* S_cap: slots per (sequence, KV head) of k_cache / v_cache */
  int32_t max_tree;            /* T_max <= 64: tree nodes are numbered 0 .. T_max-1; row count of features_in */
  int32_t path_cap;            /* entries per row of accepted_path */
  int32_t feature_dim;         /* F: elements per feature vector, a multiple of 8; 0 when no features are passed */
  int32_t* status;             /* device int32 or NULL */
} eagle_commit_desc;

/*
 * Commit of the accepted path: what the verification phase leaves behind for the next drafting phase (Sec. 3.3, last
 * sentence: the accepted tokens and their features are recorded).  The paper does not say where anything is stored;
 * with the cache layout of eagle_tree_verify_attn (tree node m at slot L_b + m) it is this:
 *
 *   k_cache, v_cache  device bf16 [B, Hkv, S_cap, D], updated IN PLACE (either may be NULL): for every sequence b with
 *                     accepted nodes path[0..a-1], slot L_b + j <- slot L_b + path[j] for all j < a at once (the
 *                     sources are read before any destination is written); all other slots keep their contents
 *   seq_lens          device int32 [B]          L_b, the committed prefix before the step
 *   accepted_path     device int32 [B, path_cap] node indices from the top of the tree down, then -1 (the output of
 *                                               eagle_tree_accept); entries after the first -1 are ignored
 *   features_in       device bf16 [B, T_max, F] or NULL   one vector per tree node (the target model's features)
 *   features_out      device bf16 [B, path_cap, F] or NULL  row j <- features_in row path[j] for j < a, zeros for j >= a
 *   new_seq_lens      device int32 [B] or NULL  L_b + a  (may alias seq_lens)
 *
 * One call serves one layer's cache; the token of the step's extra draw is not part of the path (its K/V do not
 * exist yet).  A row that is not strictly increasing, leaves [0, T_max), or points at a slot >= S_cap (or L_b < 0)
 * sets *status to EAGLE_ERR_PATH: nothing of that sequence is moved, its length is unchanged and its feature rows are
 * zeros.  All pointers must be 16-byte aligned.  One launch, asynchronous on `stream`; no workspace.
 * A cache of fp8 codes (uint8 [B, Hkv, S_cap, 128], see eagle_tree_verify_attn_fp8) is committed by the same call with
 * head_dim = 64: a row of 128 codes is a row of 64 16-bit elements and rows are moved as bytes (the scales do not change).
 */
int eagle_tree_commit(const eagle_commit_desc* desc, void* k_cache, void* v_cache, const int32_t* seq_lens,
                      const int32_t* accepted_path, const void* features_in, void* features_out,
                      int32_t* new_seq_lens, eagle_stream_t stream);

/*
 * eagle_tree_commit on a paged cache (see eagle_paged_kv): the pages named by kv->k_pages / kv->v_pages are updated IN
 * PLACE although the struct declares them const (either may be NULL).  Rows are copied between, or within, the pages
 * the sequence already owns; no page is allocated, freed or moved.  desc->kv_capacity is ignored (the capacity is
 * max_pages_per_seq * page_size).  A source or destination slot whose block-table entry is outside [0, num_pages)
 * sets *status to EAGLE_ERR_PAGE and the sequence is left alone, as for an invalid path.  Everything else as above.
 */
int eagle_tree_commit_paged(const eagle_commit_desc* desc, const eagle_paged_kv* kv, const int32_t* seq_lens,
                            const int32_t* accepted_path, const void* features_in, void* features_out,
                            int32_t* new_seq_lens, eagle_stream_t stream);

/*
 * Tree-mask builder alone (the mask "tree attention" implies: Sec. 3.1, Sec. 3.3): for every node the bit set
 * of its ancestors and itself, and its depth (top-level nodes: 1).
 *   tree_parent device int32 [B, T_max]; tree_sizes device int32 [B] or NULL;
 *   anc_mask device uint64 [B, T_max]; depth device uint8 [B, T_max] or NULL; status device int32 or NULL.
 * Entries of nodes >= tree size, and of sequences with an invalid tree, are 0.
 */
int eagle_tree_build_mask(const int32_t* tree_parent, const int32_t* tree_sizes, int32_t batch, int32_t max_tree,
                          uint64_t* anc_mask, uint8_t* depth, int32_t* status, eagle_stream_t stream);

/* Human-readable name of a return / status code (host function; never NULL). */
const char* eagle_status_string(int code);

/* Number of kernels this library has launched in this process so far (host counter, for accounting). */
uint64_t eagle_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* EAGLE_VERIFY_H_ */
