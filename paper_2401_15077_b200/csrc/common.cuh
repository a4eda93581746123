// Shared definitions of the tree-verification kernels (device-side plan records, workspace layout).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "eagle_verify.h"

namespace eagle {

constexpr int kMaxTree = EAGLE_MAX_TREE;
constexpr int kBlockM = 128;          // query rows (tree node x head-in-group) per work unit
constexpr int kMaxGroup = 16;         // largest GQA group size supported
constexpr int kMaxPlanCtas = 256;     // upper bound on the CTAs of the persistent attention kernel (one per SM)

// A work unit is one 128-row query tile of one (sequence, KV head); its work is the sequence's KV tiles.  The
// planner groups query tiles in pairs (super-units), lays the super-units end to end and gives every pair of CTAs
// (a team) an equal contiguous share; see plan.cu.  A work item is what one CTA does for one team piece.
struct WorkItem {
  int32_t b, g, mt;
  int32_t tile_begin, tile_end;  // KV tiles [begin, end) of `tile_keys` keys each
  int32_t slot;                  // partial slot, or -1: the unit is in one piece, write the output directly
  int32_t pad0, pad1;
};

struct SeqPlan {
  int32_t n;           // tree size used (0 when the sequence is invalid or empty)
  int32_t L;           // committed prefix length
  int32_t mtiles;      // 128-row query tiles per KV head
  int32_t ntiles;      // KV tiles covering prefix + tree
  int32_t unit_base;   // index of this sequence's first super-unit; super-unit = unit_base + g * ceil(mtiles/2) + mt/2
  int32_t pad0;
  long long start;     // position of the first super-unit on the work line
};

struct UnitPlan {        // one per super-unit
  int32_t first_item;  // its team pieces are first_item .. first_item + n_pieces - 1; piece tp owns items 2*tp and 2*tp+1
  int32_t n_pieces;
  int32_t slot_base;   // first partial slot when its query tiles end up in several items, else -1
  int32_t pad0;        // its sequence
};

// A query tile whose output has to be merged from several items' partials: everything the combine kernel needs, so
// that it reads one record instead of walking unit -> item -> sequence.  The tile's pieces are the items
// item0 + k * item_stride and the partial slots slot0 + k, k < count (an empty item's slot holds nothing).
struct CutTile {
  int32_t b, g, mt;
  int32_t m_valid;     // query rows of the (sequence, KV head) that belong to tree nodes: tree size x group size
  int32_t item0, item_stride;
  int32_t slot0, count;
};

struct PlanHeader {
  int32_t n_items;
  int32_t n_slots;
  int32_t n_units;
  int32_t ctas_used;
  long long total_tiles;
  int32_t n_cut;       // query tiles whose output has to be merged from several pieces
  int32_t pad[9];
};

// Workspace carving (all offsets multiples of 256 bytes).
struct Workspace {
  PlanHeader* hdr;
  SeqPlan* seq;        // [B]
  uint64_t* anc;       // [B, T_max]
  UnitPlan* units;     // [unit_cap]
  CutTile* cut_tiles;  // [2 * unit_cap]: the cut query tiles, in no particular order
  int32_t* cta_first;  // [kMaxPlanCtas + 1]: team j owns the team pieces cta_first[j] .. cta_first[j+1] - 1
  WorkItem* items;     // [item_cap]
  float2* part_ml;     // [slot_cap, 128]   (reference max in the log2 domain, row sum)
  float* part_o;       // [slot_cap, 128, D] unnormalised partial outputs
  int32_t unit_cap, item_cap, slot_cap;
  size_t bytes;
};

__host__ inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

// `num_ctas` bounds the CTAs of the attention kernel the plan may be made for (the library-wide bound by default; the
// fixed-array entry point passes the current device's count so that common shapes fit its array).
__host__ inline bool carve_workspace(const eagle_attn_desc& d, void* base, Workspace* w, int num_ctas = kMaxPlanCtas) {
  if (d.batch < 0 || d.num_kv_heads <= 0 || d.num_q_heads <= 0 || d.num_q_heads % d.num_kv_heads) return false;
  const int G = d.num_q_heads / d.num_kv_heads;
  if (G > kMaxGroup || d.max_tree < 0 || d.max_tree > kMaxTree || (d.head_dim != 64 && d.head_dim != 128)) return false;
  if (d.num_splits < 0 || d.num_splits > 1024) return false;
  const long long mtiles = (static_cast<long long>(d.max_tree) * G + kBlockM - 1) / kBlockM;
  const long long units = static_cast<long long>(d.batch) * d.num_kv_heads * (mtiles > 0 ? (mtiles + 1) / 2 : 1);   // super-units
  // team pieces: one per super-unit plus at most one per share boundary (or num_splits per super-unit when forced);
  // two items per team piece
  const long long teams = num_ctas / 2;
  const long long pieces = d.num_splits > 0 ? units * d.num_splits : units + teams;
  const long long items = 2 * pieces;
  // Partial slots: one per item when the split is forced.  With equal shares only cut super-units and lone tiles take
  // slots, two per piece: a share boundary cuts at most one super-unit, so the cut pairs and twins hold at most
  // 2 * (cuts + cut units) <= 4 * (teams - 1) slots, and a lone tile (one per sequence, only with an odd number of
  // KV heads) holds 2 * (its cuts + 1).
  long long slots = items;
  if (d.num_splits == 0) {
    const long long bound = 4 * teams + 2ll * d.batch * (d.num_kv_heads & 1);
    if (bound < slots) slots = bound;
  }
  if (items > (1ll << 30)) return false;
  char* p = static_cast<char*>(base);
  size_t off = 0;
  auto take = [&](size_t n) { char* r = p ? p + off : nullptr; off += align256(n); return r; };
  w->hdr = reinterpret_cast<PlanHeader*>(take(sizeof(PlanHeader)));
  w->seq = reinterpret_cast<SeqPlan*>(take(sizeof(SeqPlan) * (size_t)(d.batch > 0 ? d.batch : 1)));
  w->anc = reinterpret_cast<uint64_t*>(take(sizeof(uint64_t) * (size_t)(d.batch > 0 ? d.batch : 1) * (d.max_tree > 0 ? d.max_tree : 1)));
  w->units = reinterpret_cast<UnitPlan*>(take(sizeof(UnitPlan) * (size_t)(units > 0 ? units : 1)));
  w->cut_tiles = reinterpret_cast<CutTile*>(take(sizeof(CutTile) * 2 * (size_t)(units > 0 ? units : 1)));
  w->cta_first = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * (kMaxPlanCtas + 1)));
  w->items = reinterpret_cast<WorkItem*>(take(sizeof(WorkItem) * (size_t)(items > 0 ? items : 1)));
  w->part_ml = reinterpret_cast<float2*>(take(sizeof(float2) * (size_t)slots * kBlockM));
  w->part_o = reinterpret_cast<float*>(take(sizeof(float) * (size_t)slots * kBlockM * d.head_dim));
  w->unit_cap = static_cast<int32_t>(units);
  w->item_cap = static_cast<int32_t>(items);
  w->slot_cap = static_cast<int32_t>(slots);
  w->bytes = off;
  return true;
}

struct AttnParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  __nv_bfloat16* out;
  int32_t B, Hq, Hkv, G, D, T_max, S_cap;
  float scale_log2;      // sm_scale * log2(e)
  int32_t q_tma;         // set by the launcher: query tiles are fetched with TMA (group size divides 128)
  const PlanHeader* hdr;
  const SeqPlan* seq;
  const uint64_t* anc;
  const UnitPlan* units;
  const CutTile* cut_tiles;
  const int32_t* cta_first;
  const WorkItem* items;
  float2* part_ml;
  float* part_o;
  int32_t* status;
  // paged cache (page_size > 0): k / v are [num_pages, Hkv, page_size, D], slot j of sequence b is row j % page_size of
  // page block_table[b * max_pages + j / page_size]; page_size is a power of two
  const int32_t* block_table;
  int32_t page_size, page_shift, max_pages, num_pages;
  // cache stored as fp8 (e4m3) codes: k / v point to uint8 [B, Hkv, S_cap, D] and every (sequence, KV head) has one scale
  // for its keys and one for its values, fp32 [B, Hkv] (null: the cache is bf16)
  const float* k_scale;
  const float* v_scale;
  unsigned long long wait_limit_ns;   // a wait that makes no progress for this long aborts the CTA (EAGLE_ERR_TIMEOUT)
  int32_t stall_after_tiles;          // test hook: the K/V producer stops issuing after this many tiles (negative: off)
};

struct PlanParams {
  const int32_t* seq_lens;
  const int32_t* tree_sizes;
  const int32_t* tree_parent;
  int32_t B, Hkv, G, T_max, S_cap;
  int32_t tile_keys;       // keys per KV tile of the attention kernel
  int32_t num_ctas;        // CTAs of the persistent attention kernel (<= kMaxPlanCtas)
  int32_t forced_splits;   // 0: equal shares; s > 0: every unit in min(s, KV tiles) equal pieces
  int32_t snap_tiles;      // a share boundary closer than this to a unit's edge moves to the edge
  int32_t item_overhead_tiles;   // fixed cost of starting a unit, in KV-tile equivalents
  int32_t unit_cap, item_cap, slot_cap;
  PlanHeader* hdr;
  SeqPlan* seq;
  uint64_t* anc;
  UnitPlan* units;
  CutTile* cut_tiles;
  int32_t* cta_first;
  WorkItem* items;
  int32_t* status;
  const int32_t* block_table;   // paged cache: [B, max_pages] (null: contiguous cache)
  int32_t page_size, max_pages, num_pages;
  int32_t shared_tree;          // tree_parent is [T_max] and tree_sizes [1] (or null): one tree for every sequence
};

struct CommitParams {
  __nv_bfloat16* k;          // [B, Hkv, S_cap, D], in place (may be null)
  __nv_bfloat16* v;
  const int32_t* seq_lens;   // [B]
  const int32_t* path;       // [B, path_cap], -1 padded
  const __nv_bfloat16* features_in;   // [B, T_max, F] or null
  __nv_bfloat16* features_out;        // [B, path_cap, F] or null
  int32_t* new_seq_lens;     // [B] or null
  int32_t B, Hkv, D, S_cap, T_max, path_cap, F;
  int32_t* status;
  const int32_t* block_table;   // paged cache: k / v are [num_pages, Hkv, page_size, D]; null: contiguous
  int32_t page_size, max_pages, num_pages;
};

constexpr int kMaxChildren = 16;

struct ExpandParams {
  const float* probs;          // [B, R, V]
  const int32_t* num_children; // [B, R]
  const uint8_t* greedy;       // [B] or null
  const float* uniforms;       // [B, R, K] or null
  int32_t* tokens;             // [B, R, K]
  float* token_probs;          // [B, R, K] or null
  int32_t B, R, V, K;
  int32_t* status;
};

struct AcceptParams {
  const float* target;   // [B, T+1, V]
  const float* draft;    // [B, T, V]
  const int32_t* tokens; // [B, T]
  const int32_t* parent; // [B, T]
  const float* uniforms; // [B, T+1]
  const int32_t* tree_sizes;
  const uint8_t* greedy;
  int32_t* path;         // [B, path_cap]
  int32_t* bonus;        // [B]
  int32_t* accept_len;   // [B] or null
  int32_t* status;
  int32_t B, T, V, path_cap;
  int32_t logits;        // target / draft hold logits: rows are softmax(logits / temperature)
  float inv_temp_log2;   // log2(e) / temperature
  int32_t shared_tree;   // parent is [T] and tree_sizes [1] (or null): one tree for every sequence
};

__device__ inline void report_status(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// Launchers (defined one per .cu file).
cudaError_t launch_plan(const PlanParams& p, cudaStream_t stream);
cudaError_t launch_build_mask(const int32_t* tree_parent, const int32_t* tree_sizes, int batch, int max_tree,
                              uint64_t* anc, uint8_t* depth, int32_t* status, cudaStream_t stream);
cudaError_t launch_attn(const AttnParams& p, int num_ctas, cudaStream_t stream);
int attn_tile_keys();
cudaError_t attn_prepare(int head_dim);
cudaError_t launch_combine(const AttnParams& p, int unit_cap, int sm_count, cudaStream_t stream);
cudaError_t launch_accept(const AcceptParams& p, int sm_count, cudaStream_t stream);
int accept_cluster_width(int batch, int vocab, int sm_count, bool all_greedy = false);   // 0: a warp per tree; else CTAs per cluster

cudaError_t launch_commit(const CommitParams& p, cudaStream_t stream);
cudaError_t launch_expand(const ExpandParams& p, int sm_count, cudaStream_t stream);
void count_launch();

}  // namespace eagle
