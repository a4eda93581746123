// Shared definitions of the tree-verification kernels (device-side plan records, workspace layout).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "eagle_verify.h"

namespace eagle {

constexpr int kMaxTree = EAGLE_MAX_TREE;
constexpr int kBlockM = 128;          // query rows (tree node x head-in-group) per work item
constexpr int kMaxGroup = 16;         // largest GQA group size supported
constexpr int kSlotBudgetAuto = 2048; // partial slots the planner may use when it chooses the splits itself

// One unit of attention work: a 128-row query tile of one (sequence, KV head) over a range of KV tiles.
struct WorkItem {
  int32_t b, g, mt;
  int32_t tile_begin, tile_end;  // KV tiles [begin, end) of `tile_keys` keys each
  int32_t slot;                  // first partial slot, or -1: the only split, write the output directly
  int32_t mode;                  // paired planning only: 0 = one query tile (mt), 1 = two query tiles (mt, mt+1)
  int32_t pad1;
};

struct SeqPlan {
  int32_t item_base;   // first work item of this sequence
  int32_t splits;      // KV splits of every (KV head, row tile) of this sequence
  int32_t n;           // tree size used (0 when the sequence is invalid or empty)
  int32_t L;           // committed prefix length
  int32_t slot_base;   // first partial slot (splits > 1), else -1
  int32_t mtiles;      // 128-row query tiles per KV head
  int32_t ntiles;      // KV tiles covering prefix + tree
  int32_t key;         // KV tiles per work item (sort key of the planner)
};

struct PlanHeader {
  int32_t n_items;
  int32_t next_item;   // work counter of the persistent attention kernel
  int32_t chunk_tiles;
  int32_t n_slots;
  int32_t pad[12];
};

// Workspace carving (all offsets multiples of 256 bytes).
struct Workspace {
  PlanHeader* hdr;
  SeqPlan* seq;        // [B]
  uint64_t* anc;       // [B, T_max]
  WorkItem* items;     // [item_cap]
  float2* part_ml;     // [slot_cap, 128]   (running max in the log2 domain, running sum)
  float* part_o;       // [slot_cap, 128, D] unnormalised partial outputs
  int32_t item_cap, slot_cap;
  size_t bytes;
};

__host__ inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

__host__ inline bool carve_workspace(const eagle_attn_desc& d, void* base, Workspace* w) {
  if (d.batch < 0 || d.num_kv_heads <= 0 || d.num_q_heads <= 0 || d.num_q_heads % d.num_kv_heads) return false;
  const int G = d.num_q_heads / d.num_kv_heads;
  if (G > kMaxGroup || d.max_tree < 0 || d.max_tree > kMaxTree || (d.head_dim != 64 && d.head_dim != 128)) return false;
  if (d.num_splits < 0 || d.num_splits > 1024) return false;
  const long long mtiles = (static_cast<long long>(d.max_tree) * G + kBlockM - 1) / kBlockM;
  const long long units = static_cast<long long>(d.batch) * d.num_kv_heads * (mtiles > 0 ? mtiles : 1);
  // two slots per item leave room for plans that pair query tiles (one slot per query tile of the pair)
  const long long slots = 2 * (d.num_splits > 1 ? units * d.num_splits : (d.num_splits == 1 ? 0 : kSlotBudgetAuto));
  const long long items = units + slots;
  if (items > (1ll << 30)) return false;
  char* p = static_cast<char*>(base);
  size_t off = 0;
  auto take = [&](size_t n) { char* r = p ? p + off : nullptr; off += align256(n); return r; };
  w->hdr = reinterpret_cast<PlanHeader*>(take(sizeof(PlanHeader)));
  w->seq = reinterpret_cast<SeqPlan*>(take(sizeof(SeqPlan) * (size_t)(d.batch > 0 ? d.batch : 1)));
  w->anc = reinterpret_cast<uint64_t*>(take(sizeof(uint64_t) * (size_t)(d.batch > 0 ? d.batch : 1) * (d.max_tree > 0 ? d.max_tree : 1)));
  w->items = reinterpret_cast<WorkItem*>(take(sizeof(WorkItem) * (size_t)(items > 0 ? items : 1)));
  w->part_ml = reinterpret_cast<float2*>(take(sizeof(float2) * (size_t)slots * kBlockM));
  w->part_o = reinterpret_cast<float*>(take(sizeof(float) * (size_t)slots * kBlockM * d.head_dim));
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
  int32_t pair;          // 1: items cover pairs of query tiles and own two consecutive partial slots
  PlanHeader* hdr;
  const SeqPlan* seq;
  const uint64_t* anc;
  const WorkItem* items;
  float2* part_ml;
  float* part_o;
  int32_t* status;
};

struct PlanParams {
  const int32_t* seq_lens;
  const int32_t* tree_sizes;
  const int32_t* tree_parent;
  int32_t B, Hkv, G, T_max, S_cap;
  int32_t tile_keys;       // keys per KV tile of the attention kernel
  int32_t num_ctas;        // CTAs of the persistent attention kernel
  int32_t forced_splits;   // 0: choose
  int32_t min_chunk_tiles;
  int32_t pair;            // 1: one item per pair of query tiles, two partial slots per item
  int32_t item_cap, slot_cap;
  PlanHeader* hdr;
  SeqPlan* seq;
  uint64_t* anc;
  WorkItem* items;
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
};

__device__ inline void report_status(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// Launchers (defined one per .cu file).
cudaError_t launch_plan(const PlanParams& p, cudaStream_t stream);
cudaError_t launch_build_mask(const int32_t* tree_parent, const int32_t* tree_sizes, int batch, int max_tree,
                              uint64_t* anc, uint8_t* depth, int32_t* status, cudaStream_t stream);
cudaError_t launch_attn_mma(const AttnParams& p, int num_ctas, cudaStream_t stream);
int attn_mma_tile_keys();
int attn_mma_ctas_per_sm(int head_dim);
cudaError_t attn_mma_prepare(int head_dim);
cudaError_t launch_attn_tc(const AttnParams& p, int num_ctas, cudaStream_t stream);
int attn_tc_tile_keys();
cudaError_t attn_tc_prepare(int head_dim);
cudaError_t launch_attn_tc2(const AttnParams& p, int num_ctas, cudaStream_t stream);
int attn_tc2_tile_keys();
cudaError_t attn_tc2_prepare(int head_dim);
cudaError_t launch_combine(const AttnParams& p, const int32_t* tree_sizes_unused, cudaStream_t stream);

cudaError_t launch_accept(const AcceptParams& p, int sm_count, cudaStream_t stream);

void count_launch();

}  // namespace eagle
