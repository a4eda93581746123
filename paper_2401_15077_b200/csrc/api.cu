// C ABI of the tree-verification library: argument checks, workspace carving and kernel launches.
// Nothing here allocates or synchronises; every launch goes to the caller's stream.
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace eagle {

namespace {

// Planner cost model, in KV-tile positions: what starting an item costs the attention kernel (pipeline fill, output
// write), and how close to a super-unit's edge a share boundary snaps to the edge.
#ifndef EAGLE_ITEM_OVERHEAD
#define EAGLE_ITEM_OVERHEAD 6
#endif
#ifndef EAGLE_SNAP_TILES
#define EAGLE_SNAP_TILES 2
#endif
constexpr int kPlanItemOverheadTiles = EAGLE_ITEM_OVERHEAD;
constexpr int kPlanSnapTiles = EAGLE_SNAP_TILES;

std::atomic<uint64_t> g_launches{0};
// How long a wait inside the attention kernel may last before the kernel gives up (EAGLE_ERR_TIMEOUT), and the
// fault-injection hook of the time-out test: the K/V producer issues no copy after this many tiles (negative: off).
constexpr uint64_t kDefaultWaitLimitNs = 2000000000ull;
std::atomic<uint64_t> g_wait_limit_ns{kDefaultWaitLimitNs};
std::atomic<int32_t> g_stall_after_tiles{-1};

struct DeviceInfo {
  bool ready = false;
  int sm_count = 0;
  int cc_major = 0;
  bool attn_prepared[2] = {false, false};
};
constexpr int kMaxDevices = 64;
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;

// Per-device facts, queried once.  Returns nullptr if the current device is unusable.
DeviceInfo* device_info(int* err) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    *err = EAGLE_ERR_DEVICE;
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  DeviceInfo& d = g_dev[dev];
  if (!d.ready) {
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || d.sm_count <= 0) {
      *err = EAGLE_ERR_DEVICE;
      return nullptr;
    }
    d.ready = true;
  }
  if (d.cc_major != 10) {
    *err = EAGLE_ERR_DEVICE;
    return nullptr;
  }
  return &d;
}

}  // namespace

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

}  // namespace eagle

using namespace eagle;

extern "C" {

size_t eagle_tree_verify_attn_workspace(const eagle_attn_desc* desc) {
  if (!desc) return 0;
  Workspace w;
  if (!carve_workspace(*desc, nullptr, &w)) return 0;
  return w.bytes;
}

namespace {

// Where the keys and values of an attention call live: a contiguous cache, or pages behind a block table.
struct KvSource {
  const void* k;
  const void* v;
  int64_t capacity;             // slots per sequence
  const int32_t* block_table;   // null: contiguous
  int32_t num_pages, page_size, max_pages;
  const float* k_scale = nullptr;   // non-null: k / v hold fp8 (e4m3) codes with these scales per (sequence, KV head)
  const float* v_scale = nullptr;
};

// The planner launch: tree masks and work list into the workspace.  Depends on the lengths, the trees and the shape
// only, so one plan serves every layer of a verification pass.
int plan_call(const eagle_attn_desc& d, const Workspace& w, int num_ctas, const KvSource& kv, const int32_t* seq_lens,
              const int32_t* tree_parent, cudaStream_t stream) {
  if (!seq_lens || !tree_parent) return EAGLE_ERR_NULL;
  PlanParams pp;
  pp.seq_lens = seq_lens;
  pp.tree_sizes = d.tree_sizes;
  pp.tree_parent = tree_parent;
  pp.B = d.batch;
  pp.Hkv = d.num_kv_heads;
  pp.G = d.num_q_heads / d.num_kv_heads;
  pp.T_max = d.max_tree;
  pp.S_cap = static_cast<int32_t>(kv.capacity < 0x7fffffff ? kv.capacity : 0x7fffffff);
  pp.tile_keys = attn_tile_keys();
  pp.num_ctas = num_ctas;
  pp.forced_splits = d.num_splits;
  pp.snap_tiles = kPlanSnapTiles;
  pp.item_overhead_tiles = kPlanItemOverheadTiles;
  pp.unit_cap = w.unit_cap;
  pp.item_cap = w.item_cap;
  pp.slot_cap = w.slot_cap;
  pp.hdr = w.hdr;
  pp.seq = w.seq;
  pp.anc = w.anc;
  pp.units = w.units;
  pp.cut_tiles = w.cut_tiles;
  pp.cta_first = w.cta_first;
  pp.items = w.items;
  pp.status = d.status;
  pp.block_table = kv.block_table;
  pp.page_size = kv.page_size;
  pp.max_pages = kv.max_pages;
  pp.num_pages = kv.num_pages;
  pp.shared_tree = d.shared_tree != 0;
  // Nothing in the workspace has to start at zero: the planner rebuilds every table it or the later kernels read, and
  // a partial slot is always written by the attention kernel before the combine kernel reads it.
  if (launch_plan(pp, stream) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  return EAGLE_OK;
}

// The attention and combine launches over a plan that is already in the workspace.
int attend_call(const eagle_attn_desc& d, const Workspace& w, int num_ctas, DeviceInfo* dev, const void* q, const KvSource& kv,
                void* out, cudaStream_t stream) {
  if (!q || !kv.k || !kv.v || !out) return EAGLE_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(kv.k) & 15) || (reinterpret_cast<uintptr_t>(kv.v) & 15) || (reinterpret_cast<uintptr_t>(q) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 31))
    return EAGLE_ERR_SHAPE;
  const int di = d.head_dim == 128 ? 1 : 0;
  if (!dev->attn_prepared[di]) {
    if (attn_prepare(d.head_dim) != cudaSuccess) return EAGLE_ERR_DEVICE;
    dev->attn_prepared[di] = true;
  }
  AttnParams ap;
  ap.q = static_cast<const __nv_bfloat16*>(q);
  ap.k = static_cast<const __nv_bfloat16*>(kv.k);
  ap.v = static_cast<const __nv_bfloat16*>(kv.v);
  ap.out = static_cast<__nv_bfloat16*>(out);
  ap.B = d.batch;
  ap.Hq = d.num_q_heads;
  ap.Hkv = d.num_kv_heads;
  ap.G = d.num_q_heads / d.num_kv_heads;
  ap.D = d.head_dim;
  ap.T_max = d.max_tree;
  ap.S_cap = static_cast<int32_t>(kv.capacity < 0x7fffffff ? kv.capacity : 0x7fffffff);
  const float scale = d.sm_scale != 0.f ? d.sm_scale : 1.0f / std::sqrt(static_cast<float>(d.head_dim));
  ap.scale_log2 = scale * 1.4426950408889634f;
  ap.q_tma = 0;
  ap.hdr = w.hdr;
  ap.seq = w.seq;
  ap.anc = w.anc;
  ap.units = w.units;
  ap.cut_tiles = w.cut_tiles;
  ap.cta_first = w.cta_first;
  ap.items = w.items;
  ap.part_ml = w.part_ml;
  ap.part_o = w.part_o;
  ap.status = d.status;
  ap.block_table = kv.block_table;
  ap.page_size = kv.block_table ? kv.page_size : 0;
  ap.page_shift = 0;
  while (kv.block_table && (1 << ap.page_shift) < kv.page_size) ++ap.page_shift;
  ap.max_pages = kv.max_pages;
  ap.num_pages = kv.num_pages;
  ap.k_scale = kv.k_scale;
  ap.v_scale = kv.v_scale;
  ap.wait_limit_ns = g_wait_limit_ns.load(std::memory_order_relaxed);
  ap.stall_after_tiles = g_stall_after_tiles.load(std::memory_order_relaxed);
  if (d.ev_attn_begin && cudaEventRecord(static_cast<cudaEvent_t>(d.ev_attn_begin), stream) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  if (launch_attn(ap, num_ctas, stream) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  if (d.ev_attn_end && cudaEventRecord(static_cast<cudaEvent_t>(d.ev_attn_end), stream) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  if (launch_combine(ap, w.unit_cap, dev->sm_count, stream) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  return EAGLE_OK;
}

// Which of the two halves of an attention call an entry point runs.
enum AttnPhase { kPlanOnly = 1, kAttendOnly = 2, kPlanAndAttend = 3 };

// Entry with a caller-provided workspace, for either kind of cache.
int attention_with_workspace(const eagle_attn_desc* desc, int phase, const void* q, const KvSource& kv, const int32_t* seq_lens,
                             const int32_t* tree_parent, void* out, eagle_stream_t stream_) {
  const eagle_attn_desc& d = *desc;
  Workspace w;
  if (kv.capacity < 0 || !(d.sm_scale >= 0.f) || !carve_workspace(d, d.workspace, &w)) return EAGLE_ERR_SHAPE;
  if (d.batch == 0 || d.max_tree == 0) return EAGLE_OK;
  if ((phase & kPlanOnly) && (!seq_lens || !tree_parent)) return EAGLE_ERR_NULL;
  if ((phase & kAttendOnly) && (!q || !kv.k || !kv.v || !out)) return EAGLE_ERR_NULL;
  if (!d.workspace || (reinterpret_cast<uintptr_t>(d.workspace) & 255) || d.workspace_bytes < w.bytes) return EAGLE_ERR_WORKSPACE;
  if ((phase & kAttendOnly) &&
      ((reinterpret_cast<uintptr_t>(kv.k) & 15) || (reinterpret_cast<uintptr_t>(kv.v) & 15) || (reinterpret_cast<uintptr_t>(q) & 15) ||
       (reinterpret_cast<uintptr_t>(out) & 31)))
    return EAGLE_ERR_SHAPE;
  int err = 0;
  DeviceInfo* dev = device_info(&err);
  if (!dev) return err;
  const int num_ctas = (dev->sm_count < kMaxPlanCtas ? dev->sm_count : kMaxPlanCtas) & ~1;   // one persistent CTA per SM, in pairs
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (phase & kPlanOnly) {
    const int rc = plan_call(d, w, num_ctas, kv, seq_lens, tree_parent, stream);
    if (rc != EAGLE_OK) return rc;
  }
  if (phase & kAttendOnly) return attend_call(d, w, num_ctas, dev, q, kv, out, stream);
  return EAGLE_OK;
}

bool paged_source(const eagle_attn_desc* desc, const eagle_paged_kv* pk, KvSource* kv, int* rc) {
  if (!desc || !pk) { *rc = EAGLE_ERR_NULL; return false; }
  if (pk->num_pages < 1 || pk->page_size < 16 || (pk->page_size & (pk->page_size - 1)) || pk->max_pages_per_seq < 0) { *rc = EAGLE_ERR_SHAPE; return false; }
  if (static_cast<int64_t>(pk->num_pages) * desc->num_kv_heads > 0x7fffffffll) { *rc = EAGLE_ERR_SHAPE; return false; }
  if (desc->batch > 0 && desc->max_tree > 0 && !pk->block_table) { *rc = EAGLE_ERR_NULL; return false; }
  *kv = {pk->k_pages, pk->v_pages, static_cast<int64_t>(pk->max_pages_per_seq) * pk->page_size, pk->block_table,
         pk->num_pages, pk->page_size, pk->max_pages_per_seq};
  return true;
}

}  // namespace

int eagle_tree_verify_attn(const eagle_attn_desc* desc, const void* q, const void* k_cache, const void* v_cache,
                           const int32_t* seq_lens, const int32_t* tree_parent, void* out, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  const KvSource kv = {k_cache, v_cache, desc->kv_capacity, nullptr, 0, 0, 0};
  return attention_with_workspace(desc, kPlanAndAttend, q, kv, seq_lens, tree_parent, out, stream_);
}

int eagle_tree_verify_attn_paged(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* pk, const int32_t* seq_lens,
                                 const int32_t* tree_parent, void* out, eagle_stream_t stream_) {
  KvSource kv;
  int rc = EAGLE_OK;
  if (!paged_source(desc, pk, &kv, &rc)) return rc;
  return attention_with_workspace(desc, kPlanAndAttend, q, kv, seq_lens, tree_parent, out, stream_);
}

int eagle_tree_verify_attn_fp8(const eagle_attn_desc* desc, const void* q, const void* k_codes, const void* v_codes,
                               const float* k_scale, const float* v_scale, const int32_t* seq_lens, const int32_t* tree_parent,
                               void* out, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  if (desc->head_dim != 128) return EAGLE_ERR_SHAPE;
  if (desc->batch > 0 && desc->max_tree > 0 && (!k_scale || !v_scale)) return EAGLE_ERR_NULL;
  KvSource kv = {k_codes, v_codes, desc->kv_capacity, nullptr, 0, 0, 0};
  kv.k_scale = k_scale;
  kv.v_scale = v_scale;
  return attention_with_workspace(desc, kPlanAndAttend, q, kv, seq_lens, tree_parent, out, stream_);
}

int eagle_tree_verify_attn_planned_fp8(const eagle_attn_desc* desc, const void* q, const void* k_codes, const void* v_codes,
                                       const float* k_scale, const float* v_scale, void* out, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  if (desc->head_dim != 128) return EAGLE_ERR_SHAPE;
  if (desc->batch > 0 && desc->max_tree > 0 && (!k_scale || !v_scale)) return EAGLE_ERR_NULL;
  KvSource kv = {k_codes, v_codes, desc->kv_capacity, nullptr, 0, 0, 0};
  kv.k_scale = k_scale;
  kv.v_scale = v_scale;
  return attention_with_workspace(desc, kAttendOnly, q, kv, nullptr, nullptr, out, stream_);
}

int eagle_tree_verify_attn_paged_fp8(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* pk, const float* k_scale,
                                     const float* v_scale, const int32_t* seq_lens, const int32_t* tree_parent, void* out,
                                     eagle_stream_t stream_) {
  KvSource kv;
  int rc = EAGLE_OK;
  if (!paged_source(desc, pk, &kv, &rc)) return rc;
  if (desc->head_dim != 128) return EAGLE_ERR_SHAPE;
  if (desc->batch > 0 && desc->max_tree > 0 && (!k_scale || !v_scale)) return EAGLE_ERR_NULL;
  kv.k_scale = k_scale;
  kv.v_scale = v_scale;
  return attention_with_workspace(desc, kPlanAndAttend, q, kv, seq_lens, tree_parent, out, stream_);
}

int eagle_tree_verify_attn_planned_paged_fp8(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* pk,
                                             const float* k_scale, const float* v_scale, void* out, eagle_stream_t stream_) {
  KvSource kv;
  int rc = EAGLE_OK;
  if (!paged_source(desc, pk, &kv, &rc)) return rc;
  if (desc->head_dim != 128) return EAGLE_ERR_SHAPE;
  if (desc->batch > 0 && desc->max_tree > 0 && (!k_scale || !v_scale)) return EAGLE_ERR_NULL;
  kv.k_scale = k_scale;
  kv.v_scale = v_scale;
  return attention_with_workspace(desc, kAttendOnly, q, kv, nullptr, nullptr, out, stream_);
}

int eagle_tree_verify_plan(const eagle_attn_desc* desc, const int32_t* seq_lens, const int32_t* tree_parent,
                           const eagle_paged_kv* pk, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  KvSource kv = {nullptr, nullptr, desc->kv_capacity, nullptr, 0, 0, 0};
  int rc = EAGLE_OK;
  if (pk && !paged_source(desc, pk, &kv, &rc)) return rc;
  return attention_with_workspace(desc, kPlanOnly, nullptr, kv, seq_lens, tree_parent, nullptr, stream_);
}

int eagle_tree_verify_attn_planned(const eagle_attn_desc* desc, const void* q, const void* k_cache, const void* v_cache,
                                   void* out, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  const KvSource kv = {k_cache, v_cache, desc->kv_capacity, nullptr, 0, 0, 0};
  return attention_with_workspace(desc, kAttendOnly, q, kv, nullptr, nullptr, out, stream_);
}

int eagle_tree_verify_attn_planned_paged(const eagle_attn_desc* desc, const void* q, const eagle_paged_kv* pk, void* out,
                                         eagle_stream_t stream_) {
  KvSource kv;
  int rc = EAGLE_OK;
  if (!paged_source(desc, pk, &kv, &rc)) return rc;
  return attention_with_workspace(desc, kAttendOnly, q, kv, nullptr, nullptr, out, stream_);
}

const uint64_t* eagle_tree_verify_plan_masks(const eagle_attn_desc* desc) {
  Workspace w;
  if (!desc || !desc->workspace || !carve_workspace(*desc, desc->workspace, &w)) return nullptr;
  return w.anc;
}

void eagle_set_wait_limit_ns(uint64_t ns) { g_wait_limit_ns.store(ns ? ns : kDefaultWaitLimitNs, std::memory_order_relaxed); }

void eagle_test_stall_kv_producer(int32_t after_tiles) { g_stall_after_tiles.store(after_tiles, std::memory_order_relaxed); }

namespace {

// Shared by the two acceptance entry points: `temperature` < 0 means the rows are probabilities.
int accept_call(const eagle_accept_desc* desc, const float* target, const float* draft, const int32_t* draft_tokens,
                const int32_t* tree_parent, const float* uniforms, float temperature, int32_t* accepted_path,
                int32_t* bonus_token, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  const eagle_accept_desc& d = *desc;
  if (d.batch < 0 || d.max_tree < 0 || d.max_tree > kMaxTree || d.vocab < 1 || d.path_cap < 0) return EAGLE_ERR_SHAPE;
  if (d.batch == 0) return EAGLE_OK;
  if (!target || !draft_tokens || !tree_parent || !accepted_path || !bonus_token) return EAGLE_ERR_NULL;
  // stochastic sequences need the draft rows and the uniforms; only an all-greedy call may omit them
  if ((!draft || !uniforms) && !d.greedy) return EAGLE_ERR_NULL;
  int err = 0;
  DeviceInfo* dev = device_info(&err);
  if (!dev) return err;
  AcceptParams ap;
  ap.target = target;
  ap.draft = draft;
  ap.tokens = draft_tokens;
  ap.parent = tree_parent;
  ap.uniforms = uniforms;
  ap.tree_sizes = d.tree_sizes;
  ap.greedy = d.greedy;
  ap.path = accepted_path;
  ap.bonus = bonus_token;
  ap.accept_len = d.accept_len;
  ap.status = d.status;
  ap.B = d.batch;
  ap.T = d.max_tree;
  ap.V = d.vocab;
  ap.path_cap = d.path_cap;
  ap.logits = temperature >= 0.f ? 1 : 0;
  ap.inv_temp_log2 = temperature > 0.f ? 1.4426950408889634f / temperature : 0.f;
  ap.shared_tree = d.shared_tree != 0;
  if (launch_accept(ap, dev->sm_count, static_cast<cudaStream_t>(stream_)) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  return EAGLE_OK;
}

}  // namespace

int eagle_tree_accept(const eagle_accept_desc* desc, const float* target_probs, const float* draft_probs,
                      const int32_t* draft_tokens, const int32_t* tree_parent, const float* uniforms,
                      int32_t* accepted_path, int32_t* bonus_token, eagle_stream_t stream_) {
  return accept_call(desc, target_probs, draft_probs, draft_tokens, tree_parent, uniforms, -1.f, accepted_path, bonus_token, stream_);
}

int eagle_tree_accept_logits(const eagle_accept_desc* desc, const float* target_logits, const float* draft_logits,
                             const int32_t* draft_tokens, const int32_t* tree_parent, const float* uniforms,
                             float temperature, int32_t* accepted_path, int32_t* bonus_token, eagle_stream_t stream_) {
  if (!(temperature > 0.f) || !(temperature < 3.0e38f)) return EAGLE_ERR_SHAPE;
  return accept_call(desc, target_logits, draft_logits, draft_tokens, tree_parent, uniforms, temperature, accepted_path, bonus_token,
                     stream_);
}

int eagle_tree_accept_cluster_width(int32_t batch, int32_t vocab) {
  if (batch < 0 || vocab < 1) return EAGLE_ERR_SHAPE;
  int err = 0;
  DeviceInfo* dev = device_info(&err);
  if (!dev) return err;
  return accept_cluster_width(batch, vocab, dev->sm_count);
}

int eagle_tree_accept_cluster_width_greedy(int32_t batch, int32_t vocab) {
  if (batch < 0 || vocab < 1) return EAGLE_ERR_SHAPE;
  int err = 0;
  DeviceInfo* dev = device_info(&err);
  if (!dev) return err;
  return accept_cluster_width(batch, vocab, dev->sm_count, true);
}

int eagle_tree_build_mask(const int32_t* tree_parent, const int32_t* tree_sizes, int32_t batch, int32_t max_tree,
                          uint64_t* anc_mask, uint8_t* depth, int32_t* status, eagle_stream_t stream_) {
  if (batch < 0 || max_tree < 0 || max_tree > kMaxTree) return EAGLE_ERR_SHAPE;
  if (batch == 0 || max_tree == 0) return EAGLE_OK;
  if (!tree_parent || !anc_mask) return EAGLE_ERR_NULL;
  int err = 0;
  if (!device_info(&err)) return err;
  if (launch_build_mask(tree_parent, tree_sizes, batch, max_tree, anc_mask, depth, status,
                        static_cast<cudaStream_t>(stream_)) != cudaSuccess)
    return EAGLE_ERR_LAUNCH;
  return EAGLE_OK;
}

// ---------------------------------------------------------------------------------------------------------
// Attention without a caller-provided workspace.
//
// Some hosts of this library can hand over device pointers for tensors but have no way to get device scratch
// at call time: an inference-server backend whose memory pool is frozen after start-up, a plug-in that runs
// inside another engine's execution context, a latency-critical decode loop in which cudaMalloc (which
// synchronises the whole device) is off limits.  For them the planner tables and split partials live in the
// fixed array below, which every GPU that loads the library keeps until the process exits.
constexpr size_t kStaticScratchBytes = 24u << 20;   // 24 MiB
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

// Device address of the fixed scratch array on the current device.  The array's name is only a host-side handle:
// the address a kernel can use comes from cudaGetSymbolAddress, asked once per device with that device current.
void* g_static_ptr[kMaxDevices] = {nullptr};
std::mutex g_static_mutex;

void* static_scratch_ptr() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) return nullptr;
    g_static_ptr[dev] = ptr;
  }
  return g_static_ptr[dev];
}

}  // namespace

size_t eagle_tree_verify_attn_static_capacity(void) { return kStaticScratchBytes; }

int eagle_tree_verify_attn_static(const eagle_attn_desc* desc, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* seq_lens, const int32_t* tree_parent, void* out, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  const eagle_attn_desc& d = *desc;
  if (d.kv_capacity < 0 || !(d.sm_scale >= 0.f)) return EAGLE_ERR_SHAPE;
  int err = 0;
  DeviceInfo* dev = device_info(&err);
  if (!dev) return err;
  const int num_ctas = (dev->sm_count < kMaxPlanCtas ? dev->sm_count : kMaxPlanCtas) & ~1;
  void* scratch = static_scratch_ptr();
  if (!scratch) return EAGLE_ERR_DEVICE;
  // carved for the CTAs this device really runs (one per SM) instead of the library-wide bound, so that common shapes fit
  Workspace w;
  if (!carve_workspace(d, scratch, &w, num_ctas)) return EAGLE_ERR_SHAPE;
  if (w.bytes > kStaticScratchBytes) return EAGLE_ERR_WORKSPACE;   // this shape needs more than the fixed array holds
  if (d.batch == 0 || d.max_tree == 0) return EAGLE_OK;
  const KvSource kv = {k_cache, v_cache, d.kv_capacity, nullptr, 0, 0, 0};
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int rc = plan_call(d, w, num_ctas, kv, seq_lens, tree_parent, stream);
  if (rc != EAGLE_OK) return rc;
  return attend_call(d, w, num_ctas, dev, q, kv, out, stream);
}

// ---------------------------------------------------------------------------------------------------------
// One step from host buffers: copies in, the two device calls, copies out; everything on the caller's stream.
namespace {

struct HostStepLayout {
  size_t q, k, v, seq_lens, tree_sizes, tree_parent, target, draft, tokens, uniforms, greedy, out, path, bonus, alen, status, ws;
  size_t n_q, n_kv, n_target, n_draft, n_bt, n_b, n_u, n_path, ws_bytes, total;
};

bool host_step_layout(const eagle_host_step& s, HostStepLayout* L) {
  if (s.batch < 0 || s.max_tree < 0 || s.vocab < 1 || s.path_cap < 0 || s.kv_capacity < 0) return false;
  eagle_attn_desc d = {};
  d.batch = s.batch; d.num_q_heads = s.num_q_heads; d.num_kv_heads = s.num_kv_heads; d.head_dim = s.head_dim;
  d.max_tree = s.max_tree; d.kv_capacity = s.kv_capacity;
  Workspace w;
  if (!carve_workspace(d, nullptr, &w)) return false;
  const size_t B = static_cast<size_t>(s.batch), T = static_cast<size_t>(s.max_tree);
  L->n_q = B * T * s.num_q_heads * s.head_dim * 2;
  L->n_kv = B * s.num_kv_heads * static_cast<size_t>(s.kv_capacity) * s.head_dim * 2;
  L->n_target = B * (T + 1) * s.vocab * 4;
  L->n_draft = B * T * s.vocab * 4;
  L->n_bt = B * T * 4;
  L->n_b = B * 4;
  L->n_u = B * (T + 1) * 4;
  L->n_path = B * static_cast<size_t>(s.path_cap) * 4;
  L->ws_bytes = w.bytes;
  size_t off = 0;
  auto take = [&](size_t n) { const size_t r = off; off += align256(n > 0 ? n : 1); return r; };
  L->q = take(L->n_q); L->k = take(L->n_kv); L->v = take(L->n_kv);
  L->seq_lens = take(L->n_b); L->tree_sizes = take(L->n_b); L->tree_parent = take(L->n_bt);
  L->target = take(L->n_target); L->draft = take(L->n_draft); L->tokens = take(L->n_bt);
  L->uniforms = take(L->n_u); L->greedy = take(B);
  L->out = take(L->n_q); L->path = take(L->n_path); L->bonus = take(L->n_b); L->alen = take(L->n_b);
  L->status = take(4); L->ws = take(w.bytes);
  L->total = off;
  return true;
}

// What one host-driven step really has to bring to the device: of the caches only the slots a sequence can see
// (prefix + tree), of the probability tensors only the rows of nodes that exist.  Slots and rows past those are never
// read by the kernels, so they are left as they are in the arena.  Copying sequence by sequence costs one call per
// sequence and tensor; it is done when the bytes it saves are worth more than those calls.
struct HostStepTrim {
  bool per_sequence;
  size_t h2d_bytes, d2h_bytes;
};

inline void host_seq_extent(const eagle_host_step& s, int b, int* nodes, long long* slots) {
  int n = s.tree_sizes ? s.tree_sizes[b] : s.max_tree;
  n = n < 0 ? 0 : (n > s.max_tree ? s.max_tree : n);
  long long vis = n > 0 ? static_cast<long long>(s.seq_lens[b]) + n : 0;   // an empty tree reads nothing
  vis = vis < 0 ? 0 : (vis > s.kv_capacity ? s.kv_capacity : vis);
  *nodes = n;
  *slots = vis;
}

HostStepTrim host_step_trim(const eagle_host_step& s, const HostStepLayout& L) {
  HostStepTrim t;
  const size_t small = L.n_q + 2 * L.n_b + 2 * L.n_bt + L.n_u + (s.greedy ? static_cast<size_t>(s.batch) : 0) -
                       (s.tree_sizes ? 0 : L.n_b) - (s.uniforms ? 0 : L.n_u);
  const size_t full = small + 2 * L.n_kv + L.n_target + (s.draft_probs ? L.n_draft : 0);
  size_t trimmed = small;
  const size_t slot_bytes = static_cast<size_t>(s.num_kv_heads) * s.head_dim * 2, row_bytes = static_cast<size_t>(s.vocab) * 4;
  for (int b = 0; b < s.batch; ++b) {
    int n;
    long long vis;
    host_seq_extent(s, b, &n, &vis);
    trimmed += 2 * static_cast<size_t>(vis) * slot_bytes + (static_cast<size_t>(n) + 1) * row_bytes +
               (s.draft_probs ? static_cast<size_t>(n) * row_bytes : 0);
  }
  const size_t calls = static_cast<size_t>(s.batch) * 4;
  t.per_sequence = full > trimmed && full - trimmed > calls * (200u << 10);   // a call costs about what 200 KB take on the link
  t.h2d_bytes = t.per_sequence ? trimmed : full;
  t.d2h_bytes = L.n_q + L.n_path + 2 * L.n_b + 4;
  return t;
}

}  // namespace

size_t eagle_tree_verify_step_host_arena(const eagle_host_step* step) {
  HostStepLayout L;
  if (!step || !host_step_layout(*step, &L)) return 0;
  return L.total;
}

int eagle_tree_verify_step_host_bytes(const eagle_host_step* step, size_t* h2d_bytes, size_t* d2h_bytes) {
  HostStepLayout L;
  if (!step) return EAGLE_ERR_NULL;
  if (!host_step_layout(*step, &L)) return EAGLE_ERR_SHAPE;
  if (step->batch > 0 && !step->seq_lens) return EAGLE_ERR_NULL;
  HostStepTrim t = {false, 0, 0};
  if (step->batch > 0) t = host_step_trim(*step, L);
  if (h2d_bytes) *h2d_bytes = t.h2d_bytes;
  if (d2h_bytes) *d2h_bytes = t.d2h_bytes;
  return EAGLE_OK;
}

int eagle_tree_verify_step_host(const eagle_host_step* step, eagle_stream_t stream_) {
  if (!step) return EAGLE_ERR_NULL;
  const eagle_host_step& s = *step;
  HostStepLayout L;
  if (!host_step_layout(s, &L)) return EAGLE_ERR_SHAPE;
  if (s.batch == 0) return EAGLE_OK;
  if (!s.q || !s.k_cache || !s.v_cache || !s.seq_lens || !s.tree_parent || !s.target_probs || !s.draft_tokens || !s.out ||
      !s.accepted_path || !s.bonus_token)
    return EAGLE_ERR_NULL;
  if ((!s.draft_probs || !s.uniforms) && !s.greedy) return EAGLE_ERR_NULL;
  if (!s.arena || (reinterpret_cast<uintptr_t>(s.arena) & 255) || s.arena_bytes < L.total) return EAGLE_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  char* A = static_cast<char*>(s.arena);
  auto h2d = [&](size_t off, const void* src, size_t n) {
    return !src || n == 0 || cudaMemcpyAsync(A + off, src, n, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  };
  auto d2h = [&](void* dst, size_t off, size_t n) {
    return !dst || n == 0 || cudaMemcpyAsync(dst, A + off, n, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  };
  bool ok = cudaMemsetAsync(A + L.status, 0, 4, stream) == cudaSuccess;
  ok = ok && h2d(L.q, s.q, L.n_q) && h2d(L.seq_lens, s.seq_lens, L.n_b) && h2d(L.tree_sizes, s.tree_sizes, L.n_b) &&
       h2d(L.tree_parent, s.tree_parent, L.n_bt) && h2d(L.tokens, s.draft_tokens, L.n_bt) && h2d(L.uniforms, s.uniforms, L.n_u) &&
       h2d(L.greedy, s.greedy, static_cast<size_t>(s.batch));
  if (host_step_trim(s, L).per_sequence) {
    // per sequence: the visible slots of every KV head (a 2-D copy: one row per head) and the rows of existing nodes
    const size_t slot = static_cast<size_t>(s.head_dim) * 2, pitch = static_cast<size_t>(s.kv_capacity) * slot;
    const size_t row = static_cast<size_t>(s.vocab) * 4, T = static_cast<size_t>(s.max_tree);
    for (int b = 0; b < s.batch && ok; ++b) {
      int n;
      long long vis;
      host_seq_extent(s, b, &n, &vis);
      const size_t kv_off = static_cast<size_t>(b) * s.num_kv_heads * pitch;
      if (vis > 0) {
        ok = cudaMemcpy2DAsync(A + L.k + kv_off, pitch, static_cast<const char*>(s.k_cache) + kv_off, pitch, static_cast<size_t>(vis) * slot,
                               static_cast<size_t>(s.num_kv_heads), cudaMemcpyHostToDevice, stream) == cudaSuccess &&
             cudaMemcpy2DAsync(A + L.v + kv_off, pitch, static_cast<const char*>(s.v_cache) + kv_off, pitch, static_cast<size_t>(vis) * slot,
                               static_cast<size_t>(s.num_kv_heads), cudaMemcpyHostToDevice, stream) == cudaSuccess;
      }
      const size_t t_off = static_cast<size_t>(b) * (T + 1) * row, d_off = static_cast<size_t>(b) * T * row;
      ok = ok && h2d(L.target + t_off, static_cast<const char*>(static_cast<const void*>(s.target_probs)) + t_off, (static_cast<size_t>(n) + 1) * row);
      if (s.draft_probs && n > 0)
        ok = ok && h2d(L.draft + d_off, static_cast<const char*>(static_cast<const void*>(s.draft_probs)) + d_off, static_cast<size_t>(n) * row);
    }
  } else {
    ok = ok && h2d(L.k, s.k_cache, L.n_kv) && h2d(L.v, s.v_cache, L.n_kv) && h2d(L.target, s.target_probs, L.n_target) &&
         h2d(L.draft, s.draft_probs, L.n_draft);
  }
  if (!ok) return EAGLE_ERR_LAUNCH;
  int32_t* d_status = reinterpret_cast<int32_t*>(A + L.status);
  const int32_t* d_sizes = s.tree_sizes ? reinterpret_cast<const int32_t*>(A + L.tree_sizes) : nullptr;
  eagle_attn_desc ad = {};
  ad.batch = s.batch; ad.num_q_heads = s.num_q_heads; ad.num_kv_heads = s.num_kv_heads; ad.head_dim = s.head_dim;
  ad.max_tree = s.max_tree; ad.kv_capacity = s.kv_capacity; ad.tree_sizes = d_sizes; ad.sm_scale = s.sm_scale;
  ad.workspace = A + L.ws; ad.workspace_bytes = L.ws_bytes; ad.status = d_status;
  int rc = eagle_tree_verify_attn(&ad, A + L.q, A + L.k, A + L.v, reinterpret_cast<const int32_t*>(A + L.seq_lens),
                                  reinterpret_cast<const int32_t*>(A + L.tree_parent), A + L.out, stream_);
  if (rc != EAGLE_OK) return rc;
  eagle_accept_desc cd = {};
  cd.batch = s.batch; cd.max_tree = s.max_tree; cd.vocab = s.vocab; cd.path_cap = s.path_cap; cd.tree_sizes = d_sizes;
  cd.greedy = s.greedy ? reinterpret_cast<const uint8_t*>(A + L.greedy) : nullptr;
  cd.accept_len = reinterpret_cast<int32_t*>(A + L.alen); cd.status = d_status;
  rc = eagle_tree_accept(&cd, reinterpret_cast<const float*>(A + L.target),
                         s.draft_probs ? reinterpret_cast<const float*>(A + L.draft) : nullptr,
                         reinterpret_cast<const int32_t*>(A + L.tokens), reinterpret_cast<const int32_t*>(A + L.tree_parent),
                         s.uniforms ? reinterpret_cast<const float*>(A + L.uniforms) : nullptr,
                         reinterpret_cast<int32_t*>(A + L.path), reinterpret_cast<int32_t*>(A + L.bonus), stream_);
  if (rc != EAGLE_OK) return rc;
  ok = d2h(s.out, L.out, L.n_q) && d2h(s.accepted_path, L.path, L.n_path) && d2h(s.bonus_token, L.bonus, L.n_b) &&
       d2h(s.accept_len, L.alen, L.n_b) && d2h(s.status, L.status, 4);
  return ok ? EAGLE_OK : EAGLE_ERR_LAUNCH;
}

namespace {

int commit_call(const eagle_commit_desc* desc, const KvSource& kv, const int32_t* seq_lens, const int32_t* accepted_path,
                const void* features_in, void* features_out, int32_t* new_seq_lens, eagle_stream_t stream_) {
  const eagle_commit_desc& d = *desc;
  if (d.batch < 0 || d.batch > 65535 || d.num_kv_heads < 0 || d.num_kv_heads > 65535 || (d.head_dim != 64 && d.head_dim != 128) ||
      kv.capacity < 0 || d.max_tree < 0 || d.max_tree > kMaxTree || d.path_cap < 0 || d.feature_dim < 0 || d.feature_dim % 8)
    return EAGLE_ERR_SHAPE;
  if (d.batch == 0) return EAGLE_OK;
  if (!seq_lens || (d.path_cap > 0 && !accepted_path)) return EAGLE_ERR_NULL;
  const bool feats = d.feature_dim > 0 && features_out != nullptr;
  if (feats && !features_in) return EAGLE_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(kv.k) & 15) || (reinterpret_cast<uintptr_t>(kv.v) & 15) ||
      (reinterpret_cast<uintptr_t>(features_in) & 15) || (reinterpret_cast<uintptr_t>(features_out) & 15))
    return EAGLE_ERR_SHAPE;
  int err = 0;
  if (!device_info(&err)) return err;
  CommitParams cp;
  cp.k = static_cast<__nv_bfloat16*>(const_cast<void*>(kv.k));
  cp.v = static_cast<__nv_bfloat16*>(const_cast<void*>(kv.v));
  cp.seq_lens = seq_lens;
  cp.path = accepted_path;
  cp.features_in = feats ? static_cast<const __nv_bfloat16*>(features_in) : nullptr;
  cp.features_out = feats ? static_cast<__nv_bfloat16*>(features_out) : nullptr;
  cp.new_seq_lens = new_seq_lens;
  cp.B = d.batch;
  cp.Hkv = d.num_kv_heads;
  cp.D = d.head_dim;
  cp.S_cap = static_cast<int32_t>(kv.capacity < 0x7fffffff ? kv.capacity : 0x7fffffff);
  cp.T_max = d.max_tree;
  cp.path_cap = d.path_cap;
  cp.F = d.feature_dim;
  cp.status = d.status;
  cp.block_table = kv.block_table;
  cp.page_size = kv.page_size;
  cp.max_pages = kv.max_pages;
  cp.num_pages = kv.num_pages;
  if (launch_commit(cp, static_cast<cudaStream_t>(stream_)) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  return EAGLE_OK;
}

}  // namespace

int eagle_tree_commit(const eagle_commit_desc* desc, void* k_cache, void* v_cache, const int32_t* seq_lens,
                      const int32_t* accepted_path, const void* features_in, void* features_out,
                      int32_t* new_seq_lens, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  const KvSource kv = {k_cache, v_cache, desc->kv_capacity, nullptr, 0, 0, 0};
  return commit_call(desc, kv, seq_lens, accepted_path, features_in, features_out, new_seq_lens, stream_);
}

int eagle_tree_commit_paged(const eagle_commit_desc* desc, const eagle_paged_kv* pk, const int32_t* seq_lens,
                            const int32_t* accepted_path, const void* features_in, void* features_out,
                            int32_t* new_seq_lens, eagle_stream_t stream_) {
  if (!desc || !pk) return EAGLE_ERR_NULL;
  if (pk->num_pages < 1 || pk->page_size < 16 || (pk->page_size & (pk->page_size - 1)) || pk->max_pages_per_seq < 0) return EAGLE_ERR_SHAPE;
  if (desc->batch > 0 && !pk->block_table) return EAGLE_ERR_NULL;
  const KvSource kv = {pk->k_pages, pk->v_pages, static_cast<int64_t>(pk->max_pages_per_seq) * pk->page_size, pk->block_table,
                       pk->num_pages, pk->page_size, pk->max_pages_per_seq};
  return commit_call(desc, kv, seq_lens, accepted_path, features_in, features_out, new_seq_lens, stream_);
}

int eagle_tree_expand(const eagle_expand_desc* desc, const float* draft_probs, const int32_t* num_children,
                      const float* uniforms, int32_t* child_tokens, float* child_probs, eagle_stream_t stream_) {
  if (!desc) return EAGLE_ERR_NULL;
  const eagle_expand_desc& d = *desc;
  if (d.batch < 0 || d.batch > 65535 || d.rows < 0 || d.vocab < 1 || d.max_children < 0 || d.max_children > kMaxChildren)
    return EAGLE_ERR_SHAPE;
  if (d.batch == 0 || d.rows == 0 || d.max_children == 0) return EAGLE_OK;
  if (!draft_probs || !num_children || !child_tokens) return EAGLE_ERR_NULL;
  if (!uniforms && !d.greedy) return EAGLE_ERR_NULL;
  int err = 0;
  DeviceInfo* dev = device_info(&err);
  if (!dev) return err;
  ExpandParams ep;
  ep.probs = draft_probs;
  ep.num_children = num_children;
  ep.greedy = d.greedy;
  ep.uniforms = uniforms;
  ep.tokens = child_tokens;
  ep.token_probs = child_probs;
  ep.B = d.batch;
  ep.R = d.rows;
  ep.V = d.vocab;
  ep.K = d.max_children;
  ep.status = d.status;
  if (launch_expand(ep, dev->sm_count, static_cast<cudaStream_t>(stream_)) != cudaSuccess) return EAGLE_ERR_LAUNCH;
  return EAGLE_OK;
}

const char* eagle_status_string(int code) {
  switch (code) {
    case EAGLE_OK: return "ok";
    case EAGLE_ERR_NULL: return "a required pointer is NULL";
    case EAGLE_ERR_SHAPE: return "unsupported shape or misaligned tensor";
    case EAGLE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case EAGLE_ERR_LAUNCH: return "CUDA launch failed";
    case EAGLE_ERR_TREE: return "invalid tree (parent outside [-1, i-1] or tree size out of range)";
    case EAGLE_ERR_SEQ: return "invalid sequence length (negative, or prefix + tree exceeds kv_capacity)";
    case EAGLE_ERR_TOKEN: return "draft token outside the vocabulary";
    case EAGLE_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case EAGLE_ERR_DEVICE: return "no usable sm_100 device is current";
    case EAGLE_ERR_PATH: return "invalid accepted path (not increasing, outside the tree, or past the cache)";
    case EAGLE_ERR_PAGE: return "block-table entry of a page in use outside the page pool";
    default: return "unknown status";
  }
}

uint64_t eagle_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
