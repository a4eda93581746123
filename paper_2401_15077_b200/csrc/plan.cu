// Device-side planner of the tree-verification attention call, and the stand-alone tree-mask builder.
//
// The host never reads seq_lens or tree_sizes (they are device arrays and the call must not synchronise),
// so one small CTA turns them into (1) the per-node ancestor-or-self bit masks that define tree attention
// (Sec. 3.1 / 3.3: a draft token attends to the context and to its own root path) and (2) a list of work
// items for the persistent split-KV attention kernel, longest first, sized so that every SM gets work.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kPlanThreads = 1024;

__device__ inline long long block_sum(long long v, long long* scratch) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) scratch[w] = v;
  __syncthreads();
  long long t = (l < (kPlanThreads >> 5)) ? scratch[l] : 0;
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  return t;
}

// anc[i] = bit i | anc[parent[i]] in node order (parents come first).  Returns false on an invalid entry.
__device__ inline bool build_masks_one(const int32_t* par, int n, uint64_t* anc, uint8_t* depth) {
  for (int i = 0; i < n; ++i) {
    const int pi = par[i];
    if (pi < -1 || pi >= i) return false;
    const uint64_t up = pi >= 0 ? anc[pi] : 0ull;
    anc[i] = up | (1ull << i);
    if (depth) depth[i] = static_cast<uint8_t>(__popcll(up) + 1);
  }
  return true;
}

// work units per KV head: query tiles, or pairs of them
__device__ __forceinline__ int units_of(int mtiles, int pair) { return pair ? (mtiles + 1) / 2 : mtiles; }

__global__ void __launch_bounds__(kPlanThreads) plan_kernel(PlanParams p) {
  __shared__ long long s_red[32];
  __shared__ int s_chunk;
  const int tid = threadIdx.x;
  const int T = p.T_max;

  // ---- per sequence: validate, build masks, count tiles
  long long work = 0;
  for (int b = tid; b < p.B; b += kPlanThreads) {
    int n = p.tree_sizes ? p.tree_sizes[b] : T;
    int L = p.seq_lens[b];
    int bad = 0;
    if (n < 0 || n > T) bad = EAGLE_ERR_TREE;
    else if (L < 0 || static_cast<long long>(L) + n > p.S_cap) bad = EAGLE_ERR_SEQ;
    uint64_t* anc = p.anc + static_cast<size_t>(b) * T;
    if (!bad && !build_masks_one(p.tree_parent + static_cast<size_t>(b) * T, n, anc, nullptr)) bad = EAGLE_ERR_TREE;
    if (bad) {
      report_status(p.status, bad);
      n = 0;
      L = 0;
    }
    for (int i = n; i < T; ++i) anc[i] = 0ull;
    SeqPlan sp;
    sp.n = n;
    sp.L = L;
    sp.mtiles = (n * p.G + kBlockM - 1) / kBlockM;
    sp.item_base = 0;
    sp.splits = 1;
    sp.slot_base = -1;
    sp.ntiles = n > 0 ? (L + n + p.tile_keys - 1) / p.tile_keys : 0;
    sp.key = 0;
    p.seq[b] = sp;
    work += static_cast<long long>(p.Hkv) * units_of(sp.mtiles, p.pair) * sp.ntiles;
  }
  const long long total_work = block_sum(work, s_red);

  // ---- choose the chunk length (KV tiles per item)
  if (tid == 0) {
    long long c = p.min_chunk_tiles;
    if (p.forced_splits == 0) {
      const long long target = (total_work + 2ll * p.num_ctas - 1) / (2ll * p.num_ctas);
      if (target > c) c = target;
    }
    s_chunk = static_cast<int>(c < (1 << 28) ? c : (1 << 28));
  }
  __syncthreads();
  if (p.forced_splits == 0) {
    for (int iter = 0; iter < 28; ++iter) {
      const int chunk = s_chunk;
      long long slots = 0;
      for (int b = tid; b < p.B; b += kPlanThreads) {
        const SeqPlan sp = p.seq[b];
        const int splits = (sp.ntiles + chunk - 1) / chunk;
        if (splits > 1) slots += static_cast<long long>(p.Hkv) * units_of(sp.mtiles, p.pair) * splits * (p.pair ? 2 : 1);
      }
      const long long total_slots = block_sum(slots, s_red);
      if (total_slots <= p.slot_cap) break;
      __syncthreads();
      if (tid == 0) s_chunk = chunk < (1 << 28) ? chunk * 2 : chunk;
      __syncthreads();
    }
  }
  const int chunk = s_chunk;

  // ---- splits per sequence
  for (int b = tid; b < p.B; b += kPlanThreads) {
    SeqPlan sp = p.seq[b];
    int splits;
    if (p.forced_splits > 0) splits = sp.ntiles < p.forced_splits ? sp.ntiles : p.forced_splits;
    else splits = (sp.ntiles + chunk - 1) / chunk;
    if (splits < 1) splits = 1;
    sp.splits = splits;
    sp.key = (sp.ntiles + splits - 1) / splits;   // tiles per item: the sort key
    p.seq[b] = sp;
  }
  __syncthreads();

  // ---- order sequences by item length (longest first) and lay out items and partial slots
  long long my_items = 0;
  for (int b = tid; b < p.B; b += kPlanThreads) {
    const SeqPlan me = p.seq[b];
    long long item_base = 0, slot_base = 0;
    for (int o = 0; o < p.B; ++o) {
      // read only the planning fields: item_base / slot_base of other records are being written
      const int o_key = p.seq[o].key, o_splits = p.seq[o].splits, o_mtiles = p.seq[o].mtiles;
      const bool before = o_key > me.key || (o_key == me.key && o < b);
      if (before) {
        const long long cnt = static_cast<long long>(p.Hkv) * units_of(o_mtiles, p.pair) * o_splits;
        item_base += cnt;
        if (o_splits > 1) slot_base += cnt * (p.pair ? 2 : 1);
      }
    }
    const int units = units_of(me.mtiles, p.pair), per_item = p.pair ? 2 : 1;
    const long long cnt = static_cast<long long>(p.Hkv) * units * me.splits;
    my_items += cnt;
    const bool fits = item_base + cnt <= p.item_cap && (me.splits == 1 || slot_base + cnt * per_item <= p.slot_cap);
    // cannot happen with a workspace of the advertised size; refuse rather than overrun
    if (!fits && cnt > 0) report_status(p.status, EAGLE_ERR_WORKSPACE);
    if (fits) {
      int idx = static_cast<int>(item_base);
      for (int g = 0; g < p.Hkv; ++g)
        for (int mu = 0; mu < units; ++mu)
          for (int s = 0; s < me.splits; ++s, ++idx) {
            WorkItem it;
            it.b = b;
            it.g = g;
            it.mt = p.pair ? 2 * mu : mu;
            it.mode = (p.pair && 2 * mu + 1 < me.mtiles) ? 1 : 0;
            it.tile_begin = static_cast<int>(static_cast<long long>(me.ntiles) * s / me.splits);
            it.tile_end = static_cast<int>(static_cast<long long>(me.ntiles) * (s + 1) / me.splits);
            it.slot = me.splits > 1 ? static_cast<int>(slot_base) + (idx - static_cast<int>(item_base)) * per_item : -1;
            it.pad1 = 0;
            p.items[idx] = it;
          }
    }
    // item_base / slot_base are fields no other thread reads while planning
    p.seq[b].item_base = static_cast<int>(item_base);
    p.seq[b].slot_base = me.splits > 1 ? static_cast<int>(slot_base) : -1;
  }
  const long long n_items = block_sum(my_items, s_red);
  if (tid == 0) {
    p.hdr->n_items = n_items <= p.item_cap ? static_cast<int>(n_items) : 0;
    p.hdr->next_item = 0;
    p.hdr->chunk_tiles = chunk;
    p.hdr->n_slots = 0;
  }
}

__global__ void build_mask_kernel(const int32_t* __restrict__ tree_parent, const int32_t* __restrict__ tree_sizes,
                                  int batch, int T, uint64_t* __restrict__ anc, uint8_t* __restrict__ depth,
                                  int32_t* status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  int n = tree_sizes ? tree_sizes[b] : T;
  uint64_t* a = anc + static_cast<size_t>(b) * T;
  uint8_t* d = depth ? depth + static_cast<size_t>(b) * T : nullptr;
  bool ok = n >= 0 && n <= T;
  if (ok) ok = build_masks_one(tree_parent + static_cast<size_t>(b) * T, n, a, d);
  if (!ok) {
    report_status(status, EAGLE_ERR_TREE);
    n = 0;
  }
  for (int i = n; i < T; ++i) {
    a[i] = 0ull;
    if (d) d[i] = 0;
  }
}

}  // namespace

cudaError_t launch_plan(const PlanParams& p, cudaStream_t stream) {
  plan_kernel<<<1, kPlanThreads, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_build_mask(const int32_t* tree_parent, const int32_t* tree_sizes, int batch, int max_tree,
                              uint64_t* anc, uint8_t* depth, int32_t* status, cudaStream_t stream) {
  const int threads = 128;
  build_mask_kernel<<<(batch + threads - 1) / threads, threads, 0, stream>>>(tree_parent, tree_sizes, batch, max_tree,
                                                                               anc, depth, status);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
