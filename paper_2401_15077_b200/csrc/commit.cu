// Commit of the accepted path (Sec. 3.3: the accepted tokens and their features are kept for the next drafting
// phase).  The K/V rows of the accepted tree nodes, which sit at cache slots L + path[j], become the next slots of the
// committed prefix, L + j, in place; their feature vectors are gathered into a dense [path_cap, F] block.
//
// One CTA per (sequence, KV head).  The moves of a sequence overlap (slot L + 1 can be the source of position 0 and
// the destination of position 1), so the CTA first reads every row it has to move into registers, then synchronises,
// then writes: at most 64 rows of 256 bytes per tensor, eight 16-byte vectors per thread.  Rows already in place
// (path[j] == j) are skipped.  The CTA of KV head 0 also writes the new prefix length and gathers the features.
// The work is a few hundred KB per call: the kernel is bound by launch and memory latency, not bandwidth.
// With a paged cache (power-of-two page size) slot j of a sequence is row j % page_size of the page its block-table
// row names; the pages of the source and destination slots are looked up once, while the path is checked.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCommitThreads = 256;
constexpr int kMaxVecsPerThread = 4;   // 64 rows x 16 vectors (D = 128) / 256 threads

__global__ void __launch_bounds__(kCommitThreads) commit_kernel(CommitParams p) {
  __shared__ int s_path[kMaxTree];
  __shared__ int s_src_page[kMaxTree], s_dst_page[kMaxTree];   // paged cache: page of slot L + path[j] / of slot L + j
  __shared__ int s_len, s_ok;
  const int b = blockIdx.y, g = blockIdx.x, tid = threadIdx.x;
  const int L = p.seq_lens[b];
  const int32_t* path = p.path + static_cast<size_t>(b) * p.path_cap;
  if (tid < 32) {
    // accepted length: entries before the first -1 (at most max_tree of them can be valid)
    const int cap = p.path_cap < kMaxTree ? p.path_cap : kMaxTree;
    int bad = L < 0 ? 1 : 0;
    int first_end = cap;
    for (int j = tid; j < cap; j += 32) {
      const int m = path[j];
      s_path[j] = m;
      if (m == -1 && j < first_end) first_end = j;
    }
    for (int o = 16; o > 0; o >>= 1) first_end = min(first_end, __shfl_xor_sync(0xffffffffu, first_end, o));
    // a row of more than 64 entries without a -1 cannot be a path of a tree of at most 64 nodes
    if (first_end == cap && p.path_cap > kMaxTree && path[kMaxTree] != -1) bad = 1;
    __syncwarp();
    int bad_page = 0;
    for (int j = tid; j < first_end; j += 32) {
      const int m = s_path[j];
      if (m < 0 || m >= p.T_max) bad = 1;                                   // a tree node
      else if (j > 0 && m <= s_path[j - 1]) bad = 1;                        // a child comes after its parent
      else if (static_cast<long long>(L) + m >= p.S_cap) bad = 1;           // its slot exists
      else if (p.block_table && L >= 0) {
        const int32_t* table = p.block_table + static_cast<size_t>(b) * p.max_pages;
        const int src = table[(L + m) / p.page_size], dst = table[(L + j) / p.page_size];
        s_src_page[j] = src;
        s_dst_page[j] = dst;
        if (src < 0 || src >= p.num_pages || dst < 0 || dst >= p.num_pages) bad_page = 1;   // and so does its page
      }
    }
    bad = __any_sync(0xffffffffu, bad);
    bad_page = __any_sync(0xffffffffu, bad_page);
    if (tid == 0) {
      s_len = first_end;
      s_ok = !bad && !bad_page;
      if (g == 0 && (bad || bad_page)) report_status(p.status, bad ? EAGLE_ERR_PATH : EAGLE_ERR_PAGE);
    }
  }
  __syncthreads();
  const int a = s_ok ? s_len : 0;
  if (g == 0) {
    if (tid == 0 && p.new_seq_lens) p.new_seq_lens[b] = L + a;
    if (p.features_out) {
      // features_out[b, j] = features_in[b, path[j]] for j < a, zeros after
      const int vecs = p.F / 8;
      const uint4* src = reinterpret_cast<const uint4*>(p.features_in) + static_cast<size_t>(b) * p.T_max * vecs;
      uint4* dst = reinterpret_cast<uint4*>(p.features_out) + static_cast<size_t>(b) * p.path_cap * vecs;
      for (int i = tid; i < p.path_cap * vecs; i += kCommitThreads) {
        const int j = i / vecs, c = i % vecs;
        dst[i] = j < a ? src[static_cast<size_t>(s_path[j]) * vecs + c] : make_uint4(0u, 0u, 0u, 0u);
      }
    }
  }
  if (a == 0 || g >= p.Hkv) return;
  const int vpr = p.D / 8;                       // 16-byte vectors per row
  const int total = a * vpr;
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    __nv_bfloat16* cache = t == 0 ? p.k : p.v;
    if (!cache) continue;                        // uniform over the CTA
    // row of slot `slot` (whose page is `page` when the cache is paged), as 16-byte vectors
    auto row = [&](int slot, int page) -> uint4* {
      const size_t r = p.block_table ? (static_cast<size_t>(page) * p.Hkv + g) * p.page_size + (slot & (p.page_size - 1))
                                     : (static_cast<size_t>(b) * p.Hkv + g) * static_cast<size_t>(p.S_cap) + slot;
      return reinterpret_cast<uint4*>(cache) + r * vpr;
    };
    uint4 held[kMaxVecsPerThread];
#pragma unroll
    for (int q = 0; q < kMaxVecsPerThread; ++q) {
      const int i = tid + q * kCommitThreads;
      if (i < total) {
        const int j = i / vpr, c = i % vpr, m = s_path[j];
        if (m != j) held[q] = row(L + m, s_src_page[j])[c];
      }
    }
    __syncthreads();                             // every source row has been read
#pragma unroll
    for (int q = 0; q < kMaxVecsPerThread; ++q) {
      const int i = tid + q * kCommitThreads;
      if (i < total) {
        const int j = i / vpr, c = i % vpr, m = s_path[j];
        if (m != j) row(L + j, s_dst_page[j])[c] = held[q];
      }
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_commit(const CommitParams& p, cudaStream_t stream) {
  if (p.B == 0) return cudaSuccess;
  const dim3 grid(static_cast<unsigned>(p.Hkv > 0 ? p.Hkv : 1), static_cast<unsigned>(p.B));
  commit_kernel<<<grid, kCommitThreads, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
