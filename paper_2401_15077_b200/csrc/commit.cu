// Commit of the accepted path (Sec. 3.3: the accepted tokens and their features are kept for the next drafting
// phase).  The K/V rows of the accepted tree nodes, which sit at cache slots L + path[j], become the next slots of the
// committed prefix, L + j, in place; their feature vectors are gathered into a dense [path_cap, F] block.
//
// One CTA per (sequence, KV head).  The moves of a sequence overlap (slot L + 1 can be the source of position 0 and
// the destination of position 1), so the CTA first reads every row it has to move into registers, then synchronises,
// then writes: at most 64 rows of 256 bytes per tensor, eight 16-byte vectors per thread.  Rows already in place
// (path[j] == j) are skipped.  The CTA of KV head 0 also writes the new prefix length and gathers the features.
// The work is a few hundred KB per call: the kernel is bound by launch and memory latency, not bandwidth.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCommitThreads = 256;
constexpr int kMaxVecsPerThread = 4;   // 64 rows x 16 vectors (D = 128) / 256 threads

__global__ void __launch_bounds__(kCommitThreads) commit_kernel(CommitParams p) {
  __shared__ int s_path[kMaxTree];
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
    for (int j = tid; j < first_end; j += 32) {
      const int m = s_path[j];
      if (m < 0 || m >= p.T_max) bad = 1;                                   // a tree node
      else if (j > 0 && m <= s_path[j - 1]) bad = 1;                        // a child comes after its parent
      else if (static_cast<long long>(L) + m >= p.S_cap) bad = 1;           // its slot exists
    }
    bad = __any_sync(0xffffffffu, bad);
    if (tid == 0) {
      s_len = first_end;
      s_ok = !bad;
      if (bad && g == 0) report_status(p.status, EAGLE_ERR_PATH);
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
    uint4* base = reinterpret_cast<uint4*>(cache + (static_cast<size_t>(b) * p.Hkv + g) * static_cast<size_t>(p.S_cap) * p.D);
    uint4 held[kMaxVecsPerThread];
#pragma unroll
    for (int q = 0; q < kMaxVecsPerThread; ++q) {
      const int i = tid + q * kCommitThreads;
      if (i < total) {
        const int j = i / vpr, c = i % vpr, m = s_path[j];
        if (m != j) held[q] = base[static_cast<size_t>(L + m) * vpr + c];
      }
    }
    __syncthreads();                             // every source row has been read
#pragma unroll
    for (int q = 0; q < kMaxVecsPerThread; ++q) {
      const int i = tid + q * kCommitThreads;
      if (i < total) {
        const int j = i / vpr, c = i % vpr, m = s_path[j];
        if (m != j) base[static_cast<size_t>(L + j) * vpr + c] = held[q];
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
