// Child tokens of draft-tree nodes (App. A.1: in the greedy setting the k most probable tokens of a node's draft
// distribution become its children, otherwise k tokens are sampled; k differs from node to node).
//
// A row (128 KB at V = 32000) that fits shared memory is staged there by a CTA of 1024 threads with coalesced 16-byte
// loads, so HBM is read once and everything else runs out of shared memory; one such CTA per SM walks the rows and
// fetches its next row into registers meanwhile.  Longer rows are read through L1 / L2 by one CTA of 256 threads each.
// Greedy: every thread keeps the largest key among its own tokens that is still available; a round is a block-wide
// maximum over those, and only the round's winner rescans its tokens.  The key (value bits in sortable order,
// inverted token id) is unique, so ties go to the lower id and the result is exact.
// Stochastic: thread t owns the contiguous tokens [t * chunk, (t + 1) * chunk); one sweep gives the per-thread masses,
// one scan their prefix sums (fp64, fixed order), and every draw j is found by the thread whose range holds
// u_j * total, which repeats the additions of its own range.  Draws are independent (with replacement).
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kExpandThreadsGlobal = 256;    // rows read from global memory: several CTAs per SM
constexpr int kExpandThreadsStaged = 1024;   // rows staged in shared memory: one CTA per SM, many loads in flight

__device__ __forceinline__ unsigned int sortable_bits(float f) {
  const unsigned int u = __float_as_uint(f + 0.0f);   // -0 becomes +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Largest 64-bit key over a warp: the hardware warp reduction works on 32-bit words, so the high words go first and
// the low words of the lanes that hold the largest high word second.
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
  const unsigned int hi = static_cast<unsigned int>(v >> 32), lo = static_cast<unsigned int>(v);
  const unsigned int hi_max = __reduce_max_sync(0xffffffffu, hi);
  const unsigned int lo_max = __reduce_max_sync(0xffffffffu, hi == hi_max ? lo : 0u);
  return (static_cast<unsigned long long>(hi_max) << 32) | lo_max;
}

// Largest key among the per-warp maxima in s_red, by every warp on its own.
__device__ __forceinline__ unsigned long long max_of_warp_maxima(const unsigned long long* s_red, int n_warps, int lane) {
  return warp_max_u64(lane < n_warps ? s_red[lane] : 0ull);
}

// One row: `row` points at its V probabilities (shared memory when staged, else global).  Called by the whole CTA.
template <int kExpandThreads>
__device__ __forceinline__ void expand_row(const ExpandParams& p, size_t node, const float* row, int k, bool greedy,
                                           unsigned long long* s_red, double* s_sum, int* s_tok, float* s_un) {
  constexpr int kExpandWarps = kExpandThreads / 32;
  static_assert(kExpandWarps <= 32, "the warp maxima are reduced by one warp");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = p.V, K = p.K;
  int32_t* out = p.tokens + node * K;
  float* outp = p.token_probs ? p.token_probs + node * K : nullptr;
  if (tid < K) s_tok[tid] = -1;
  __syncthreads();
  if (greedy) {
    // Every thread keeps the two largest keys among its own tokens that have not been taken yet; a round is a
    // block-wide maximum over the first of them, after which the winning thread moves its second key up.  Only a thread
    // that wins twice in a row has to look through its tokens again (a one-thread chain of ~30 shared-memory reads,
    // which used to follow every round).
    unsigned long long mine = 0ull, second = 0ull;   // keys are never 0: the id part of a real token is at least 1
    auto make_key = [](unsigned int bits, int v) {
      return (static_cast<unsigned long long>(bits) << 32) | static_cast<unsigned int>(~static_cast<unsigned int>(v));
    };
    // the two largest keys below `below` among this thread's tokens.  Tokens are visited in ascending id, so among equal
    // values the first one met is the larger key and strict 32-bit compares on the value bits keep the order right.
    auto rescan = [&](unsigned long long below) {
      const unsigned int below_bits = static_cast<unsigned int>(below >> 32);
      const int below_v = static_cast<int>(~static_cast<unsigned int>(below & 0xffffffffull));
      const bool all = below == ~0ull;
      unsigned int b1 = 0u, b2 = 0u;    // value bits of the best and the second best (valid when v1 / v2 >= 0)
      int v1 = -1, v2 = -1;
#pragma unroll 4
      for (int v = tid; v < V; v += kExpandThreads) {
        const unsigned int u = sortable_bits(row[v]);
        const bool ok = all || u < below_bits || (u == below_bits && v > below_v);
        if (ok && (v1 < 0 || u > b1)) {
          b2 = b1;
          v2 = v1;
          b1 = u;
          v1 = v;
        } else if (ok && (v2 < 0 || u > b2)) {
          b2 = u;
          v2 = v;
        }
      }
      mine = v1 >= 0 ? make_key(b1, v1) : 0ull;
      second = v2 >= 0 ? make_key(b2, v2) : 0ull;
    };
    bool second_known = true;
    if (k > 0) rescan(~0ull);   // every key is below ~0
    for (int j = 0; j < k; ++j) {
      unsigned long long best = warp_max_u64(mine);
      if (lane == 0) s_red[warp] = best;
      __syncthreads();
      best = max_of_warp_maxima(s_red, kExpandWarps, lane);
      __syncthreads();
      if (mine == best) {                // keys are unique: exactly one thread
        s_tok[j] = static_cast<int>(~static_cast<unsigned int>(best & 0xffffffffull));
        if (second_known) {
          mine = second;                 // (0 when the thread has no other token: it never wins again)
          second_known = false;
        } else {
          rescan(best);
          second_known = true;
        }
      }
    }
  } else if (k > 0) {
    const int chunk = ((V + kExpandThreads - 1) / kExpandThreads) | 1;   // odd: neighbouring threads' ranges start in different banks
    const int v0 = min(tid * chunk, V), v1 = min(v0 + chunk, V);
    double s = 0.0;
    int last_pos = -1;
    for (int v = v0; v < v1; ++v) {
      const float x = row[v];
      s += static_cast<double>(x);
      if (x > 0.f) last_pos = v;
    }
    // exclusive scan of the per-thread masses: within the warp by shuffles, across warps through shared memory
    double inc = s;
    for (int o = 1; o < 32; o <<= 1) {
      const double x = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += x;
    }
    if (lane == 31) s_sum[warp] = inc;
    // the last token with positive mass, for draws that rounding pushes past the end
    unsigned long long lp = __reduce_max_sync(0xffffffffu, static_cast<unsigned int>(last_pos + 1));
    if (lane == 0) s_red[warp] = lp;
    if (tid < k) s_un[tid] = __ldg(p.uniforms + node * K + tid);   // all draws' uniforms at once, not one load per draw
    __syncthreads();
    // prefix sums that tile [0, total) without gaps: a thread's upper bound is computed exactly as its successor's
    // lower bound (same operands, same order)
    const double up = __shfl_up_sync(0xffffffffu, inc, 1);
    // inclusive scan of the warps' masses, by every warp on its own; warp w starts where warp w - 1 ends (the same value)
    double wincl = lane < kExpandWarps ? s_sum[lane] : 0.0;
    for (int o = 1; o < 32; o <<= 1) {
      const double x = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += x;
    }
    const double total = __shfl_sync(0xffffffffu, wincl, kExpandWarps - 1);
    const double warp_end = __shfl_sync(0xffffffffu, wincl, warp);
    const double warp_prev = __shfl_sync(0xffffffffu, wincl, warp > 0 ? warp - 1 : 0);
    const double warp_off = warp > 0 ? warp_prev : 0.0;
    lp = max_of_warp_maxima(s_red, kExpandWarps, lane);
    const double before = lane ? warp_off + up : warp_off;
    const double upto = lane == 31 ? warp_end : warp_off + inc;
    const int fallback = lp > 0 ? static_cast<int>(lp) - 1 : V - 1;
    for (int j = 0; j < k; ++j) {
      const double thr = static_cast<double>(s_un[j]) * total;
      if (before <= thr && upto > thr) {
        // this thread's range holds the threshold: repeat its additions
        double c = 0.0;
        int x = v1 - 1;
#pragma unroll 4
        for (int v = v0; v < v1; ++v) {
          c += static_cast<double>(row[v]);
          if (before + c > thr) x = min(x, v);      // no early exit: the loads of the whole range stay in flight together
        }
        s_tok[j] = x;
      }
    }
    __syncthreads();
    if (tid < k && s_tok[tid] < 0) s_tok[tid] = fallback;   // no range claimed the draw
  }
  __syncthreads();
  if (tid < K) {
    const int t = tid < k ? s_tok[tid] : -1;
    out[tid] = t;
    if (outp) outp[tid] = t >= 0 ? row[t] : 0.f;
  }
}

// k of a node after the checks (0 and a status word when it is unusable)
__device__ __forceinline__ int checked_children(const ExpandParams& p, size_t node, bool greedy) {
  int k = p.num_children[node];
  const bool bad = k < 0 || k > p.K || (greedy && k > p.V) || (!greedy && k > 0 && !p.uniforms);
  if (bad) {
    if (threadIdx.x == 0) report_status(p.status, EAGLE_ERR_SHAPE);
    k = 0;
  }
  return k;
}

// Rows read straight from global memory (they do not fit shared memory): one CTA per row.
template <int kExpandThreads>
__global__ void __launch_bounds__(kExpandThreads) expand_kernel_global(ExpandParams p) {
  __shared__ unsigned long long s_red[kExpandThreads / 32];
  __shared__ double s_sum[kExpandThreads / 32];
  __shared__ int s_tok[kMaxChildren];
  __shared__ float s_un[kMaxChildren];
  const size_t node = static_cast<size_t>(blockIdx.y) * p.R + blockIdx.x;
  const bool greedy = p.greedy && p.greedy[blockIdx.y] != 0;
  const int k = checked_children(p, node, greedy);
  expand_row<kExpandThreads>(p, node, p.probs + node * p.V, k, greedy, s_red, s_sum, s_tok, s_un);
}

// Rows staged in shared memory.  A fixed grid (one CTA per SM) walks the rows; while a row is worked on out of shared
// memory, the next row of this CTA is already on its way from HBM into registers (kVecs 16-byte vectors per thread),
// and is written to shared memory when the current row is finished: loading and selecting overlap.
template <int kExpandThreads, int kVecs>
__global__ void __launch_bounds__(kExpandThreads) expand_kernel_staged(ExpandParams p, int vectors) {
  extern __shared__ __align__(16) float s_row[];
  __shared__ unsigned long long s_red[kExpandThreads / 32];
  __shared__ double s_sum[kExpandThreads / 32];
  __shared__ int s_tok[kMaxChildren];
  __shared__ float s_un[kMaxChildren];
  const int tid = threadIdx.x, V = p.V;
  const size_t n_rows = static_cast<size_t>(p.B) * p.R;
  const int nvec = V / 4;   // used when `vectors` (V % 4 == 0 and the tensor is 16-byte aligned: every row is aligned)
  float4 held[kVecs];
  auto fetch = [&](size_t node) {
    const float4* src = reinterpret_cast<const float4*>(p.probs + node * V);
#pragma unroll
    for (int j = 0; j < kVecs; ++j) {
      const int i = tid + j * kExpandThreads;
      if (i < nvec) held[j] = __ldg(src + i);
    }
  };
  auto stash = [&]() {
    float4* dst = reinterpret_cast<float4*>(s_row);
#pragma unroll
    for (int j = 0; j < kVecs; ++j) {
      const int i = tid + j * kExpandThreads;
      if (i < nvec) dst[i] = held[j];
    }
  };
  size_t node = blockIdx.x;
  if (node >= n_rows) return;
  if (vectors) fetch(node);
  while (node < n_rows) {
    if (vectors) {
      stash();
    } else {
      const float* row = p.probs + node * V;
      for (int v = tid; v < V; v += kExpandThreads) s_row[v] = row[v];
    }
    const size_t next = node + gridDim.x;
    if (vectors && next < n_rows) fetch(next);      // in flight while this row is worked on
    const int b = static_cast<int>(node / p.R);
    const bool greedy = p.greedy && p.greedy[b] != 0;
    const int k = checked_children(p, node, greedy);
    expand_row<kExpandThreads>(p, node, s_row, k, greedy, s_red, s_sum, s_tok, s_un);   // starts with a block barrier
    __syncthreads();                                 // everyone is done with s_row
    node = next;
  }
}

}  // namespace

cudaError_t launch_expand(const ExpandParams& p, int sm_count, cudaStream_t stream) {
  if (p.B == 0 || p.R == 0 || p.K == 0) return cudaSuccess;
  // a row is staged in shared memory when it fits one SM's shared memory with room to spare (V <= 51200)
  const size_t row_bytes = static_cast<size_t>(p.V) * sizeof(float);
  if (row_bytes <= 200 * 1024) {
    const size_t smem = (row_bytes + 15) & ~size_t(15);
    const long long rows = static_cast<long long>(p.B) * p.R;
    const unsigned blocks = static_cast<unsigned>(rows < sm_count ? rows : (sm_count > 0 ? sm_count : 1));
    const int vectors = (p.V & 3) == 0 && (reinterpret_cast<uintptr_t>(p.probs) & 15) == 0;
    // up to 8 vectors per thread (V <= 32768) stay in 32 registers; longer rows take 13
    const bool short_row = p.V <= 8 * 4 * kExpandThreadsStaged;
    auto kernel = short_row ? expand_kernel_staged<kExpandThreadsStaged, 8> : expand_kernel_staged<kExpandThreadsStaged, 13>;
    if (smem > 48 * 1024) {
      const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return e;
    }
    kernel<<<blocks, kExpandThreadsStaged, smem, stream>>>(p, vectors);
  } else {
    const dim3 grid(static_cast<unsigned>(p.R), static_cast<unsigned>(p.B));
    expand_kernel_global<kExpandThreadsGlobal><<<grid, kExpandThreadsGlobal, 0, stream>>>(p);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
