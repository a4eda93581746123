// Child tokens of draft-tree nodes (App. A.1: in the greedy setting the k most probable tokens of a node's draft
// distribution become its children, otherwise k tokens are sampled; k differs from node to node).
//
// One CTA per (sequence, node): 1024 threads when the row is staged in shared memory, else 256.  The row (128 KB at
// V = 32000) is first copied into shared memory with coalesced 16-byte loads (when it fits; else it is re-read
// through L1 / L2), so HBM is read once and everything below runs out of shared memory.
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

template <int kExpandThreads>
__global__ void __launch_bounds__(kExpandThreads) expand_kernel(ExpandParams p, int stage_row) {
  constexpr int kExpandWarps = kExpandThreads / 32;
  extern __shared__ __align__(16) float s_row[];
  __shared__ unsigned long long s_red[kExpandWarps];
  __shared__ double s_sum[kExpandWarps];
  __shared__ int s_tok[kMaxChildren];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t node = static_cast<size_t>(blockIdx.y) * p.R + blockIdx.x;
  const int b = blockIdx.y, V = p.V, K = p.K;
  const float* row = p.probs + node * V;
  int32_t* out = p.tokens + node * K;
  float* outp = p.token_probs ? p.token_probs + node * K : nullptr;
  int k = p.num_children[node];
  const bool greedy = p.greedy && p.greedy[b] != 0;
  bool bad = k < 0 || k > K || (greedy && k > V) || (!greedy && k > 0 && !p.uniforms);
  if (bad) {
    if (tid == 0) report_status(p.status, EAGLE_ERR_SHAPE);
    k = 0;
  }
  if (tid < K) s_tok[tid] = -1;
  if (stage_row && k > 0) {
    // rows start 16-byte aligned when V % 4 == 0 and the tensor does
    if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(p.probs) & 15) == 0) {
      const float4* src = reinterpret_cast<const float4*>(row);
      float4* dst = reinterpret_cast<float4*>(s_row);
#pragma unroll 8
      for (int i = tid; i < V / 4; i += kExpandThreads) dst[i] = __ldg(src + i);
    } else {
      for (int v = tid; v < V; v += kExpandThreads) s_row[v] = row[v];
    }
    row = s_row;
  }
  __syncthreads();

  if (greedy) {
    // Every thread keeps the largest key among its own tokens that has not been taken yet; a round is a block-wide
    // maximum over those, after which only the winning thread looks for its next one.
    auto local_best = [&](unsigned long long below) {
      unsigned long long best = 0ull;  // keys are never 0: the id part of a real token is at least 1
      for (int v = tid; v < V; v += kExpandThreads) {
        const unsigned long long key = (static_cast<unsigned long long>(sortable_bits(row[v])) << 32) |
                                       static_cast<unsigned int>(~static_cast<unsigned int>(v));
        if (key < below && key > best) best = key;
      }
      return best;
    };
    unsigned long long mine = local_best(~0ull);   // every key is below ~0
    for (int j = 0; j < k; ++j) {
      unsigned long long best = mine;
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long x = __shfl_xor_sync(0xffffffffu, best, o);
        best = x > best ? x : best;
      }
      if (lane == 0) s_red[warp] = best;
      __syncthreads();
      best = s_red[0];
      for (int w = 1; w < kExpandWarps; ++w) best = s_red[w] > best ? s_red[w] : best;
      __syncthreads();
      if (mine == best) {                // keys are unique: exactly one thread
        s_tok[j] = static_cast<int>(~static_cast<unsigned int>(best & 0xffffffffull));
        mine = local_best(best);
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
    unsigned long long lp = static_cast<unsigned long long>(static_cast<unsigned int>(last_pos + 1));
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long x = __shfl_xor_sync(0xffffffffu, lp, o);
      lp = x > lp ? x : lp;
    }
    if (lane == 0) s_red[warp] = lp;
    __syncthreads();
    // prefix sums that tile [0, total) without gaps: a thread's upper bound is computed exactly as its successor's
    // lower bound (same operands, same order)
    const double up = __shfl_up_sync(0xffffffffu, inc, 1);
    double warp_off = 0.0, total = 0.0;
    for (int w = 0; w < kExpandWarps; ++w) {
      if (w == warp) warp_off = total;
      total += s_sum[w];
      lp = s_red[w] > lp ? s_red[w] : lp;
    }
    const double before = lane ? warp_off + up : warp_off;
    const double upto = lane == 31 ? warp_off + s_sum[warp] : warp_off + inc;
    const int fallback = lp > 0 ? static_cast<int>(lp) - 1 : V - 1;
    const float* un = p.uniforms + node * K;
    for (int j = 0; j < k; ++j) {
      const double thr = static_cast<double>(__ldg(un + j)) * total;
      if (before <= thr && upto > thr) {
        // this thread's range holds the threshold: repeat its additions
        double c = 0.0;
        int x = v1 - 1;
        for (int v = v0; v < v1; ++v) {
          c += static_cast<double>(row[v]);
          if (before + c > thr) {
            x = v;
            break;
          }
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

}  // namespace

cudaError_t launch_expand(const ExpandParams& p, cudaStream_t stream) {
  if (p.B == 0 || p.R == 0 || p.K == 0) return cudaSuccess;
  const dim3 grid(static_cast<unsigned>(p.R), static_cast<unsigned>(p.B));
  // a row is staged in shared memory when it fits one SM's shared memory with room to spare (V <= 51200)
  const size_t row_bytes = static_cast<size_t>(p.V) * sizeof(float);
  const int stage = row_bytes <= 200 * 1024 ? 1 : 0;
  const size_t smem = stage ? ((row_bytes + 15) & ~size_t(15)) : 0;
  if (stage) {
    if (smem > 48 * 1024) {
      const cudaError_t e = cudaFuncSetAttribute(expand_kernel<kExpandThreadsStaged>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return e;
    }
    expand_kernel<kExpandThreadsStaged><<<grid, kExpandThreadsStaged, smem, stream>>>(p, 1);
  } else {
    expand_kernel<kExpandThreadsGlobal><<<grid, kExpandThreadsGlobal, 0, stream>>>(p, 0);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
