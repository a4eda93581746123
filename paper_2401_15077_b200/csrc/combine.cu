// Merge of the split-KV partials: m* = max_s m_s, l* = sum_s l_s 2^(m_s - m*), O = sum_s O_s 2^(m_s - m*) / l*.
// One warp per output row (sequence, node, query head).  Rows of work units that stayed in one piece were already
// written by the attention kernel and are skipped; rows of nodes past the tree size are written as zeros.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCombineThreads = 128;

template <int D>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(AttnParams p) {
  constexpr int E = D / 32;  // elements per lane
  const int lane = threadIdx.x & 31;
  const long long row = static_cast<long long>(blockIdx.x) * (kCombineThreads / 32) + (threadIdx.x >> 5);
  const long long rows = static_cast<long long>(p.B) * p.T_max * p.Hq;
  if (row >= rows) return;
  const int h = static_cast<int>(row % p.Hq);
  const int i = static_cast<int>((row / p.Hq) % p.T_max);
  const int b = static_cast<int>(row / (static_cast<long long>(p.Hq) * p.T_max));
  const SeqPlan sp = p.seq[b];
  __nv_bfloat16* dst = p.out + static_cast<size_t>(row) * D + lane * E;
  if (i >= sp.n) {
    if (E == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(0u, 0u);
    else *reinterpret_cast<uint32_t*>(dst) = 0u;
    return;
  }
  const int g = h / p.G, R = i * p.G + h % p.G;
  const int mt = R / kBlockM, r = R % kBlockM;
  const UnitPlan up = p.units[sp.unit_base + g * sp.mtiles + mt];
  if (up.n_pieces <= 1) return;   // written directly by the attention kernel
  const size_t slot0 = static_cast<size_t>(up.slot_base);
  const int splits = up.n_pieces;
  float m_star = -INFINITY;
  for (int s = 0; s < splits; ++s) {
    const float2 ml = p.part_ml[(slot0 + s) * kBlockM + r];
    if (ml.y > 0.f) m_star = fmaxf(m_star, ml.x);
  }
  float acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  float l_star = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float2 ml = p.part_ml[(slot0 + s) * kBlockM + r];
    if (!(ml.y > 0.f)) continue;   // a split in which this row saw no key
    const float w = exp2f(ml.x - m_star);
    l_star += ml.y * w;
    const float* po = p.part_o + ((slot0 + s) * kBlockM + r) * D + lane * E;
    if (E == 4) {
      const float4 v = *reinterpret_cast<const float4*>(po);
      acc[0] += v.x * w; acc[1] += v.y * w; acc[2 % E] += v.z * w; acc[3 % E] += v.w * w;
    } else {
      const float2 v = *reinterpret_cast<const float2*>(po);
      acc[0] += v.x * w; acc[1] += v.y * w;
    }
  }
  const float inv = l_star > 0.f ? 1.f / l_star : 0.f;
  __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
  if (E == 4) {
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc[2 % E] * inv, acc[3 % E] * inv);
    *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  } else {
    *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<uint32_t*>(&lo);
  }
}

}  // namespace

cudaError_t launch_combine(const AttnParams& p, cudaStream_t stream) {
  const long long rows = static_cast<long long>(p.B) * p.T_max * p.Hq;
  if (rows == 0) return cudaSuccess;
  const unsigned blocks = static_cast<unsigned>((rows + kCombineThreads / 32 - 1) / (kCombineThreads / 32));
  if (p.D == 128) combine_kernel<128><<<blocks, kCombineThreads, 0, stream>>>(p);
  else combine_kernel<64><<<blocks, kCombineThreads, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
