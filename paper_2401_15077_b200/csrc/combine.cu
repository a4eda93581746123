// Merge of the split-KV partials: m* = max_s m_s, l* = sum_s l_s 2^(m_s - m*), O = sum_s O_s 2^(m_s - m*) / l*,
// and the zero rows of padded tree nodes.
// Eight blocks per query tile (16 rows each, two rows per warp): a tile that stayed in one item was written by the
// attention kernel and costs one table look-up here; otherwise its rows are merged from the items that hold it.  One more block per sequence
// writes zeros to the rows of nodes past the tree size (one contiguous range of the output).
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCombineThreads = 256;
constexpr int kBlocksPerUnit = 8;                       // 16 rows per block
constexpr int kRowsPerBlock = kBlockM / kBlocksPerUnit;

template <int D>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(AttnParams p, int unit_blocks) {
  constexpr int E = D / 32;  // elements per lane
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (static_cast<int>(blockIdx.x) >= unit_blocks) {
    // ---- padding rows of one sequence: out[b, n:, :, :]
    const int b = blockIdx.x - unit_blocks;
    const int n = p.seq[b].n;
    const size_t row_elems = static_cast<size_t>(p.Hq) * D;
    uint4* dst = reinterpret_cast<uint4*>(p.out + (static_cast<size_t>(b) * p.T_max + n) * row_elems);
    const size_t vecs = static_cast<size_t>(p.T_max - n) * row_elems / 8;   // 8 bf16 per 16 bytes; D is a multiple of 64
    for (size_t i = threadIdx.x; i < vecs; i += kCombineThreads) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  // blocks are laid out per query tile: (super-unit, tile-in-pair, 16-row chunk)
  const int su = blockIdx.x / (2 * kBlocksPerUnit), which = (blockIdx.x / kBlocksPerUnit) & 1;
  const int row0 = (blockIdx.x % kBlocksPerUnit) * kRowsPerBlock;
  if (su >= p.hdr->n_units) return;
  const UnitPlan up = p.units[su];
  if (up.slot_base < 0) return;   // every query tile of this super-unit was written directly by the attention kernel
  const int b = up.pad0;
  const SeqPlan sp = p.seq[b];
  const int npairs = (sp.mtiles + 1) / 2;
  const int k = su - sp.unit_base, g = k / npairs, mp = k % npairs;
  const bool paired = 2 * mp + 1 < sp.mtiles;
  const int mt = 2 * mp + which;
  if (mt >= sp.mtiles) return;    // a lone tile has no sibling
  const int m_valid = sp.n * p.G;
  // the items that hold this query tile: one per team piece for a pair, both for a lone tile (its two halves)
  const int first = 2 * up.first_item, count = paired ? up.n_pieces : 2 * up.n_pieces;
  for (int r = row0 + warp; r < row0 + kRowsPerBlock; r += kCombineThreads / 32) {
    const int R = mt * kBlockM + r;
    if (R >= m_valid) break;
    const int i = R / p.G, h = g * p.G + R % p.G;
    float m_star = -INFINITY;
    for (int s = 0; s < count; ++s) {
      const WorkItem it = p.items[paired ? first + 2 * s + which : first + s];
      if (it.tile_end <= it.tile_begin) continue;
      const float2 ml = p.part_ml[static_cast<size_t>(it.slot) * kBlockM + r];
      if (ml.y > 0.f) m_star = fmaxf(m_star, ml.x);
    }
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    float l_star = 0.f;
    for (int s = 0; s < count; ++s) {
      const WorkItem it = p.items[paired ? first + 2 * s + which : first + s];
      if (it.tile_end <= it.tile_begin) continue;
      const float2 ml = p.part_ml[static_cast<size_t>(it.slot) * kBlockM + r];
      if (!(ml.y > 0.f)) continue;   // a piece in which this row saw no key
      const float w = exp2f(ml.x - m_star);
      l_star += ml.y * w;
      const float* po = p.part_o + (static_cast<size_t>(it.slot) * kBlockM + r) * D + lane * E;
      if constexpr (E == 4) {
        const float4 v = *reinterpret_cast<const float4*>(po);
        acc[0] += v.x * w; acc[1] += v.y * w; acc[2] += v.z * w; acc[3] += v.w * w;
      } else {
        const float2 v = *reinterpret_cast<const float2*>(po);
        acc[0] += v.x * w; acc[1] += v.y * w;
      }
    }
    const float inv = l_star > 0.f ? 1.f / l_star : 0.f;
    __nv_bfloat16* dst = p.out + ((static_cast<size_t>(b) * p.T_max + i) * p.Hq + h) * D + lane * E;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
    if constexpr (E == 4) {
      __nv_bfloat162 hi = __floats2bfloat162_rn(acc[2] * inv, acc[3] * inv);
      *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    } else {
      *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<uint32_t*>(&lo);
    }
  }
}

}  // namespace

cudaError_t launch_combine(const AttnParams& p, int unit_cap, cudaStream_t stream) {
  if (p.B == 0 || p.T_max == 0) return cudaSuccess;
  const unsigned unit_blocks = static_cast<unsigned>(unit_cap) * 2 * kBlocksPerUnit;   // unit_cap super-units, two query tiles each
  const unsigned blocks = unit_blocks + static_cast<unsigned>(p.B);
  if (p.D == 128) combine_kernel<128><<<blocks, kCombineThreads, 0, stream>>>(p, static_cast<int>(unit_blocks));
  else combine_kernel<64><<<blocks, kCombineThreads, 0, stream>>>(p, static_cast<int>(unit_blocks));
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
