// Merge of the split-KV partials: m* = max_s m_s, l* = sum_s l_s 2^(m_s - m*), O = sum_s O_s 2^(m_s - m*) / l*,
// and the zero rows of padded tree nodes.
// A fixed grid (a few blocks per SM) walks the planner's list of cut query tiles, sixteen work items per tile
// (8 rows each, one row per warp), then one work item per sequence that writes zeros to the rows of nodes past
// the tree size (one contiguous range of the output).  Query tiles that stayed in one item were written by the
// attention kernel and do not appear in the list.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCombineThreads = 256;
constexpr int kBlocksPerUnit = 16;                      // 8 rows per block: one per warp
constexpr int kRowsPerBlock = kBlockM / kBlocksPerUnit;

template <int D>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(AttnParams p) {
  constexpr int E = D / 32;  // elements per lane
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tile_items = p.hdr->n_cut * kBlocksPerUnit, total = tile_items + p.B;
  for (int work = blockIdx.x; work < total; work += gridDim.x) {
  if (work >= tile_items) {
    // ---- padding rows of one sequence: out[b, n:, :, :]
    const int b = work - tile_items;
    const int n = p.seq[b].n;
    const size_t row_elems = static_cast<size_t>(p.Hq) * D;
    uint4* dst = reinterpret_cast<uint4*>(p.out + (static_cast<size_t>(b) * p.T_max + n) * row_elems);
    const size_t vecs = static_cast<size_t>(p.T_max - n) * row_elems / 8;   // 8 bf16 per 16 bytes; D is a multiple of 64
    for (size_t i = threadIdx.x; i < vecs; i += kCombineThreads) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    continue;
  }
  // work items of a query tile: (cut tile, 16-row chunk)
  const int code = p.cut_tiles[work / kBlocksPerUnit];
  const bool paired = ((code >> 30) & 1) == 0;        // a pair or twin: this tile's pieces are one CTA's items
  const int su = (code & 0x3fffffff) >> 1, which = code & 1;
  const int row0 = (work % kBlocksPerUnit) * kRowsPerBlock;
  const UnitPlan up = p.units[su];
  // which query tile this is: every item of it says so, empty or not
  const WorkItem it0 = p.items[2 * up.first_item + (paired ? which : 0)];
  const int b = it0.b, g = it0.g, mt = it0.mt;
  const SeqPlan sp = p.seq[b];
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
}

}  // namespace

cudaError_t launch_combine(const AttnParams& p, int unit_cap, int sm_count, cudaStream_t stream) {
  if (p.B == 0 || p.T_max == 0) return cudaSuccess;
  // the number of cut tiles is only known on the device: a few blocks per SM loop over them
  const long long most = static_cast<long long>(unit_cap) * 2 * kBlocksPerUnit + p.B;
  const long long want = static_cast<long long>(sm_count > 0 ? sm_count : 1) * 8;
  const unsigned blocks = static_cast<unsigned>(want < most ? want : most);
  if (p.D == 128) combine_kernel<128><<<blocks, kCombineThreads, 0, stream>>>(p);
  else combine_kernel<64><<<blocks, kCombineThreads, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
