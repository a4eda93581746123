// Merge of the split-KV partials: m* = max_s m_s, l* = sum_s l_s 2^(m_s - m*), O = sum_s O_s 2^(m_s - m*) / l*
// (taken four pieces at a time, rescaling what has been summed when a later group raises the maximum),
// and the zero rows of padded tree nodes.
// A fixed grid (a few blocks per SM) first writes zeros to the rows of nodes past the tree size (one contiguous range
// of the output per sequence, eight work items each), then walks the planner's list of cut query tiles, sixteen work
// items per tile (8 rows each; a thread takes 4 columns of a row).  Query tiles that stayed in one item were written by the
// attention kernel and do not appear in the list.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kCombineThreads = 256;
constexpr int kBlocksPerUnit = 16;                      // 8 rows per block
constexpr int kRowsPerBlock = kBlockM / kBlocksPerUnit;
constexpr int kZeroChunks = 8;                          // work items that share the zeroing of one sequence's padding rows
constexpr int kPiecesAtOnce = 4;                        // pieces of a tile whose loads are in flight together
static_assert(kRowsPerBlock == 8 && kCombineThreads == 256, "a warp reads four 8-row groups of 4 columns: 8 warps cover 128 columns");

template <int D>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(AttnParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int zero_items = p.B * kZeroChunks, total = zero_items + p.hdr->n_cut * kBlocksPerUnit;
  for (int work_all = blockIdx.x; work_all < total; work_all += gridDim.x) {
  if (work_all < zero_items) {
    // ---- a share of the padding rows of one sequence: out[b, n:, :, :] is one contiguous range
    const int b = work_all / kZeroChunks, part = work_all % kZeroChunks;
    const int n = p.seq[b].n;
    const size_t row_elems = static_cast<size_t>(p.Hq) * D;
    uint4* dst = reinterpret_cast<uint4*>(p.out + (static_cast<size_t>(b) * p.T_max + n) * row_elems);
    const size_t vecs = static_cast<size_t>(p.T_max - n) * row_elems / 8;   // 8 bf16 per 16 bytes; D is a multiple of 64
    const size_t lo = vecs * part / kZeroChunks, hi = vecs * (part + 1) / kZeroChunks;
    for (size_t i = lo + threadIdx.x; i < hi; i += kCombineThreads) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    continue;
  }
  const int work = work_all - zero_items;
  // work items of a query tile: (cut tile, 8-row chunk).  A partial is stored [piece][4 columns][row] (the attention
  // kernel writes a row per thread, so this is the order in which its stores are contiguous): a thread takes 4 columns
  // of one row, the eight lanes of a row group read 128 consecutive bytes, a warp four such groups.  Everything a row
  // needs hangs off the planner's record, so the loads of up to four pieces (item extent, (max, sum), partial values)
  // are issued together.
  const CutTile ct = p.cut_tiles[work / kBlocksPerUnit];
  const int r = (work % kBlocksPerUnit) * kRowsPerBlock + (lane & 7);
  const int c4 = warp * 4 + (lane >> 3);           // which 4 columns
  const int R = ct.mt * kBlockM + r;
  if (c4 >= D / 4 || R >= ct.m_valid) continue;
  const int i = R / p.G, h = ct.g * p.G + R % p.G;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float m_star = -INFINITY, l_star = 0.f;
  for (int s0 = 0; s0 < ct.count; s0 += kPiecesAtOnce) {
    float2 ml[kPiecesAtOnce];
    float4 v[kPiecesAtOnce];
    int t0[kPiecesAtOnce], t1[kPiecesAtOnce];
#pragma unroll
    for (int u = 0; u < kPiecesAtOnce; ++u) {
      const int s = s0 + u < ct.count ? s0 + u : ct.count - 1;     // (clamped: the extra loads are discarded)
      const WorkItem* it = p.items + ct.item0 + ct.item_stride * s;
      t0[u] = it->tile_begin;
      t1[u] = it->tile_end;
      const size_t slot = static_cast<size_t>(ct.slot0 + s);
      ml[u] = p.part_ml[slot * kBlockM + r];
      v[u] = *reinterpret_cast<const float4*>(p.part_o + (slot * (D / 4) + c4) * (kBlockM * 4) + r * 4);
    }
    // a piece counts when its item is not empty (an empty item never wrote its slot) and the row saw a key in it
    // (a row all of whose keys in the piece were masked keeps the reference -inf; its sum may hold rounding dust)
    bool use[kPiecesAtOnce];
    float m_new = m_star;
#pragma unroll
    for (int u = 0; u < kPiecesAtOnce; ++u) {
      use[u] = s0 + u < ct.count && t1[u] > t0[u] && ml[u].y > 0.f && ml[u].x > -INFINITY;
      if (use[u]) m_new = fmaxf(m_new, ml[u].x);
    }
    if (m_new == -INFINITY) continue;
    const float keep = exp2f(m_star - m_new);     // 1 when the maximum did not move, 0 for the first pieces
    l_star *= keep;
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] *= keep;
    m_star = m_new;
#pragma unroll
    for (int u = 0; u < kPiecesAtOnce; ++u) {
      if (!use[u]) continue;
      const float w = exp2f(ml[u].x - m_star);
      l_star += ml[u].y * w;
      acc[0] += v[u].x * w;
      acc[1] += v[u].y * w;
      acc[2] += v[u].z * w;
      acc[3] += v[u].w * w;
    }
  }
  const float inv = l_star > 0.f ? 1.f / l_star : 0.f;
  __nv_bfloat16* dst = p.out + ((static_cast<size_t>(ct.b) * p.T_max + i) * p.Hq + h) * D + c4 * 4;
  __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
  __nv_bfloat162 hi = __floats2bfloat162_rn(acc[2] * inv, acc[3] * inv);
  *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  }
}

}  // namespace

cudaError_t launch_combine(const AttnParams& p, int unit_cap, int sm_count, cudaStream_t stream) {
  if (p.B == 0 || p.T_max == 0) return cudaSuccess;
  // the number of cut tiles is only known on the device: a few blocks per SM loop over them
  const long long most = static_cast<long long>(unit_cap) * 2 * kBlocksPerUnit + static_cast<long long>(p.B) * kZeroChunks;
  const long long want = static_cast<long long>(sm_count > 0 ? sm_count : 1) * 8;
  const unsigned blocks = static_cast<unsigned>(want < most ? want : most);
  if (p.D == 128) combine_kernel<128><<<blocks, kCombineThreads, 0, stream>>>(p);
  else combine_kernel<64><<<blocks, kCombineThreads, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
