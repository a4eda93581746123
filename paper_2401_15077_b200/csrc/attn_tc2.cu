// Split-KV tree attention for sm_100a, two softmax warpgroups per CTA.
//
// TMA stages 128-key K and V tiles (128-byte swizzled boxes) through one ring of five 32 KB shared-memory
// slots; tcgen05 MMAs compute S = Q K^T and O += P V with accumulators in TMEM; one persistent CTA per SM
// walks a static slice of the planner's work list.  An item covers a range of KV tiles of one (sequence,
// KV head) for either
//   mode 1: two 128-row query tiles (rows = tree node * G + head-in-group): warpgroup w owns query tile w;
//           every K / V tile in shared memory feeds both, so the cache is read once for 256 query rows; or
//   mode 0: one query tile: warpgroup 0 takes the even KV tiles of the range, warpgroup 1 the odd ones,
//           each with its own running max / sum / accumulator; the two are merged in the epilogue.
// Either way each warpgroup runs the chain  QK -> softmax -> PV  on its own TMEM columns (S_w, with P_w
// written over the first half of S_w; O_w), and the tensor pipe interleaves the two chains, so one
// warpgroup's exponentials overlap the other's MMAs.
// Warp roles: warps 0-3 and 4-7 softmax warpgroups (thread r <-> query row r <-> TMEM lane r), warp 8 TMA
// producer, warp 9 MMA issuer.  Softmax is fp32 in the log2 domain; the tree mask is applied in registers
// only on tiles that reach past the committed prefix; rows of a V tile past prefix + tree are zeroed in
// shared memory before the MMA reads them.  The accumulator is rescaled only when the running max grows by
// more than 2^8.  Every wait is bounded (mbarrier try_wait + timer); on expiry the CTA raises
// EAGLE_ERR_TIMEOUT, all roles leave their loops, TMEM is released and the kernel returns.
#include <cuda.h>

#include "common.cuh"

namespace eagle {

namespace {

constexpr int kTileN = 128;          // keys per KV tile
constexpr int kSlots = 5;            // ring slots; tile g uses slot (2g) % 5 for K and (2g+1) % 5 for V
constexpr int kThreads = 320;
constexpr int kWgThreads = 128;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;        // S_w at w*128; P_w (packed bf16, 64 columns) overwrites its first half
constexpr uint32_t kColO = 256;      // O_w at 256 + w*128
constexpr float kRescaleThreshold = 8.0f;   // log2 units
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// ---------------------------------------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false if the CTA has been aborted or the time limit passed (and raises the abort flag).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer();
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (global_timer() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Same, with a verdict that is uniform over the warp (the callers go on to warp-collective tcgen05 instructions).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(addr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t addr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
        "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
        "r"(r[30]), "r"(r[31])
      : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
//   K-major operand (Q, K): rows of 128 bytes (64 bf16 along the contraction), LBO unused.
//   MN-major operand (V):   rows of 128 bytes (64 bf16 along N), `lbo_bytes` between 64-wide N chunks.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr >> 4) & 0x3fffu);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= static_cast<uint64_t>((1024u >> 4) & 0x3fffu) << 32;   // stride between 8-row groups
  d |= 1ull << 46;                                            // descriptor version of sm_100
  d |= 2ull << 61;                                            // SWIZZLE_128B
  return d;
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}


template <int D>
struct Smem2 {
  static constexpr int kSlabs = D / 64;                     // 64 bf16 = one 128-byte swizzled row
  static constexpr int kSlabBytes = kTileN * 128;            // 128 rows x 128 bytes
  static constexpr int kTileBytes = kSlabs * kSlabBytes;     // one Q / K / V tile
  static constexpr int kQ = 0;                               // two query tiles
  static constexpr int kRing = 2 * kTileBytes;
  static constexpr int kMl = kRing + kSlots * kTileBytes;    // float2 [2][128]: (max, sum) exchange of mode 0
  static constexpr int kBar = kMl + 2 * kBlockM * 8;
  static constexpr int kNumBars = 2 * kSlots + 2 + 2 + 2 + 4;
  static constexpr int kMisc = kBar + 8 * kNumBars;           // tmem base, abort flag
  static constexpr int kBytes = kMisc + 16;
};

struct Bars2 {
  uint32_t full[kSlots], empty[kSlots];
  uint32_t s_full[2], p_full[2], o_done[2];
  uint32_t q_full, q_empty, o_free, ml_full;
};

__device__ __forceinline__ int item_index(int row, int cta, int grid) {
  return row * grid + ((row & 1) ? (grid - 1 - cta) : cta);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc2_kernel(AttnParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  using S = Smem2<D>;
  extern __shared__ __align__(1024) unsigned char smem[];
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (sbase & 1023u) {   // the swizzled tiles need a 1024-byte aligned base; uniform over the CTA
    if (tid == 0) report_status(p.status, EAGLE_ERR_DEVICE);
    return;
  }

  Bars2 B;
  {
    uint32_t b = sbase + S::kBar;
    for (int i = 0; i < kSlots; ++i) { B.full[i] = b; b += 8; }
    for (int i = 0; i < kSlots; ++i) { B.empty[i] = b; b += 8; }
    for (int i = 0; i < 2; ++i) { B.s_full[i] = b; b += 8; }
    for (int i = 0; i < 2; ++i) { B.p_full[i] = b; b += 8; }
    for (int i = 0; i < 2; ++i) { B.o_done[i] = b; b += 8; }
    B.q_full = b; b += 8;
    B.q_empty = b; b += 8;
    B.o_free = b; b += 8;
    B.ml_full = b;
  }
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + S::kMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + S::kMisc + 4);

  if (tid == 0) {
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(B.full[i], 1);
      mbar_init(B.empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(B.s_full[i], 1);
      mbar_init(B.p_full[i], kWgThreads);
      mbar_init(B.o_done[i], 1);
    }
    mbar_init(B.q_full, 2 * kWgThreads);
    mbar_init(B.q_empty, 1);
    mbar_init(B.o_free, 2 * kWgThreads);
    mbar_init(B.ml_full, 2 * kWgThreads);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + S::kMisc), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  const int n_items = p.hdr->n_items;
  const int grid = gridDim.x, cta = blockIdx.x;

  if (warp == 8) {
    // =========================================================================== TMA producer
    if (lane == 0) {
      uint32_t g = 0;   // KV tiles issued by this CTA so far
      bool ok = true;
      for (int row = 0; ok; ++row) {
        const int idx = item_index(row, cta, grid);
        if (idx >= n_items) break;
        const WorkItem it = p.items[idx];
        const int z = it.b * p.Hkv + it.g;
        for (int tile = it.tile_begin; tile < it.tile_end && ok; ++tile, ++g) {
#pragma unroll
          for (int kv = 0; kv < 2; ++kv) {
            const uint32_t n = 2 * g + kv, slot = n % kSlots, par = ((n / kSlots) & 1u) ^ 1u;
            ok = mbar_wait(B.empty[slot], par, s_abort);
            if (!ok) break;
            mbar_expect_tx(B.full[slot], S::kTileBytes);
#pragma unroll
            for (int s = 0; s < S::kSlabs; ++s)
              tma_load_3d(sbase + S::kRing + slot * S::kTileBytes + s * S::kSlabBytes, kv ? &map_v : &map_k, s * 64, tile * kTileN, z,
                          B.full[slot]);
          }
        }
      }
    }
  } else if (warp == 9) {
    // =========================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kBlockM, kTileN, false);
      constexpr uint32_t idesc_pv = instr_desc(kBlockM, D, true);
      uint32_t g_base = 0, item_count = 0;
      uint32_t cw[2] = {0u, 0u};       // steps issued per warpgroup stream (phase counters of s_full / p_full / o_done)
      bool ok = true;
      for (int row = 0; ok; ++row) {
        const int idx = item_index(row, cta, grid);
        if (idx >= n_items) break;
        const WorkItem it = p.items[idx];
        const int nt = it.tile_end - it.tile_begin, mode = it.mode;
        const int steps[2] = {mode ? nt : (nt + 1) / 2, mode ? nt : nt / 2};
        int qk_left = steps[0] + steps[1];
        bool first_pv = true;
        ok = mbar_wait(B.q_full, item_count & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        auto issue_qk = [&](int w, int k) -> bool {
          const uint32_t g = g_base + (mode ? k : 2 * k + w);
          const uint32_t n = 2 * g, slot = n % kSlots, par = (n / kSlots) & 1u;
          if (!mbar_wait(B.full[slot], par, s_abort)) return false;
          tc_fence_after();
          const uint32_t d_tmem = tmem + kColS + w * kTileN;
          const uint32_t q_addr = sbase + S::kQ + (mode ? w : 0) * S::kTileBytes;
          const uint32_t k_addr = sbase + S::kRing + slot * S::kTileBytes;
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk / 4) * S::kSlabBytes + (kk % 4) * 32;
            umma_ss(d_tmem, smem_desc(q_addr + off, 16), smem_desc(k_addr + off, 16), idesc_qk, kk > 0 ? 1u : 0u);
          }
          tc_commit(B.s_full[w]);
          if (!mode || w == 1) tc_commit(B.empty[slot]);   // last reader of this K tile
          if (--qk_left == 0) tc_commit(B.q_empty);         // every QK of this item has been issued
          return true;
        };
        auto issue_pv = [&](int w, int k) -> bool {
          const uint32_t g = g_base + (mode ? k : 2 * k + w);
          const uint32_t n = 2 * g + 1, slot = n % kSlots, par = (n / kSlots) & 1u;
          if (!mbar_wait(B.p_full[w], cw[w] & 1u, s_abort)) return false;
          if (!mbar_wait(B.full[slot], par, s_abort)) return false;
          if (first_pv && item_count > 0) {
            if (!mbar_wait(B.o_free, (item_count - 1) & 1u, s_abort)) return false;   // previous epilogue has read O
          }
          first_pv = false;
          tc_fence_after();
          const uint32_t a_tmem = tmem + kColS + w * kTileN;
          const uint32_t v_addr = sbase + S::kRing + slot * S::kTileBytes;
#pragma unroll
          for (int kk = 0; kk < kTileN / 16; ++kk)
            umma_ts(tmem + kColO + w * kTileN, a_tmem + kk * 8, smem_desc(v_addr + kk * 2048, S::kSlabBytes), idesc_pv,
                    (k > 0 || kk > 0) ? 1u : 0u);
          tc_commit(B.o_done[w]);
          if (!mode || w == 1) tc_commit(B.empty[slot]);   // last reader of this V tile
          ++cw[w];
          return true;
        };
        ok = issue_qk(0, 0);
        if (ok && steps[1] > 0) ok = issue_qk(1, 0);
        for (int k = 0; k < steps[0] && ok; ++k) {
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            if (!ok || k >= steps[w]) continue;
            ok = issue_pv(w, k);
            if (ok && k + 1 < steps[w]) ok = issue_qk(w, k + 1);
          }
        }
        g_base += nt;
        ++item_count;
      }
    }
  } else {
    // =========================================================================== softmax warpgroups + epilogue
    const int w = warp >> 2;                              // warpgroup = stream
    const int r = tid & (kWgThreads - 1);                 // query row of this thread within its tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    uint32_t g_base = 0, item_count = 0, cws = 0, mode0_count = 0;
    bool ok = true;
    for (int row = 0; ok; ++row) {
      const int idx = item_index(row, cta, grid);
      if (idx >= n_items) break;
      const WorkItem it = p.items[idx];
      const SeqPlan sp = p.seq[it.b];
      const int L = sp.L, n = sp.n, G = p.G, mode = it.mode;
      const int m_valid = n * G;
      const int R = (it.mt + (mode ? w : 0)) * kBlockM + r;
      const bool row_valid = R < m_valid;
      const int node = row_valid ? R / G : 0, hh = row_valid ? R % G : 0;
      const uint64_t anc = row_valid ? p.anc[static_cast<size_t>(it.b) * p.T_max + node] : 0ull;
      const int kv_end = L + n;
      const int nt = it.tile_end - it.tile_begin;
      const int steps = mode ? nt : (w == 0 ? (nt + 1) / 2 : nt / 2);

      // ---- stage Q: mode 1: this warpgroup's own tile, whole rows; mode 0: the shared tile, 64-column slab per warpgroup
      ok = mbar_wait_warp(B.q_empty, (item_count & 1u) ^ 1u, s_abort);
      if (!ok) break;
      {
        const uint4* src = reinterpret_cast<const uint4*>(p.q + ((static_cast<size_t>(it.b) * p.T_max + node) * p.Hq + it.g * G + hh) * D);
        unsigned char* qdst = smem + S::kQ + (mode ? w : 0) * S::kTileBytes;
        if (mode || D == 64) {
          if (mode || w == 0) {
#pragma unroll
            for (int c = 0; c < D / 8; ++c) {
              const uint4 v = row_valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
              *reinterpret_cast<uint4*>(qdst + (c / 8) * S::kSlabBytes + r * 128 + (((c % 8) ^ (r & 7)) << 4)) = v;
            }
          }
        } else {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 v = row_valid ? __ldg(src + w * 8 + c) : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(qdst + w * S::kSlabBytes + r * 128 + ((c ^ (r & 7)) << 4)) = v;
          }
        }
      }
      fence_proxy_async();
      mbar_arrive(B.q_full);

      float m_ref = -INFINITY;   // reference max (scaled, log2 domain) of every exponential taken so far
      float l_sum = 0.f;
      for (int k = 0; k < steps && ok; ++k, ++cws) {
        const uint32_t g = g_base + (mode ? k : 2 * k + w);
        ok = mbar_wait_warp(B.s_full[w], cws & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        const int key0 = (it.tile_begin + static_cast<int>(g - g_base)) * kTileN;
        const bool tail = key0 + kTileN > L;   // the tile reaches past the committed prefix: tree mask + cache tail
        const uint32_t s_addr = tmem + lane_addr + kColS + w * kTileN;
        uint32_t raw[64];
        // 64 score columns starting at column h*64, masked on tail tiles (two passes over TMEM keep registers low)
        auto load_half = [&](int h) {
          tmem_ld32(s_addr + h * 64, raw);
          tmem_ld32(s_addr + h * 64 + 32, raw + 32);
          tc_wait_ld();
          if (tail) {
#pragma unroll
            for (int e = 0; e < 64; ++e) {
              const int mrel = key0 + h * 64 + e - L;
              const bool vis = mrel < 0 || (mrel < n && ((anc >> mrel) & 1ull));
              raw[e] = vis ? raw[e] : 0xff800000u;   // -inf
            }
          }
        };
        // ---- pass 1: row max
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          load_half(h);
#pragma unroll
          for (int e = 0; e < 64; e += 4) {
            mx[0] = fmaxf(mx[0], __uint_as_float(raw[e]));
            mx[1] = fmaxf(mx[1], __uint_as_float(raw[e + 1]));
            mx[2] = fmaxf(mx[2], __uint_as_float(raw[e + 2]));
            mx[3] = fmaxf(mx[3], __uint_as_float(raw[e + 3]));
          }
        }
        const float tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * p.scale_log2;   // scale > 0

        if (key0 + kTileN > kv_end) {
          // rows of the V tile past prefix + tree may hold anything: zero them so that 0 * garbage cannot reach O
          const uint32_t nv = 2 * g + 1, slot = nv % kSlots, par = (nv / kSlots) & 1u;
          ok = mbar_wait_warp(B.full[slot], par, s_abort);
          if (!ok) break;
          if (key0 + r >= kv_end) {
#pragma unroll
            for (int sl = 0; sl < S::kSlabs; ++sl)
#pragma unroll
              for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(smem + S::kRing + slot * S::kTileBytes + sl * S::kSlabBytes + r * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();
        }

        // lazy rescale: move the reference only when the row max outgrows it by more than the threshold.
        // (PV of the previous step of this stream has completed: the QK that produced this S was issued after it.)
        const bool grow = tmax > m_ref + kRescaleThreshold || (m_ref == -INFINITY && tmax > -INFINITY);
        float factor = 1.f;
        if (grow) {
          factor = fast_exp2(m_ref - tmax);     // 0 when there was no reference yet
          m_ref = tmax;
          l_sum *= factor;
        }
        if (k > 0 && __any_sync(0xffffffffu, grow)) {
          uint32_t o[32];
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            tmem_ld32(tmem + lane_addr + kColO + w * kTileN + c * 32, o);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
            tmem_st32(tmem + lane_addr + kColO + w * kTileN + c * 32, o);
          }
          tc_wait_st();
        }
        // ---- pass 2: exponentials; packed bf16 P goes over score columns that have already been read
        const float neg_base = m_ref == -INFINITY ? 0.f : -m_ref;
        float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          load_half(h);
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(raw[2 * e]), p.scale_log2, neg_base));
            const float p1 = fast_exp2(fmaf(__uint_as_float(raw[2 * e + 1]), p.scale_log2, neg_base));
            const float p2 = fast_exp2(fmaf(__uint_as_float(raw[2 * e + 2]), p.scale_log2, neg_base));
            const float p3 = fast_exp2(fmaf(__uint_as_float(raw[2 * e + 3]), p.scale_log2, neg_base));
            ls[0] += p0; ls[1] += p1; ls[2] += p2; ls[3] += p3;
            raw[e] = pack_bf16(p0, p1);          // packed P overwrites entries already consumed
            raw[e + 1] = pack_bf16(p2, p3);
          }
          tmem_st32(s_addr + h * 32, raw);
        }
        l_sum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(B.p_full[w]);
      }
      if (!ok) break;

      // ---- epilogue
      if (steps > 0) {
        ok = mbar_wait_warp(B.o_done[w], (cws - 1) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
      }
      if (mode) {
        // two query tiles: each warpgroup owns its rows outright
        const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
        __nv_bfloat16* out_row = p.out + ((static_cast<size_t>(it.b) * p.T_max + node) * p.Hq + it.g * G + hh) * D;
        float* part_row = it.slot >= 0 ? p.part_o + (static_cast<size_t>(it.slot + w) * kBlockM + r) * D : nullptr;
        uint32_t o[32];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          tmem_ld32(tmem + lane_addr + kColO + w * kTileN + c * 32, o);
          tc_wait_ld();
          if (row_valid) {
            if (it.slot < 0) {
#pragma unroll
              for (int e = 0; e < 32; e += 8) {
                uint4 v;
                v.x = pack_bf16(__uint_as_float(o[e + 0]) * inv, __uint_as_float(o[e + 1]) * inv);
                v.y = pack_bf16(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
                v.z = pack_bf16(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
                v.w = pack_bf16(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
                *reinterpret_cast<uint4*>(out_row + c * 32 + e) = v;
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<uint4*>(part_row + c * 32 + e) = make_uint4(o[e], o[e + 1], o[e + 2], o[e + 3]);
            }
          }
        }
        if (row_valid && it.slot >= 0) p.part_ml[static_cast<size_t>(it.slot + w) * kBlockM + r] = make_float2(m_ref, l_sum);
      } else {
        // one query tile split over even / odd KV tiles: merge the two streams; warpgroup w writes half the columns
        float2* ml = reinterpret_cast<float2*>(smem + S::kMl);
        ml[w * kBlockM + r] = make_float2(m_ref, l_sum);
        mbar_arrive(B.ml_full);
        ok = mbar_wait_warp(B.ml_full, mode0_count & 1u, s_abort);
        ++mode0_count;
        if (!ok) break;
        tc_fence_after();
        const float2 mine = make_float2(m_ref, l_sum), other = ml[(w ^ 1) * kBlockM + r];
        const float2 a = w == 0 ? mine : other, bq = w == 0 ? other : mine;      // stream 0, stream 1
        const float m_star = fmaxf(a.y > 0.f ? a.x : -INFINITY, bq.y > 0.f ? bq.x : -INFINITY);
        const float wa = a.y > 0.f ? fast_exp2(a.x - m_star) : 0.f, wb = bq.y > 0.f ? fast_exp2(bq.x - m_star) : 0.f;
        const float l_star = a.y * wa + bq.y * wb;
        const float inv = l_star > 0.f ? 1.f / l_star : 0.f;
        const float fa = it.slot < 0 ? wa * inv : wa, fb = it.slot < 0 ? wb * inv : wb;
        constexpr int HALF = D / 2;
        __nv_bfloat16* out_row = p.out + ((static_cast<size_t>(it.b) * p.T_max + node) * p.Hq + it.g * G + hh) * D + w * HALF;
        float* part_row = it.slot >= 0 ? p.part_o + (static_cast<size_t>(it.slot) * kBlockM + r) * D + w * HALF : nullptr;
        uint32_t oa[32], ob[32];
#pragma unroll
        for (int c = 0; c < HALF / 32; ++c) {
          tmem_ld32(tmem + lane_addr + kColO + w * HALF + c * 32, oa);
          tmem_ld32(tmem + lane_addr + kColO + kTileN + w * HALF + c * 32, ob);
          tc_wait_ld();
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float xa = wa > 0.f ? __uint_as_float(oa[e]) * fa : 0.f;   // a stream without keys left its columns untouched
            const float xb = wb > 0.f ? __uint_as_float(ob[e]) * fb : 0.f;
            v[e] = xa + xb;
          }
          if (row_valid) {
            if (it.slot < 0) {
#pragma unroll
              for (int e = 0; e < 32; e += 8) {
                uint4 u;
                u.x = pack_bf16(v[e + 0], v[e + 1]);
                u.y = pack_bf16(v[e + 2], v[e + 3]);
                u.z = pack_bf16(v[e + 4], v[e + 5]);
                u.w = pack_bf16(v[e + 6], v[e + 7]);
                *reinterpret_cast<uint4*>(out_row + c * 32 + e) = u;
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<float4*>(part_row + c * 32 + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
            }
          }
        }
        if (row_valid && it.slot >= 0 && w == 0) p.part_ml[static_cast<size_t>(it.slot) * kBlockM + r] = make_float2(m_star, l_star);
      }
      tc_fence_before();
      mbar_arrive(B.o_free);
      g_base += nt;
      ++item_count;
    }
  }

  // ---- teardown: everyone arrives here (normally or after an abort); release TMEM
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) report_status(p.status, EAGLE_ERR_TIMEOUT);
  if (warp == 9) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// [B*Hkv, S_cap, D] bf16 viewed as a 3-D tensor (d, slot, sequence-head); box = 64 x 128 x 1, 128-byte swizzle.
bool make_kv_map(CUtensorMap* map, const void* base, int D, int S_cap, long long bh) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S_cap), static_cast<cuuint64_t>(bh)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(S_cap) * D * 2};
  const cuuint32_t box[3] = {64, kTileN, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int attn_tc2_tile_keys() { return kTileN; }

cudaError_t attn_tc2_prepare(int head_dim) {
  if (head_dim == 128)
    return cudaFuncSetAttribute(attn_tc2_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem2<128>::kBytes);
  return cudaFuncSetAttribute(attn_tc2_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem2<64>::kBytes);
}

// Returns cudaErrorInvalidValue when the tensor maps cannot be encoded.
cudaError_t launch_attn_tc2(const AttnParams& p, int num_ctas, cudaStream_t stream) {
  CUtensorMap mk, mv;
  const long long bh = static_cast<long long>(p.B) * p.Hkv;
  if (!make_kv_map(&mk, p.k, p.D, p.S_cap, bh) || !make_kv_map(&mv, p.v, p.D, p.S_cap, bh)) return cudaErrorInvalidValue;
  if (p.D == 128) attn_tc2_kernel<128><<<num_ctas, kThreads, Smem2<128>::kBytes, stream>>>(p, mk, mv);
  else attn_tc2_kernel<64><<<num_ctas, kThreads, Smem2<64>::kBytes, stream>>>(p, mk, mv);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
