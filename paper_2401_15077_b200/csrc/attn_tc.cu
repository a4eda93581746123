// Split-KV tree attention for sm_100a: TMA-staged KV tiles, tcgen05 tensor-core MMAs, accumulators in TMEM.
//
// One persistent CTA per SM walks a static slice of the planner's work list (items are sorted longest
// first; CTA c takes position c of every "row" of gridDim items, rows alternating direction, so the loads
// even out).  An item is a 128-row query tile (row = tree node * G + head-in-group) of one (sequence, KV
// head) over a range of 128-key KV tiles.  Warp roles:
//   warps 0-3  softmax + epilogue: thread r owns query row r (TMEM lane r): loads the S row with tcgen05.ld,
//              applies the tree mask in registers (only on tiles that reach past the committed prefix),
//              keeps the running max / sum in fp32 (log2 domain), writes P as packed bf16 back to TMEM
//   warp 4     TMA producer: K and V tiles through two 3-deep shared-memory rings (128B-swizzled boxes)
//   warp 5     MMA issuer: S = Q K^T (A, B from shared memory), O += P V (A = P from TMEM, B = V from
//              shared memory, MN-major), completion signalled with tcgen05.commit on mbarriers
// The output accumulator is rescaled only when the running max grows by more than 2^8 (the stale max is
// a valid softmax reference; the final division uses the same reference), so the common tile touches O
// only through the tensor core.
// Every wait is bounded: when one runs out the CTA raises EAGLE_ERR_TIMEOUT, all roles leave their loops,
// TMEM is released and the kernel returns.
#include <cuda.h>

#include "common.cuh"

namespace eagle {

namespace {

constexpr int kTileN = 128;          // keys per KV tile
constexpr int kStages = 3;           // K ring depth and V ring depth
constexpr int kThreads = 192;
constexpr int kSoftmaxThreads = 128;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;        // S0 at 0, S1 at 128
constexpr uint32_t kColO = 256;
constexpr uint32_t kColP = 384;      // P0 at 384, P1 at 448 (64 columns each: 128 bf16 per row)
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
struct Smem {
  static constexpr int kSlabs = D / 64;                     // 64 bf16 = one 128-byte swizzled row
  static constexpr int kSlabBytes = kTileN * 128;            // 128 rows x 128 bytes
  static constexpr int kTileBytes = kSlabs * kSlabBytes;     // one Q / K / V tile
  static constexpr int kQ = 0;
  static constexpr int kK = kTileBytes;
  static constexpr int kV = kK + kStages * kTileBytes;
  static constexpr int kBar = kV + kStages * kTileBytes;
  static constexpr int kNumBars = 4 * kStages + 2 + 2 + 2 + 2 + 1;
  static constexpr int kMisc = kBar + 8 * kNumBars;           // tmem base, abort flag
  static constexpr int kBytes = kMisc + 16;
  static constexpr int kAlloc = kBytes + 1024;                // slack to align the base to 1024 bytes
};

struct Bars {
  uint32_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint32_t s_full[2], p_full[2], o_done[2];
  uint32_t q_full, q_empty, o_free;
};

// Static work assignment: position of this CTA in row `row` of the sorted item list (rows alternate direction).
__device__ __forceinline__ int item_index(int row, int cta, int grid) {
  return row * grid + ((row & 1) ? (grid - 1 - cta) : cta);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(AttnParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  using S = Smem<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  Bars B;
  {
    uint32_t b = sbase + S::kBar;
    for (int i = 0; i < kStages; ++i) { B.k_full[i] = b; b += 8; }
    for (int i = 0; i < kStages; ++i) { B.k_empty[i] = b; b += 8; }
    for (int i = 0; i < kStages; ++i) { B.v_full[i] = b; b += 8; }
    for (int i = 0; i < kStages; ++i) { B.v_empty[i] = b; b += 8; }
    for (int i = 0; i < 2; ++i) { B.s_full[i] = b; b += 8; }
    for (int i = 0; i < 2; ++i) { B.p_full[i] = b; b += 8; }
    for (int i = 0; i < 2; ++i) { B.o_done[i] = b; b += 8; }
    B.q_full = b; b += 8;
    B.q_empty = b; b += 8;
    B.o_free = b;
  }
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + S::kMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + S::kMisc + 4);

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(B.k_full[i], 1);
      mbar_init(B.k_empty[i], 1);
      mbar_init(B.v_full[i], 1);
      mbar_init(B.v_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(B.s_full[i], 1);
      mbar_init(B.p_full[i], kSoftmaxThreads);
      mbar_init(B.o_done[i], 1);
    }
    mbar_init(B.q_full, kSoftmaxThreads);
    mbar_init(B.q_empty, 1);
    mbar_init(B.o_free, kSoftmaxThreads);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + S::kMisc), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  const int n_items = p.hdr->n_items;
  const int grid = gridDim.x, cta = blockIdx.x;

  if (warp == 4) {
    // =========================================================================== TMA producer
    if (lane == 0) {
      uint32_t t = 0;   // KV tiles issued by this CTA so far
      bool ok = true;
      for (int row = 0; ok; ++row) {
        const int idx = item_index(row, cta, grid);
        if (idx >= n_items) break;
        const WorkItem it = p.items[idx];
        const int z = it.b * p.Hkv + it.g;
        for (int tile = it.tile_begin; tile < it.tile_end && ok; ++tile, ++t) {
          const uint32_t st = t % kStages, par = ((t / kStages) & 1u) ^ 1u;
          ok = mbar_wait(B.k_empty[st], par, s_abort);
          if (!ok) break;
          mbar_expect_tx(B.k_full[st], S::kTileBytes);
#pragma unroll
          for (int s = 0; s < S::kSlabs; ++s)
            tma_load_3d(sbase + S::kK + st * S::kTileBytes + s * S::kSlabBytes, &map_k, s * 64, tile * kTileN, z, B.k_full[st]);
          ok = mbar_wait(B.v_empty[st], par, s_abort);
          if (!ok) break;
          mbar_expect_tx(B.v_full[st], S::kTileBytes);
#pragma unroll
          for (int s = 0; s < S::kSlabs; ++s)
            tma_load_3d(sbase + S::kV + st * S::kTileBytes + s * S::kSlabBytes, &map_v, s * 64, tile * kTileN, z, B.v_full[st]);
        }
      }
    }
  } else if (warp == 5) {
    // =========================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kBlockM, kTileN, false);
      constexpr uint32_t idesc_pv = instr_desc(kBlockM, D, true);
      uint32_t t = 0;          // global tile counter
      uint32_t item_count = 0;
      bool ok = true;
      auto issue_qk = [&](uint32_t tt) -> bool {
        const uint32_t st = tt % kStages, par = (tt / kStages) & 1u;
        if (!mbar_wait(B.k_full[st], par, s_abort)) return false;
        tc_fence_after();
        const uint32_t d_tmem = tmem + kColS + (tt & 1u) * kTileN;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk / 4) * S::kSlabBytes + (kk % 4) * 32;
          umma_ss(d_tmem, smem_desc(sbase + S::kQ + off, 16), smem_desc(sbase + S::kK + st * S::kTileBytes + off, 16), idesc_qk,
                  kk > 0 ? 1u : 0u);
        }
        tc_commit(B.k_empty[st]);
        tc_commit(B.s_full[tt & 1u]);
        return true;
      };
      for (int row = 0; ok; ++row) {
        const int idx = item_index(row, cta, grid);
        if (idx >= n_items) break;
        const WorkItem it = p.items[idx];
        const int nt = it.tile_end - it.tile_begin;
        ok = mbar_wait(B.q_full, item_count & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        ok = issue_qk(t);
        if (ok && nt == 1) tc_commit(B.q_empty);
        for (int j = 0; j < nt && ok; ++j) {
          const uint32_t tt = t + j;
          if (j + 1 < nt) {
            ok = issue_qk(tt + 1);
            if (!ok) break;
            if (j + 2 == nt) tc_commit(B.q_empty);   // every QK of this item has been issued
          }
          ok = mbar_wait(B.p_full[tt & 1u], (tt >> 1) & 1u, s_abort);
          if (!ok) break;
          const uint32_t st = tt % kStages, par = (tt / kStages) & 1u;
          ok = mbar_wait(B.v_full[st], par, s_abort);
          if (!ok) break;
          if (j == 0 && item_count > 0) {
            ok = mbar_wait(B.o_free, (item_count - 1) & 1u, s_abort);   // previous epilogue has read O
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t a_tmem = tmem + kColP + (tt & 1u) * (kTileN / 2);
#pragma unroll
          for (int kk = 0; kk < kTileN / 16; ++kk) {
            umma_ts(tmem + kColO, a_tmem + kk * 8, smem_desc(sbase + S::kV + st * S::kTileBytes + kk * 2048, S::kSlabBytes), idesc_pv,
                    (j > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(B.v_empty[st]);
          tc_commit(B.o_done[tt & 1u]);
        }
        t += nt;
        ++item_count;
      }
    }
  } else {
    // =========================================================================== softmax + epilogue
    const int r = tid;                                    // query row of this thread == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
    uint32_t t = 0, item_count = 0;
    bool ok = true;
    for (int row = 0; ok; ++row) {
      const int idx = item_index(row, cta, grid);
      if (idx >= n_items) break;
      const WorkItem it = p.items[idx];
      const SeqPlan sp = p.seq[it.b];
      const int L = sp.L, n = sp.n, G = p.G;
      const int m_valid = n * G, R = it.mt * kBlockM + r;
      const bool row_valid = R < m_valid;
      const int node = row_valid ? R / G : 0, hh = row_valid ? R % G : 0;
      const uint64_t anc = row_valid ? p.anc[static_cast<size_t>(it.b) * p.T_max + node] : 0ull;
      const int kv_end = L + n;
      const int nt = it.tile_end - it.tile_begin;

      // ---- stage Q: row r, 128-byte swizzled slabs of 64 columns
      ok = mbar_wait_warp(B.q_empty, (item_count & 1u) ^ 1u, s_abort);
      if (!ok) break;
      {
        const uint4* src = reinterpret_cast<const uint4*>(p.q + ((static_cast<size_t>(it.b) * p.T_max + node) * p.Hq + it.g * G + hh) * D);
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
          const uint4 v = row_valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
          const uint32_t off = (c / 8) * S::kSlabBytes + r * 128 + (((c % 8) ^ (r & 7)) << 4);
          *reinterpret_cast<uint4*>(smem + S::kQ + off) = v;
        }
      }
      fence_proxy_async();
      mbar_arrive(B.q_full);

      float m_ref = -INFINITY;   // reference max (log2 domain) used for every exponential so far
      float l_sum = 0.f;
      for (int j = 0; j < nt && ok; ++j) {
        const uint32_t tt = t + j;
        const uint32_t buf = tt & 1u;
        ok = mbar_wait_warp(B.s_full[buf], (tt >> 1) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        float s[kTileN];
        {
          uint32_t raw[kTileN];
#pragma unroll
          for (int c = 0; c < kTileN / 32; ++c) tmem_ld32(tmem + lane_addr + kColS + buf * kTileN + c * 32, raw + c * 32);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < kTileN; ++e) s[e] = __uint_as_float(raw[e]) * p.scale_log2;
        }
        const int key0 = (it.tile_begin + j) * kTileN;
        if (key0 + kTileN > L) {          // the tile reaches past the committed prefix: tree mask + cache tail
#pragma unroll
          for (int e = 0; e < kTileN; ++e) {
            const int mrel = key0 + e - L;
            const bool vis = mrel < 0 || (mrel < n && ((anc >> mrel) & 1ull));
            s[e] = vis ? s[e] : -INFINITY;
          }
        }
        float tmax = s[0];
#pragma unroll
        for (int e = 1; e < kTileN; ++e) tmax = fmaxf(tmax, s[e]);

        // P buffer of this parity is free once PV(tt-2) has completed
        if (tt >= 2) {
          ok = mbar_wait_warp(B.o_done[buf], ((tt - 2) >> 1) & 1u, s_abort);
          if (!ok) break;
        }
        if (key0 + kTileN > kv_end) {
          // rows of the V tile past prefix + tree may hold anything: zero them so that 0 * garbage cannot reach O
          const uint32_t st = tt % kStages, par = (tt / kStages) & 1u;
          ok = mbar_wait_warp(B.v_full[st], par, s_abort);
          if (!ok) break;
          if (key0 + r >= kv_end) {
#pragma unroll
            for (int sl = 0; sl < S::kSlabs; ++sl)
#pragma unroll
              for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(smem + S::kV + st * S::kTileBytes + sl * S::kSlabBytes + r * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();
        }

        // lazy rescale: move the reference only when the row max outgrows it by more than the threshold
        const bool grow = tmax > m_ref + kRescaleThreshold || (m_ref == -INFINITY && tmax > -INFINITY);
        float factor = 1.f;
        if (grow) {
          factor = exp2f(m_ref - tmax);     // 0 when there was no reference yet
          m_ref = tmax;
          l_sum *= factor;
        }
        if (j > 0 && __any_sync(0xffffffffu, grow)) {
          ok = mbar_wait_warp(B.o_done[(tt - 1) & 1u], ((tt - 1) >> 1) & 1u, s_abort);
          if (!ok) break;
          tc_fence_after();
          uint32_t raw[32];
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            tmem_ld32(tmem + lane_addr + kColO + c * 32, raw);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) raw[e] = __float_as_uint(__uint_as_float(raw[e]) * factor);
            tmem_st32(tmem + lane_addr + kColO + c * 32, raw);
          }
          tc_wait_st();
        }
        const float base = m_ref == -INFINITY ? 0.f : m_ref;
        {
          uint32_t packed[32];
#pragma unroll
          for (int c = 0; c < kTileN / 64; ++c) {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const float p0 = fast_exp2(s[c * 64 + 2 * e] - base), p1 = fast_exp2(s[c * 64 + 2 * e + 1] - base);
              l_sum += p0 + p1;
              packed[e] = pack_bf16(p0, p1);
            }
            tmem_st32(tmem + lane_addr + kColP + buf * (kTileN / 2) + c * 32, packed);
          }
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(B.p_full[buf]);
      }
      if (!ok) break;

      // ---- epilogue: wait for the last PV, read O, write output rows or the split partial
      {
        const uint32_t tl = t + nt - 1;
        ok = mbar_wait_warp(B.o_done[tl & 1u], (tl >> 1) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after();
        const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
        __nv_bfloat16* out_row = p.out + ((static_cast<size_t>(it.b) * p.T_max + node) * p.Hq + it.g * G + hh) * D;
        float* part_row = it.slot >= 0 ? p.part_o + (static_cast<size_t>(it.slot) * kBlockM + r) * D : nullptr;
        uint32_t raw[32];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          tmem_ld32(tmem + lane_addr + kColO + c * 32, raw);
          tc_wait_ld();
          if (row_valid) {
            if (it.slot < 0) {
#pragma unroll
              for (int e = 0; e < 32; e += 8) {
                uint4 v;
                v.x = pack_bf16(__uint_as_float(raw[e + 0]) * inv, __uint_as_float(raw[e + 1]) * inv);
                v.y = pack_bf16(__uint_as_float(raw[e + 2]) * inv, __uint_as_float(raw[e + 3]) * inv);
                v.z = pack_bf16(__uint_as_float(raw[e + 4]) * inv, __uint_as_float(raw[e + 5]) * inv);
                v.w = pack_bf16(__uint_as_float(raw[e + 6]) * inv, __uint_as_float(raw[e + 7]) * inv);
                *reinterpret_cast<uint4*>(out_row + c * 32 + e) = v;
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<uint4*>(part_row + c * 32 + e) = make_uint4(raw[e], raw[e + 1], raw[e + 2], raw[e + 3]);
            }
          }
        }
        if (row_valid && it.slot >= 0) p.part_ml[static_cast<size_t>(it.slot) * kBlockM + r] = make_float2(m_ref, l_sum);
        tc_fence_before();
        mbar_arrive(B.o_free);
      }
      t += nt;
      ++item_count;
    }
  }

  // ---- teardown: everyone arrives here (normally or after an abort); release TMEM
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) report_status(p.status, EAGLE_ERR_TIMEOUT);
  if (warp == 5) {
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

int attn_tc_tile_keys() { return kTileN; }

cudaError_t attn_tc_prepare(int head_dim) {
  if (head_dim == 128)
    return cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128>::kAlloc);
  return cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<64>::kAlloc);
}

// Returns cudaErrorInvalidValue when the tensor maps cannot be encoded.
cudaError_t launch_attn_tc(const AttnParams& p, int num_ctas, cudaStream_t stream) {
  CUtensorMap mk, mv;
  const long long bh = static_cast<long long>(p.B) * p.Hkv;
  if (!make_kv_map(&mk, p.k, p.D, p.S_cap, bh) || !make_kv_map(&mv, p.v, p.D, p.S_cap, bh)) return cudaErrorInvalidValue;
  if (p.D == 128) attn_tc_kernel<128><<<num_ctas, kThreads, Smem<128>::kAlloc, stream>>>(p, mk, mv);
  else attn_tc_kernel<64><<<num_ctas, kThreads, Smem<64>::kAlloc, stream>>>(p, mk, mv);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
