// Split-KV tree attention, register-accumulator variant (mma.sync m16n8k16, cp.async staging).
//
// A persistent CTA (8 warps) pulls work items from the planner's list.  An item is a 128-row query tile
// (row r = node i * G + head-in-group) of one (sequence, KV head) over a range of 64-key KV tiles.
// Each warp owns 16 rows: S = Q K^T with tensor-core MMAs, an fp32 online softmax in the log2 domain with
// the tree mask applied in registers (only on tiles that reach past the committed prefix), O += P V.
// An item that covers the whole KV range writes bf16 output rows; otherwise it writes an (m, l, O) partial.
#include "common.cuh"

namespace eagle {

namespace {

constexpr int kThreads = 256;
constexpr int kTileN = 64;
constexpr int kStages = 3;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;  // src-size 0: the 16 bytes are zero-filled, nothing is read
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Row-major tile of rows x D bf16, 16-byte chunks XOR-swizzled by (row & 7) so that ldmatrix is conflict free.
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return static_cast<uint32_t>(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) attn_mma_kernel(AttnParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int CH = D / 8;                 // 16-byte chunks per row
  constexpr int Q_BYTES = kBlockM * D * 2;
  constexpr int KV_BYTES = kTileN * D * 2;
  unsigned char* sQ = smem;
  unsigned char* sK = smem + Q_BYTES;
  unsigned char* sV = sK + kStages * KV_BYTES;
  __shared__ int s_item;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_items = p.hdr->n_items;

  for (;;) {
    __syncthreads();  // previous item's smem reads and s_item read are done
    if (tid == 0) s_item = atomicAdd(&p.hdr->next_item, 1);
    __syncthreads();
    const int item_idx = s_item;
    if (item_idx >= n_items) break;
    const WorkItem it = p.items[item_idx];
    const SeqPlan sp = p.seq[it.b];
    const int L = sp.L, n = sp.n, G = p.G;
    const int m_valid = n * G;
    const int row0 = it.mt * kBlockM;
    const int kv_end = L + n;
    const size_t kv_base = (static_cast<size_t>(it.b) * p.Hkv + it.g) * static_cast<size_t>(p.S_cap) * D;
    const __nv_bfloat16* kg = p.k + kv_base;
    const __nv_bfloat16* vg = p.v + kv_base;

    // ---- stage Q (rows past the tree are zero-filled)
    for (int c = tid; c < kBlockM * CH; c += kThreads) {
      const int r = c / CH, ch = c % CH;
      const int R = row0 + r;
      const bool valid = R < m_valid;
      const int i = valid ? R / G : 0, hh = valid ? R % G : 0;
      const __nv_bfloat16* src = p.q + ((static_cast<size_t>(it.b) * p.T_max + i) * p.Hq + it.g * G + hh) * D + ch * 8;
      cp_async16(smem_u32(sQ + tile_off<D>(r, ch)), src, valid);
    }
    cp_async_commit();

    auto load_kv = [&](int tile, int stage) {
      const int key0 = tile * kTileN;
      for (int c = tid; c < kTileN * CH; c += kThreads) {
        const int r = c / CH, ch = c % CH;
        const int key = key0 + r;
        const bool valid = key < kv_end;   // slots past prefix + tree are never read
        const size_t off = static_cast<size_t>(valid ? key : 0) * D + ch * 8;
        cp_async16(smem_u32(sK + stage * KV_BYTES + tile_off<D>(r, ch)), kg + off, valid);
        cp_async16(smem_u32(sV + stage * KV_BYTES + tile_off<D>(r, ch)), vg + off, valid);
      }
    };
    const int t0 = it.tile_begin, t1 = it.tile_end;
    for (int s = 0; s < kStages - 1; ++s) {
      if (t0 + s < t1) load_kv(t0 + s, s);
      cp_async_commit();
    }

    // rows of this thread: rA = 16*warp + lane/4, rB = rA + 8
    const int rA = warp * 16 + (lane >> 2), rB = rA + 8;
    const bool warp_active = row0 + warp * 16 < m_valid;
    uint64_t ancA = 0, ancB = 0;
    if (row0 + rA < m_valid) ancA = p.anc[static_cast<size_t>(it.b) * p.T_max + (row0 + rA) / G];
    if (row0 + rB < m_valid) ancB = p.anc[static_cast<size_t>(it.b) * p.T_max + (row0 + rB) / G];

    float o[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
    uint32_t qf[D / 16][4];
    bool q_loaded = false;

    for (int t = t0; t < t1; ++t) {
      const int stage = (t - t0) % kStages;
      cp_async_wait<kStages - 2>();
      __syncthreads();  // tile t (and Q) landed for everyone; the stage refilled below was consumed by everyone
      {
        const int tn = t + kStages - 1;
        if (tn < t1) load_kv(tn, (tn - t0) % kStages);
        cp_async_commit();
      }
      if (!warp_active) continue;
      if (!q_loaded) {
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          ldsm_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], smem_u32(sQ + tile_off<D>(r, ks * 2 + (lane >> 4))));
        }
        q_loaded = true;
      }
      const unsigned char* kS = sK + stage * KV_BYTES;
      const unsigned char* vS = sV + stage * KV_BYTES;

      // ---- S = Q K^T  (16 x 64 per warp)
      float s[kTileN / 8][4];
#pragma unroll
      for (int j = 0; j < kTileN / 8; ++j) {
        s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < D / 16; ks += 2) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(b0, b1, b2, b3, smem_u32(kS + tile_off<D>(j * 8 + (lane & 7), ks * 2 + (lane >> 3))));
          mma_bf16(s[j], qf[ks], b0, b1);
          mma_bf16(s[j], qf[ks + 1], b2, b3);
        }
      }

      // ---- scale, tree mask (only where the tile reaches past the prefix), online softmax
      const int key0 = t * kTileN;
      const bool need_mask = key0 + kTileN > L;
      float tmaxA = -INFINITY, tmaxB = -INFINITY;
#pragma unroll
      for (int j = 0; j < kTileN / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float x = s[j][e] * p.scale_log2;
          if (need_mask) {
            const int key = key0 + j * 8 + (lane & 3) * 2 + (e & 1);
            const int m = key - L;
            const uint64_t anc = (e < 2) ? ancA : ancB;
            const bool vis = m < 0 || (m < n && ((anc >> m) & 1ull));
            x = vis ? x : -INFINITY;
          }
          s[j][e] = x;
        }
        tmaxA = fmaxf(tmaxA, fmaxf(s[j][0], s[j][1]));
        tmaxB = fmaxf(tmaxB, fmaxf(s[j][2], s[j][3]));
      }
      tmaxA = fmaxf(tmaxA, __shfl_xor_sync(0xffffffffu, tmaxA, 1));
      tmaxA = fmaxf(tmaxA, __shfl_xor_sync(0xffffffffu, tmaxA, 2));
      tmaxB = fmaxf(tmaxB, __shfl_xor_sync(0xffffffffu, tmaxB, 1));
      tmaxB = fmaxf(tmaxB, __shfl_xor_sync(0xffffffffu, tmaxB, 2));
      const float mA_new = fmaxf(mA, tmaxA), mB_new = fmaxf(mB, tmaxB);
      const float baseA = mA_new == -INFINITY ? 0.f : mA_new;   // fully masked so far: avoid inf - inf
      const float baseB = mB_new == -INFINITY ? 0.f : mB_new;
      const float corrA = exp2f(mA - baseA), corrB = exp2f(mB - baseB);
      mA = mA_new;
      mB = mB_new;
      lA *= corrA;
      lB *= corrB;
#pragma unroll
      for (int j = 0; j < D / 8; ++j) {
        o[j][0] *= corrA;
        o[j][1] *= corrA;
        o[j][2] *= corrB;
        o[j][3] *= corrB;
      }
      uint32_t pf[kTileN / 16][4];
#pragma unroll
      for (int j = 0; j < kTileN / 8; ++j) {
        const float p0 = exp2f(s[j][0] - baseA), p1 = exp2f(s[j][1] - baseA);
        const float p2 = exp2f(s[j][2] - baseB), p3 = exp2f(s[j][3] - baseB);
        lA += p0 + p1;
        lB += p2 + p3;
        pf[j >> 1][(j & 1) * 2 + 0] = pack_bf16(p0, p1);
        pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
      }

      // ---- O += P V
#pragma unroll
      for (int kk = 0; kk < kTileN / 16; ++kk) {
#pragma unroll
        for (int j = 0; j < D / 8; j += 2) {
          uint32_t b0, b1, b2, b3;
          const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          ldsm_x4_t(b0, b1, b2, b3, smem_u32(vS + tile_off<D>(key, j + (lane >> 4))));
          mma_bf16(o[j], pf[kk], b0, b1);
          mma_bf16(o[j + 1], pf[kk], b2, b3);
        }
      }
    }
    cp_async_wait<0>();

    if (!warp_active) continue;
    // ---- epilogue
    lA += __shfl_xor_sync(0xffffffffu, lA, 1);
    lA += __shfl_xor_sync(0xffffffffu, lA, 2);
    lB += __shfl_xor_sync(0xffffffffu, lB, 1);
    lB += __shfl_xor_sync(0xffffffffu, lB, 2);
    const int RA = row0 + rA, RB = row0 + rB;
    if (it.slot < 0) {
      const float invA = lA > 0.f ? 1.f / lA : 0.f, invB = lB > 0.f ? 1.f / lB : 0.f;
      if (RA < m_valid) {
        __nv_bfloat16* dst = p.out + ((static_cast<size_t>(it.b) * p.T_max + RA / G) * p.Hq + it.g * G + RA % G) * D;
#pragma unroll
        for (int j = 0; j < D / 8; ++j)
          *reinterpret_cast<uint32_t*>(dst + j * 8 + (lane & 3) * 2) = pack_bf16(o[j][0] * invA, o[j][1] * invA);
      }
      if (RB < m_valid) {
        __nv_bfloat16* dst = p.out + ((static_cast<size_t>(it.b) * p.T_max + RB / G) * p.Hq + it.g * G + RB % G) * D;
#pragma unroll
        for (int j = 0; j < D / 8; ++j)
          *reinterpret_cast<uint32_t*>(dst + j * 8 + (lane & 3) * 2) = pack_bf16(o[j][2] * invB, o[j][3] * invB);
      }
    } else {
      float* po = p.part_o + static_cast<size_t>(it.slot) * kBlockM * D;
      float2* pml = p.part_ml + static_cast<size_t>(it.slot) * kBlockM;
      if (RA < m_valid) {
#pragma unroll
        for (int j = 0; j < D / 8; ++j)
          *reinterpret_cast<float2*>(po + static_cast<size_t>(rA) * D + j * 8 + (lane & 3) * 2) = make_float2(o[j][0], o[j][1]);
        if ((lane & 3) == 0) pml[rA] = make_float2(mA, lA);
      }
      if (RB < m_valid) {
#pragma unroll
        for (int j = 0; j < D / 8; ++j)
          *reinterpret_cast<float2*>(po + static_cast<size_t>(rB) * D + j * 8 + (lane & 3) * 2) = make_float2(o[j][2], o[j][3]);
        if ((lane & 3) == 0) pml[rB] = make_float2(mB, lB);
      }
    }
  }
}

template <int D>
constexpr int smem_bytes() { return kBlockM * D * 2 + 2 * kStages * kTileN * D * 2; }

}  // namespace

int attn_mma_tile_keys() { return kTileN; }
int attn_mma_ctas_per_sm(int) { return 1; }

cudaError_t attn_mma_prepare(int head_dim) {
  if (head_dim == 128)
    return cudaFuncSetAttribute(attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<128>());
  return cudaFuncSetAttribute(attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<64>());
}

cudaError_t launch_attn_mma(const AttnParams& p, int num_ctas, cudaStream_t stream) {
  if (p.D == 128) attn_mma_kernel<128><<<num_ctas, kThreads, smem_bytes<128>(), stream>>>(p);
  else attn_mma_kernel<64><<<num_ctas, kThreads, smem_bytes<64>(), stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
