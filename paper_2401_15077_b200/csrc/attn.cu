// Split-KV tree attention for sm_100a: TMA-staged KV tiles, tcgen05 MMAs, accumulators in TMEM.
//
// One persistent CTA per SM; CTAs 2j and 2j+1 form a team that walks its share of the planner's work list.  An
// item is one 128-row query tile (row = tree node * G + head-in-group) of one (sequence, KV head) over a range of
// 128-key KV tiles; step g (counted over all of the CTA's items) handles one KV tile:
//     S[g % 3] = Q K^T   ->   softmax   ->   P (packed bf16, written over the front of S[g % 3])   ->   O += P V.
// Tensor memory holds three score buffers and the accumulator (S0 S1 S2 | O = 512 columns).  The score MMA of
// step g + 3 is issued as soon as the PV MMA of step g has released its buffer, so up to three score tiles are in
// flight and the MMAs never wait for the softmax of the step before them.
// Warp roles: warps 0-7 softmax, as two groups of four warps that take alternate steps (one query row = one
// TMEM lane per thread, all 128 score columns), so that one group computes while the other waits; warp 8 K/V
// producer (TMA, 128-byte swizzled boxes, ring of six 32 KB slots, tiles requested in the order the MMAs consume
// them); warp 9 issues the QK MMAs (and fetches the query tile of the next item once the last score MMA of the
// current one has finished), warp 10 the PV MMAs.  The group that takes an item's last step writes its output
// while the other group is already on the next item.  Softmax is fp32 in the log2 domain with two-wide FP32
// instructions; part of the exponentials is a polynomial on the FMA pipe.  The tree mask is applied only on tiles
// that reach past the committed prefix, by a pre-pass that writes -inf over the invisible scores in tensor memory;
// rows of a V tile past prefix + tree are zeroed in shared memory before the MMA reads them.  The accumulator is
// rescaled only when the row maximum outgrows the shared reference by more than 2^8.  Every wait is bounded
// (mbarrier try_wait + timer, or a bounded spin on a tagged word); on expiry the CTA raises EAGLE_ERR_TIMEOUT, all
// roles leave their loops, TMEM is released and the kernel returns.
// Instantiations: PAGED (the K/V producer gathers a tile page by page through a block table), FP8, or both (the cache holds
// e4m3 codes: tiles of codes land in a staging ring, four more warps widen them exactly into a ring of four fp16
// slots and the MMAs run fp16 x fp16; the scales go into the softmax scale and the output).
#include <cuda.h>

#include "common.cuh"

namespace eagle {

namespace {

constexpr int kTileN = 128;          // keys per KV tile
// Ring slots of K/V tiles; entry n of the load sequence (see the producer) uses slot n % slots.  A cache stored as fp8
// codes has four slots of fp16 tiles plus four staging slots of raw codes instead of six slots.
template <bool FP8>
constexpr int slots_of() { return FP8 ? 4 : 6; }
constexpr int kSBufs = 3;            // score buffers in tensor memory; step g uses buffer g % 3
constexpr int kThreads = 352;          // 8 softmax warps, K/V producer, two MMA issuers: 186 registers for every thread
constexpr int kConvWarps = 4;           // fp8 cache: warps that widen tiles of codes to fp16 tiles
constexpr int kThreadsFp8 = kThreads + 32 * kConvWarps;   // (a fifth warp per scheduler: 128 registers for every thread)
constexpr int kWarpConvert = 11;
constexpr int kSoftmaxWarps = 8;
constexpr int kGroupThreads = 128;     // one softmax group
constexpr int kWarpProducer = 8, kWarpQK = 9, kWarpPV = 10;
// One pair of exponentials in three goes through the polynomial.  The softmax loop runs at the register limit (three
// warps per scheduler: 168 registers): a variant that spills even a few values is a fifth slower, and shares of 1/4 and
// below (more exponentials in flight on the special-function unit) or 1/2 with the masking code in the loop did.
#ifndef EAGLE_POLY_STRIDE
#define EAGLE_POLY_STRIDE 3
#endif
constexpr int kPolyStride = EAGLE_POLY_STRIDE;   // one pair of exponentials in kPolyStride is evaluated as a polynomial (0: none)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;        // S[b] at b*128; P[b] (packed bf16, 64 columns) overwrites the front of S[b]
constexpr uint32_t kColO = 384;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

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
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// (A wait gives up only after the time limit has passed without progress, two seconds unless the host changed it, and
// never less than far longer than a copy takes; the K/V ring holds at most six tiles, so by then the producers have been
// blocked for all but the first microseconds of that time and no copy of theirs is still in flight when the CTA leaves.)
// The limit sits in shared memory right after the abort flag, so the wait sites pass one pointer.
__device__ __forceinline__ unsigned long long wait_limit_of(volatile int* abort_flag) {
  return *reinterpret_cast<volatile unsigned long long*>(abort_flag + 1);
}
// Slow path of a wait, kept out of line so that the dozen wait sites stay small (the kernel's hot loops have to
// live in the instruction cache next to each other).  Returns false if the CTA has been aborted or the time limit
// passed (and raises the abort flag).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  const unsigned long long t0 = global_timer();
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 63u) == 0) {
      if (*abort_flag) return false;
      if (global_timer() - t0 > wait_limit_of(abort_flag)) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}
// Bounded wait: a few non-blocking probes (most phases are complete, or complete within a few hundred cycles),
// then the suspending form with the timer.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
#pragma unroll 1
  for (int i = 0; i < 16; ++i)
    if (mbar_test_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag);
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

__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Packed pairs of floats (one 64-bit register) and the two-wide FP32 instructions of sm_100: one issue slot does the
// work of two, which matters because the softmax is bound by instruction issue, not by any single pipe.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x for a packed pair on the FMA / ALU pipes (x <= ~8): split x into an integer n and a fraction f in [-0.5, 0.5]
// with the add-a-large-constant trick, evaluate a cubic for 2^f (relative error 1e-4, far below the bf16 rounding of
// P) and put n into the exponent field.  Used for a fraction of the exponentials so that the special-function
// unit, which takes 8 cycles per warp instruction, is not the only thing the softmax waits for.
__device__ __forceinline__ void poly_exp2_pair(uint64_t x2, float& p0, float& p1) {
  float a, b;
  unpack2(x2, a, b);
  const uint64_t xc2 = pack2(fmaxf(a, -126.f), fmaxf(b, -126.f));
  const uint64_t t2 = add2(xc2, pack2(12582912.f, 12582912.f));
  const uint64_t u2 = add2(t2, pack2(-12582912.f, -12582912.f));
  const uint64_t f2 = fma2(u2, pack2(-1.f, -1.f), xc2);
  uint64_t r2 = fma2(pack2(0.05500841f, 0.05500841f), f2, pack2(0.24220926f, 0.24220926f));
  r2 = fma2(r2, f2, pack2(0.69328277f, 0.69328277f));
  r2 = fma2(r2, f2, pack2(1.0f, 1.0f));
  float ta, tb, ra, rb;
  unpack2(t2, ta, tb);
  unpack2(r2, ra, rb);
  p0 = __uint_as_float(__float_as_uint(ta) * 0x800000u + __float_as_uint(ra));   // the constant's own bits shift out
  p1 = __uint_as_float(__float_as_uint(tb) * 0x800000u + __float_as_uint(rb));
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Bounded wait for a tagged word in shared memory (low byte == want).  The word comes back by value, with bit 32 set on
// success (0: the CTA was aborted or the time limit passed); nothing is passed through memory.
__device__ __noinline__ unsigned long long tag_wait_slow(volatile uint32_t* slot, uint32_t want, volatile int* abort_flag) {
  const unsigned long long t0 = global_timer();
  for (uint32_t spins = 1;; ++spins) {
    const uint32_t t = *slot;
    if ((t & 0xffu) == want) return (1ull << 32) | t;
    if ((spins & 255u) == 0) {
      if (*abort_flag) return 0ull;
      if (global_timer() - t0 > wait_limit_of(abort_flag)) {
        *abort_flag = 1;
        return 0ull;
      }
    }
  }
}
__device__ __forceinline__ unsigned long long tag_wait(volatile uint32_t* slot, uint32_t want, volatile int* abort_flag) {
#pragma unroll 1
  for (int i = 0; i < 8; ++i) {
    const uint32_t t = *slot;
    if ((t & 0xffu) == want) return (1ull << 32) | t;
  }
  return tag_wait_slow(slot, want, abort_flag);
}

// One 32-byte store (the address must be 32-byte aligned).
__device__ __forceinline__ void st_global_v8(void* dst, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]),
               "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// kind::f16 instruction descriptor: bf16 x bf16 (or fp16 x fp16: both operands have one type) -> fp32, A K-major,
// B K-major or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major, bool fp16 = false) {
  return (1u << 4) | (fp16 ? 0u : (1u << 7) | (1u << 10)) | (b_mn_major ? (1u << 16) : 0u) |
         (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}


// Descriptor halves.  The low word holds the start address (>>4) and the leading-dimension offset, so stepping along
// the contraction is a 32-bit add on the low word; the high word (8-row-group stride, version, swizzle) is constant.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) { return ((addr >> 4) & 0x3fffu) | ((lbo_bytes >> 4) << 16); }
// One asm block per 128-key tile: the MMAs of a tile are issued back to back by one thread, so the instruction
// stream between them is kept to the descriptor adds (the tensor pipe finishes a 128x128x16 MMA in about 64 cycles).
// S[128 x 128] = Q[128 x D] K^T: D/16 MMAs; low descriptor words step 32 bytes per k step, 16 KB per 64-column slab.
template <int D>
__device__ __forceinline__ void issue_qk_tile(uint32_t d_tmem, uint32_t q_lo, uint32_t k_lo, uint32_t idesc) {
  if constexpr (D == 128) {
    asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb;\n\t"
      "add.u32 ta, %1, 0;\n\tadd.u32 tb, %2, 0;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 1024;\n\tadd.u32 tb, %2, 1024;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 1026;\n\tadd.u32 tb, %2, 1026;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 1028;\n\tadd.u32 tb, %2, 1028;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 1030;\n\tadd.u32 tb, %2, 1030;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "}"
      ::"r"(d_tmem), "r"(q_lo), "r"(k_lo), "r"(idesc), "r"(kDescHi) : "memory");
  } else {
    asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb;\n\t"
      "add.u32 ta, %1, 0;\n\tadd.u32 tb, %2, 0;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
      "}"
      ::"r"(d_tmem), "r"(q_lo), "r"(k_lo), "r"(idesc), "r"(kDescHi) : "memory");
  }
}
// O[128 x D] (+)= P[128 x 128] V[128 x D]: 8 MMAs; P steps 8 TMEM columns, V steps 16 keys (2 KB) per k step.
__device__ __forceinline__ void issue_pv_tile(uint32_t o_tmem, uint32_t p_tmem, uint32_t v_lo, uint32_t idesc, uint32_t acc0) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t.reg .b32 ta, tb;\n\t"
      "add.u32 ta, %1, 0;\n\tadd.u32 tb, %2, 0;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, %5, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "add.u32 ta, %1, 8;\n\tadd.u32 tb, %2, 128;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "add.u32 ta, %1, 16;\n\tadd.u32 tb, %2, 256;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "add.u32 ta, %1, 24;\n\tadd.u32 tb, %2, 384;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "add.u32 ta, %1, 32;\n\tadd.u32 tb, %2, 512;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "add.u32 ta, %1, 40;\n\tadd.u32 tb, %2, 640;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "add.u32 ta, %1, 48;\n\tadd.u32 tb, %2, 768;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "add.u32 ta, %1, 56;\n\tadd.u32 tb, %2, 896;\n\tmov.b64 db, {tb, %4};\n\t"
      "setp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p;\n\t"
      "}"
      ::"r"(o_tmem), "r"(p_tmem), "r"(v_lo), "r"(idesc), "r"(kDescHi), "r"(acc0) : "memory");
}

template <int D, bool FP8>
struct Smem {
  static constexpr int kSlots = slots_of<FP8>();
  static constexpr int kSlabs = D / 64;                     // 64 bf16 = one 128-byte swizzled row
  static constexpr int kSlabBytes = kTileN * 128;            // 128 rows x 128 bytes
  static constexpr int kTileBytes = kSlabs * kSlabBytes;     // one Q / K / V tile
  static constexpr int kCodeBytes = kTileN * D;              // one K / V tile of fp8 codes (128 rows x D bytes)
  static constexpr int kQ = 0;                               // the query tile of the current item
  static constexpr int kRing = kTileBytes;
  static constexpr int kStage = kRing + kSlots * kTileBytes; // fp8 only: raw code tiles on their way to the ring
  static constexpr int kTag = kStage + (FP8 ? kSlots * kCodeBytes : 0);   // uint32 [128 rows]: reference maximum | step number
  static constexpr int kLfin = kTag + kBlockM * 4;           // float [128 rows]: row sums on their way to the epilogue
  static constexpr int kBar = kLfin + kBlockM * 4;
  static constexpr int kNumBars = 2 * kSlots + 3 * kSBufs + 4 + (FP8 ? 2 * kSlots : 0);
  static constexpr int kMisc = kBar + 8 * kNumBars;           // tmem base, abort flag, wait limit (8 bytes)
  static constexpr int kBytes = kMisc + 16;
};

// The mbarriers sit next to one another in shared memory; their addresses are computed, not stored (an array of
// addresses indexed at run time would live in local memory).
template <int kSlots>
struct Bars {
  uint32_t base;
  __device__ __forceinline__ uint32_t full(uint32_t i) const { return base + 8u * i; }
  __device__ __forceinline__ uint32_t empty(uint32_t i) const { return base + 8u * (kSlots + i); }
  __device__ __forceinline__ uint32_t s_full(uint32_t i) const { return base + 8u * (2 * kSlots + i); }
  __device__ __forceinline__ uint32_t p_full(uint32_t i) const { return base + 8u * (2 * kSlots + kSBufs + i); }
  __device__ __forceinline__ uint32_t o_done(uint32_t i) const { return base + 8u * (2 * kSlots + 2 * kSBufs + i); }
  __device__ __forceinline__ uint32_t q_full() const { return base + 8u * (2 * kSlots + 3 * kSBufs); }
  __device__ __forceinline__ uint32_t q_empty() const { return base + 8u * (2 * kSlots + 3 * kSBufs + 1); }
  __device__ __forceinline__ uint32_t o_free() const { return base + 8u * (2 * kSlots + 3 * kSBufs + 2); }
  // the last PV MMA of an item has been issued
  __device__ __forceinline__ uint32_t pv_last() const { return base + 8u * (2 * kSlots + 3 * kSBufs + 3); }
  // fp8 only: a staging slot holds a tile of codes / the converter warps are done with it
  __device__ __forceinline__ uint32_t st_full(uint32_t i) const { return base + 8u * (2 * kSlots + 3 * kSBufs + 4 + i); }
  __device__ __forceinline__ uint32_t st_empty(uint32_t i) const { return base + 8u * (3 * kSlots + 3 * kSBufs + 4 + i); }
};

template <int D, bool PAGED, bool FP8>
__global__ void __launch_bounds__(FP8 ? kThreadsFp8 : kThreads, 1)
attn_kernel(AttnParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
            const __grid_constant__ CUtensorMap map_q) {
  static_assert(!(FP8 && D != 128), "the fp8 cache form is built for 128-wide heads");
  using S = Smem<D, FP8>;
  constexpr int kSlots = S::kSlots;
  extern __shared__ __align__(1024) unsigned char smem[];
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (sbase & 1023u) {   // the swizzled tiles need a 1024-byte aligned base; uniform over the CTA
    if (tid == 0) report_status(p.status, EAGLE_ERR_DEVICE);
    return;
  }

  Bars<kSlots> B;
  B.base = sbase + S::kBar;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + S::kMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + S::kMisc + 4);

  if (tid == 0) {
    // the descriptors of the three tensors are fetched ahead of the first copies that need them
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(B.full(i), FP8 ? 32 * kConvWarps : 1);   // one TMA transaction, or every thread of the converter warps
      mbar_init(B.empty(i), 1);
      if constexpr (FP8) {
        mbar_init(B.st_full(i), 1);
        mbar_init(B.st_empty(i), 32 * kConvWarps);
      }
    }
    for (int i = 0; i < kSBufs; ++i) {
      mbar_init(B.s_full(i), 1);
      mbar_init(B.p_full(i), kGroupThreads);
      mbar_init(B.o_done(i), 1);
    }
    mbar_init(B.q_full(), p.q_tma ? 1 : kGroupThreads);   // one TMA transaction, or every thread of the first softmax group
    mbar_init(B.q_empty(), 1);
    mbar_init(B.o_free(), kGroupThreads);
    mbar_init(B.pv_last(), 1);
    *s_abort = 0;
    *reinterpret_cast<volatile unsigned long long*>(smem + S::kMisc + 8) = p.wait_limit_ns;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kBlockM) reinterpret_cast<volatile uint32_t*>(smem + S::kTag)[tid] = 0xffffffffu;   // no step carries this tag yet
  if (warp == kWarpQK) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + S::kMisc), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  // CTAs 2j and 2j+1 form team j; the team owns the team pieces [tp_lo, tp_hi) of the work line and piece tp gives
  // this CTA the item 2 * tp + member (the two members walk the same KV range with sibling query tiles, or the two
  // halves of a lone tile's range, so whatever one of them pulls from HBM the other finds in L2)
  const int member = blockIdx.x & 1;
  const int tp_lo = p.cta_first[blockIdx.x >> 1], tp_hi = p.cta_first[(blockIdx.x >> 1) + 1];

  if (warp == kWarpQK) {
    // =========================================================================== QK issuer
    // Entry n of the load sequence lives in slot n % kSlots with phase parity (n / kSlots) & 1.  Positions are kept
    // as running counters (no divisions on the threads that keep the tensor pipe fed).
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kBlockM, kTileN, false, FP8);
      uint32_t ks = 0, kp = 0;       // slot / parity of the K tile of the next QK
      uint32_t gq = 0;               // steps issued so far (all items)
      uint32_t sb = 0, sph = 0;      // gq % 3 and (gq / 3) & 1
      uint32_t item_count = 0;
      const uint32_t q_lo = desc_lo(sbase + S::kQ, 16), ring_lo_k = desc_lo(sbase + S::kRing, 16);
      constexpr uint32_t kTileStep = S::kTileBytes >> 4;
      bool ok = true;
      for (int tp = tp_lo; tp < tp_hi && ok; ++tp) {
        const WorkItem it = p.items[2 * tp + member];
        if (it.tile_end <= it.tile_begin) continue;
        const int steps = it.tile_end - it.tile_begin;
        if (p.q_tma) {
          // This thread also fetches the item's query tile, as soon as the last score MMA of the item before has
          // finished with the single 32 KB buffer (the softmax groups still have two or three steps of that item to work
          // through meanwhile): box (64 columns, G heads, 128/G nodes); rows land in (node, head) order = query row order.
          ok = mbar_wait(B.q_empty(), (item_count & 1u) ^ 1u, s_abort);
          if (!ok) break;
          mbar_expect_tx(B.q_full(), S::kTileBytes);
#pragma unroll
          for (int sl = 0; sl < S::kSlabs; ++sl)
            tma_load_4d(sbase + S::kQ + sl * S::kSlabBytes, &map_q, sl * 64, it.g * p.G, it.mt * (kBlockM / p.G), it.b, B.q_full());
        }
        ok = mbar_wait(B.q_full(), item_count & 1u, s_abort);
        if (!ok) break;
        if (item_count > 0) {
          // The tensor pipe runs the MMAs in the order they were issued: a score MMA of this item issued now would run
          // before the last PV MMA of the item before, whose probabilities (the masked last tile) take longest, and the
          // read-out of that item's accumulator, which everything behind the seam waits for, would start that much later.
          ok = mbar_wait(B.pv_last(), (item_count - 1) & 1u, s_abort);
          if (!ok) break;
        }
        for (int s = 0; s < steps && ok; ++s, ++gq) {
          // the K tile arrives long before the score buffer frees up: look at it first, so that nothing but the
          // MMA issue follows the wait that matters
          ok = mbar_wait(B.full(ks), kp, s_abort);
          if (!ok) break;
          // S[gq % 3] also holds P of step gq - 3: it is free once that step's PV has finished
          if (gq >= 3) {
            ok = mbar_wait(B.o_done(sb), sph ^ 1u, s_abort);
            if (!ok) break;
          }
          tc_fence_after();
          issue_qk_tile<D>(tmem + kColS + sb * kTileN, q_lo, ring_lo_k + ks * kTileStep, idesc_qk);
          tc_commit(B.s_full(sb));
          tc_commit(B.empty(ks));
          ks += gq < 2 ? 1u : 2u;   // K(g) is entry g for g < 3, entry 2g - 2 after that
          if (ks >= kSlots) { ks -= kSlots; kp ^= 1u; }
          if (++sb == kSBufs) { sb = 0; sph ^= 1u; }
          if (s == steps - 1) tc_commit(B.q_empty());      // every QK of this item has been issued
        }
        ++item_count;
      }
    }
  } else if (warp == kWarpPV) {
    // =========================================================================== PV issuer
    if (lane == 0) {
      constexpr uint32_t idesc_pv = instr_desc(kBlockM, D, true, FP8);
      uint32_t vs = 3, vp = 0;       // slot / parity of the V tile of the next PV: V(g) is entry 2g + 3
      uint32_t gp = 0;               // steps issued so far (all items)
      uint32_t sb = 0, sph = 0;      // gp % 3 and (gp / 3) & 1
      uint32_t item_count = 0;
      const uint32_t ring_lo_v = desc_lo(sbase + S::kRing, S::kSlabBytes);
      constexpr uint32_t kTileStep = S::kTileBytes >> 4;
      bool ok = true;
      for (int tp = tp_lo; tp < tp_hi && ok; ++tp) {
        const WorkItem it = p.items[2 * tp + member];
        if (it.tile_end <= it.tile_begin) continue;
        const int steps = it.tile_end - it.tile_begin;
        for (int s = 0; s < steps && ok; ++s, ++gp) {
          ok = mbar_wait(B.full(vs), vp, s_abort);   // (arrives well before P is ready)
          if (!ok) break;
          if (s == 0 && item_count > 0) {
            ok = mbar_wait(B.o_free(), (item_count - 1) & 1u, s_abort);   // previous epilogue has read O
            if (!ok) break;
          }
          ok = mbar_wait(B.p_full(sb), sph, s_abort);
          if (!ok) break;
          tc_fence_after();
          issue_pv_tile(tmem + kColO, tmem + kColS + sb * kTileN, ring_lo_v + vs * kTileStep, idesc_pv, s == 0 ? 0u : 1u);
          tc_commit(B.o_done(sb));
          tc_commit(B.empty(vs));
          if (s == steps - 1) mbar_arrive(B.pv_last());
          vs += 2;
          if (vs >= kSlots) { vs -= kSlots; vp ^= 1u; }
          if (++sb == kSBufs) { sb = 0; sph ^= 1u; }
        }
        ++item_count;
      }
    }
  } else if (warp < kSoftmaxWarps) {
    // =========================================================================== softmax + epilogue (warps 0-7)
    // Two groups of four warps; group g takes the steps whose global number is g mod 2, so the
    // groups run half a step out of phase and each scheduler hosts one warp of either: while one waits on tensor
    // memory or a barrier, the other computes.  Thread r of a group owns query row r (= TMEM lane r), all 128 score
    // columns.  The two threads of a row share one reference maximum: the thread that handled step gs publishes it,
    // tagged with gs, and the other picks it up before it takes its exponentials of step gs + 1.  Each keeps its own
    // part of the row sum, relative to that reference.
    const uint32_t grp = static_cast<uint32_t>(warp >> 2);
    const int r = tid & (kBlockM - 1);                    // query row within the tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    volatile uint32_t* tag = reinterpret_cast<volatile uint32_t*>(smem + S::kTag) + r;   // reference | step, per row
    volatile float* lfin = reinterpret_cast<volatile float*>(smem + S::kLfin) + r;       // row sum on its way to the epilogue
    const uint32_t o_addr = tmem + lane_addr + kColO;

    uint32_t g_base = 0, item_count = 0, sg = 0;   // KV tiles, items and steps before the current item
    bool ok = true;
    for (int tp = tp_lo; tp < tp_hi && ok; ++tp) {
      const WorkItem it = p.items[2 * tp + member];
      if (it.tile_end <= it.tile_begin) continue;
      const SeqPlan sp = p.seq[it.b];
      const int L = sp.L, n = sp.n, G = p.G;
      const int m_valid = n * G, kv_end = L + n;
      const int steps = it.tile_end - it.tile_begin;
      const int R = it.mt * kBlockM + r;
      const bool row_valid = R < m_valid;
      const int node = row_valid ? R / G : 0, hh = row_valid ? R % G : 0;
      const uint64_t anc = row_valid ? p.anc[static_cast<size_t>(it.b) * p.T_max + node] : 0ull;
      // fp8 cache: the keys' scale of this (sequence, KV head) goes into the softmax scale, the values' into the output
      float scale_log2 = p.scale_log2, v_scale = 1.f;
      if constexpr (FP8) {
        scale_log2 *= p.k_scale[it.b * p.Hkv + it.g];
        v_scale = p.v_scale[it.b * p.Hkv + it.g];
      }

      if (!p.q_tma && grp == 0) {
        // group sizes that do not divide 128: the first softmax group stages the query tile itself, a row per thread
        ok = mbar_wait_warp(B.q_empty(), (item_count & 1u) ^ 1u, s_abort);
        if (!ok) break;
        const uint4* src = reinterpret_cast<const uint4*>(p.q + ((static_cast<size_t>(it.b) * p.T_max + node) * p.Hq + it.g * G + hh) * D);
        unsigned char* qdst = smem + S::kQ + r * 128;
#pragma unroll
        for (int c = 0; c < 8 * S::kSlabs; ++c) {
          uint4 v = row_valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
          if constexpr (FP8) {     // the MMAs of this form take fp16 operands: every bf16 query of magnitude 2^-14 .. 65504 is one
            v.x = pack_f16(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u));
            v.y = pack_f16(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
            v.z = pack_f16(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u));
            v.w = pack_f16(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
          }
          *reinterpret_cast<uint4*>(qdst + (c >> 3) * S::kSlabBytes + (((c & 7) ^ (r & 7)) << 4)) = v;
        }
        fence_proxy_async();
        mbar_arrive(B.q_full());
      }

      float m_ref = -INFINITY;   // reference (scaled, log2 domain) this thread's row sum is relative to
      float m_in = -INFINITY;    // reference the other group left behind at the step before this group's latest one
      float l_sum = 0.f;         // this thread's part of the row sum
      // this group's steps of the item: those whose global number has the group's parity
      for (int s = static_cast<int>((sg ^ grp) & 1u); s < steps; s += 2) {
        const uint32_t gs = sg + s;
        const uint32_t sb = gs % kSBufs, sph = (gs / kSBufs) & 1u;     // score buffer of this step and its phase
        const uint32_t s_addr = tmem + lane_addr + kColS + sb * kTileN;   // P goes over the front half of the same columns
        ok = mbar_wait_warp(B.s_full(sb), sph, s_abort);
        if (!ok) break;
        tc_fence_after();
        const int key0 = (it.tile_begin + s) * kTileN;
        // Tiles that reach past the committed prefix (an item's last one or two): a compact pre-pass writes -inf over the
        // scores of this row's invisible keys in tensor memory, so that the two passes below carry no masking code (the
        // loop they form has to stay small: the instruction cache decides a fifth of this kernel's speed).  Keys before L
        // are all visible; key L + m is visible iff bit m of the node's ancestor mask is set (the mask has no bits at or
        // above the tree size).
        if (key0 + kTileN > L) {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            const int rel = key0 + c * 32 - L;        // tree index of the chunk's first key (negative: still in the prefix)
            uint32_t w;
            if (rel >= 64) w = 0u;
            else if (rel >= 0) w = static_cast<uint32_t>(anc >> rel);
            else if (rel > -32) w = static_cast<uint32_t>(anc << (-rel)) | ((1u << (-rel)) - 1u);
            else w = 0xffffffffu;
            if (rel <= -32) continue;                 // wholly in the prefix (uniform over the warp: the loads below are collective)
            uint32_t t[32];
            if (rel < n) {                            // (uniform too) some key of the chunk belongs to the tree
              tmem_ld32(s_addr + c * 32, t);
              tc_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) t[e] = (w >> e) & 1u ? t[e] : 0xff800000u;       // -inf
            } else {                                  // wholly past the tree: nothing to keep, nothing to fetch
#pragma unroll
              for (int e = 0; e < 32; ++e) t[e] = 0xff800000u;
            }
            tmem_st32(s_addr + c * 32, t);
          }
          tc_wait_st();
        }
        // ---- pass 1: row maximum of the raw scores.  All four chunks are fetched in one round trip to tensor memory;
        // chunks 0 and 1 stay in registers for pass 2, chunks 2 and 3 are dropped after the maximum and fetched again
        // later (keeping them would leave too few registers for pass 2).  (With an fp8 cache the CTA has 512 threads and
        // 128 registers each: two round trips, chunks 2 and 3 first, then chunks 0 and 1, which stay.)
        uint32_t ra[32], rb[32];
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if constexpr (FP8) {
          tmem_ld32(s_addr + 64, ra);
          tmem_ld32(s_addr + 96, rb);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            mx[0] = max3(mx[0], __uint_as_float(ra[e]), __uint_as_float(ra[e + 1]));
            mx[1] = max3(mx[1], __uint_as_float(rb[e]), __uint_as_float(rb[e + 1]));
          }
          tmem_ld32(s_addr, ra);
          tmem_ld32(s_addr + 32, rb);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            mx[2] = max3(mx[2], __uint_as_float(ra[e]), __uint_as_float(ra[e + 1]));
            mx[3] = max3(mx[3], __uint_as_float(rb[e]), __uint_as_float(rb[e + 1]));
          }
        } else
        {
          uint32_t rc[32], rd[32];
          tmem_ld32(s_addr + 64, rc);
          tmem_ld32(s_addr + 96, rd);
          tmem_ld32(s_addr, ra);
          tmem_ld32(s_addr + 32, rb);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            mx[0] = max3(mx[0], __uint_as_float(rc[e]), __uint_as_float(rc[e + 1]));
            mx[1] = max3(mx[1], __uint_as_float(rd[e]), __uint_as_float(rd[e + 1]));
            mx[2] = max3(mx[2], __uint_as_float(ra[e]), __uint_as_float(ra[e + 1]));
            mx[3] = max3(mx[3], __uint_as_float(rb[e]), __uint_as_float(rb[e + 1]));
          }
        }
        const float tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;   // scale > 0

        if (key0 + kTileN > kv_end) {
          // rows of the V tile past prefix + tree may hold anything: zero them so that 0 * garbage cannot reach O
          const uint32_t nv = 2 * (g_base + s) + 3, slot = nv % kSlots, par = (nv / kSlots) & 1u;
          if constexpr (FP8) {
            // With four ring slots this V tile shares its slot with the V tile of two steps ago, which need not have
            // been consumed, or even converted, when this step's scores are ready; the parity wait below would then
            // take that older phase for this one and the zeros would land in the wrong tile.  Wait for that PV first.
            // (With six slots the slot's previous tile is three steps back: its PV freed this step's score buffer.)
            if (gs >= 2u) {
              ok = mbar_wait_warp(B.o_done((gs - 2u) % kSBufs), ((gs - 2u) / kSBufs) & 1u, s_abort);
              if (!ok) break;
            }
          }
          ok = mbar_wait_warp(B.full(slot), par, s_abort);
          if (!ok) break;
          if (key0 + r >= kv_end) {
#pragma unroll
            for (int c = 0; c < 8 * S::kSlabs; ++c)
              *reinterpret_cast<uint4*>(smem + S::kRing + slot * S::kTileBytes + (c >> 3) * S::kSlabBytes + r * 128 + (c & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();
        }

        // the reference the other group settled on at the previous step (waited for at an item's first step too,
        // where its value is not used: the other group must have read the tag of step gs - 2 before it is replaced)
        float m_prev = -INFINITY;
        if (gs > 0) {
          const unsigned long long t = tag_wait(tag, (gs - 1u) & 0xffu, s_abort);
          ok = __all_sync(0xffffffffu, (t >> 32) != 0ull);
          if (!ok) break;
          if (s > 0) m_prev = __uint_as_float(static_cast<uint32_t>(t) & 0xffffff00u);
        }
        if (m_prev != m_ref) {
          l_sum *= fast_exp2(m_ref - m_prev);     // m_ref = -inf: nothing summed yet, the factor is 0
          m_ref = m_prev;
        }
        m_in = m_prev;
        // lazy rescale: move the reference only when the row max outgrows it by more than the threshold
        const bool grow = tmax > m_ref + kRescaleThreshold || (m_ref == -INFINITY && tmax > -INFINITY);
        float factor = 1.f;
        if (grow) {
          const float m_new = __uint_as_float(__float_as_uint(tmax) & 0xffffff00u);   // the low byte carries the step tag
          factor = fast_exp2(m_ref - m_new);     // 0 when there was no reference yet
          m_ref = m_new;
          l_sum *= factor;
        }
        *tag = __float_as_uint(m_ref) | (gs & 0xffu);
        if (s > 0 && __any_sync(0xffffffffu, grow)) {
          // the previous step accumulated into O and may still be running
          ok = mbar_wait_warp(B.o_done((gs - 1) % kSBufs), ((gs - 1) / kSBufs) & 1u, s_abort);
          if (!ok) break;
          tc_fence_after();
          uint32_t o[32];
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            tmem_ld32(o_addr + c * 32, o);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
            tmem_st32(o_addr + c * 32, o);
          }
          tc_wait_st();
        }
        // ---- pass 2: exponentials and packed P, in column order (P overwrites score columns that have been
        // consumed).  Chunks 0 and 1 are still in registers; chunks 2 and 3 are fetched again meanwhile.
        const float neg_base = m_ref == -INFINITY ? 0.f : -m_ref;
        const uint64_t scale2 = pack2(scale_log2, scale_log2), base2 = pack2(neg_base, neg_base);
        uint64_t ls2[2] = {0ull, 0ull};   // four partial sums
        uint32_t pk[16];
        auto exp_chunk = [&](const uint32_t* raw, int c) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const uint64_t x2 = fma2(pack2(__uint_as_float(raw[2 * j]), __uint_as_float(raw[2 * j + 1])), scale2, base2);
            float p0, p1;
            if (kPolyStride > 0 && j % (kPolyStride > 0 ? kPolyStride : 1) == (kPolyStride > 0 ? kPolyStride : 1) - 1) {
              poly_exp2_pair(x2, p0, p1);
            } else {
              float a, b;
              unpack2(x2, a, b);
              p0 = fast_exp2(a);
              p1 = fast_exp2(b);
            }
            ls2[j & 1] = add2(ls2[j & 1], pack2(p0, p1));
            pk[j] = FP8 ? pack_f16(p0, p1) : pack_bf16(p0, p1);
          }
          tmem_st16(s_addr + c * 16, pk);
        };
        exp_chunk(ra, 0);
        tmem_ld32(s_addr + 64, ra);         // chunk 2, in flight while chunk 1 is worked on
        exp_chunk(rb, 1);
        tmem_ld32(s_addr + 96, rb);         // chunk 3
        tc_wait_ld();
        exp_chunk(ra, 2);
        exp_chunk(rb, 3);
        {
          float l0, l1, l2, l3;
          unpack2(ls2[0], l0, l1);
          unpack2(ls2[1], l2, l3);
          l_sum += (l0 + l1) + (l2 + l3);
        }
        if (s == steps - 2) {
          // this group's last step of the item, but not the item's: hand the row sum to the group that writes the
          // output.  A two-step item is the one case where the slot may still be in use for the previous item.
          if (s == 0 && item_count > 0) {
            ok = mbar_wait_warp(B.o_free(), (item_count - 1) & 1u, s_abort);
            if (!ok) break;
          }
          *lfin = l_sum;
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(B.p_full(sb));

        if (s == steps - 1) {
          // ---- this group took the item's last step: it writes the item's output.  Wait for the last PV (PVs
          // complete in order), add the other group's part of the row sum, then write the row: bf16 output, or
          // the unnormalised fp32 partial of a cut piece.
          ok = mbar_wait_warp(B.o_done(sb), sph, s_abort);
          if (!ok) break;
          tc_fence_after();
          float l_row = l_sum;
          if (steps > 1) {
            // the other group's sum is relative to the reference it last saw
            const float w = m_in == m_ref ? 1.f : fast_exp2(m_in - m_ref);
            l_row = fmaf(*lfin, w, l_row);
          }
          const float inv = l_row > 0.f ? v_scale / l_row : 0.f;   // (v_scale is 1 unless the cache is fp8)
          // The accumulator is read 32 columns at a time, the next chunk's load in flight while this one is scaled and
          // stored.  These stores sit on the seam between two items (the group cannot take its next step, and the next
          // item's first PV cannot start, before they are issued), and with a row per thread every lane of a store
          // instruction is in a different line whatever its width: the output row leaves in 32-byte pieces (half as
          // many instructions as with 16-byte ones), and the fp32 partial of a cut piece is laid out [4 columns][row],
          // so that the 32 lanes of a store write 512 consecutive bytes.
          uint32_t oa[32], ob[32];
          auto store_chunk = [&](uint32_t (&o)[32], int c) {
            if (!row_valid) return;
            if (it.slot < 0) {
              __nv_bfloat16* out_row = p.out + ((static_cast<size_t>(it.b) * p.T_max + node) * p.Hq + it.g * G + hh) * D;
#pragma unroll
              for (int e = 0; e < 32; e += 16) {
                uint32_t v[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) v[k] = pack_bf16(__uint_as_float(o[e + 2 * k]) * inv, __uint_as_float(o[e + 2 * k + 1]) * inv);
                st_global_v8(out_row + c * 32 + e, v);
              }
            } else {
              float* part = p.part_o + (static_cast<size_t>(it.slot) * (D / 4) + c * 8) * (kBlockM * 4) + r * 4;
              if constexpr (FP8) {
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * v_scale);
              }
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<uint4*>(part + (e / 4) * (kBlockM * 4)) = make_uint4(o[e], o[e + 1], o[e + 2], o[e + 3]);
            }
          };
          tmem_ld32(o_addr, oa);
#pragma unroll
          for (int c = 0; c < D / 32; c += 2) {
            tc_wait_ld();
            tmem_ld32(o_addr + (c + 1) * 32, ob);
            store_chunk(oa, c);
            tc_wait_ld();
            if (c + 2 < D / 32) tmem_ld32(o_addr + (c + 2) * 32, oa);
            store_chunk(ob, c + 1);
          }
          if (row_valid && it.slot >= 0) p.part_ml[static_cast<size_t>(it.slot) * kBlockM + r] = make_float2(m_ref, l_row);
          tc_fence_before();
          mbar_arrive(B.o_free());            // the next item's first PV may overwrite the accumulator
        }
      }
      g_base += steps;
      sg += steps;
      ++item_count;
    }
  } else if (warp == kWarpProducer) {
    // =========================================================================== TMA producer
    // Load order: K(0), K(1), K(2), then V(g), K(g + 3) for g = 0, 1, ... (g counts this CTA's steps across items):
    // the order in which the MMAs consume the tiles, since the score MMA runs three steps ahead of the PV MMA.
    // Entry n of that sequence lives in slot n % kSlots; with six slots the K tile of step g + 3 is requested when the
    // score MMA of step g has finished and the V tile of step g when the PV of step g - 3 has.
    // Contiguous cache: one thread does it all.  Paged cache: the whole warp walks the list in step and each lane looks up
    // and fetches one box (a page, or a page's 64-column half) of the tile, so the block-table reads of a tile are in flight together.
    if (lane == 0 || PAGED) {
      struct Cursor {
        int tp, tile, tile_end, z;
        bool valid;
        const int32_t* pages;   // paged cache: the sequence's row of the block table, and its last page in use
        int last_page;
      };
      auto advance = [&](Cursor& c) {   // moves to the next KV tile of the work list
        if (++c.tile < c.tile_end) return;
        for (++c.tp; c.tp < tp_hi; ++c.tp) {
          const WorkItem it = p.items[2 * c.tp + member];
          if (it.tile_end > it.tile_begin) {
            c.tile = it.tile_begin;
            c.tile_end = it.tile_end;
            if constexpr (PAGED) {
              const SeqPlan sp = p.seq[it.b];
              c.z = it.g;
              c.pages = p.block_table + static_cast<size_t>(it.b) * p.max_pages;
              c.last_page = (sp.L + sp.n - 1) >> p.page_shift;
            } else {
              c.z = it.b * p.Hkv + it.g;
            }
            return;
          }
        }
        c.valid = false;
      };
      bool ok = true;
      uint32_t n = 0;   // position in the load sequence
      auto load_tile = [&](const Cursor& c, bool is_v) {
        const uint32_t slot = n % kSlots, par = ((n / kSlots) & 1u) ^ 1u;
        if (p.stall_after_tiles >= 0 && n >= static_cast<uint32_t>(p.stall_after_tiles)) {
          ok = false;   // test hook: the producer falls silent (nothing further is issued), so the consumers' waits run out
          return;
        }
        if constexpr (PAGED) {
          // The tile's 128 slots come from one page (pages of 128 slots or more) or from 128 / page_size pages, one box
          // each; the boxes land one under the other, which is the tile's layout.  A box past the sequence's last page
          // fetches that last page again (its rows are masked), so the byte count of a tile never changes.  The page
          // number is read before the wait for the slot, so that its latency is not added to the slot's turnaround.
          // (A page of fp8 codes: a row is one 128-byte line, so a box is the page's rows whole, and it lands in the staging slot.)
          const int rows = p.page_size < kTileN ? p.page_size : kTileN;
          constexpr int kBoxSlabs = FP8 ? 1 : S::kSlabs;
          const int sl = lane % kBoxSlabs;                      // lane = (box, 64-column slab): one TMA box per lane
          const int r0 = (lane / kBoxSlabs) * rows, key = c.tile * kTileN + r0;
          int page = 0;
          if (r0 < kTileN) {
            const int pi = key >> p.page_shift;
            page = __ldg(c.pages + (pi < c.last_page ? pi : c.last_page));
          }
          if constexpr (FP8) {
            ok = mbar_wait_warp(B.st_empty(slot), par, s_abort);
            if (!ok) return;
            if (lane == 0) mbar_expect_tx(B.st_full(slot), S::kCodeBytes);
            __syncwarp();
            if (r0 < kTileN)
              tma_load_3d(sbase + S::kStage + slot * S::kCodeBytes + r0 * 128, is_v ? &map_v : &map_k, 0, key & (p.page_size - 1),
                          page * p.Hkv + c.z, B.st_full(slot));
          } else {
            ok = mbar_wait_warp(B.empty(slot), par, s_abort);
            if (!ok) return;
            if (lane == 0) mbar_expect_tx(B.full(slot), S::kTileBytes);
            __syncwarp();
            if (r0 < kTileN)
              tma_load_3d(sbase + S::kRing + slot * S::kTileBytes + sl * S::kSlabBytes + r0 * 128, is_v ? &map_v : &map_k, sl * 64,
                          key & (p.page_size - 1), page * p.Hkv + c.z, B.full(slot));
          }
        } else if constexpr (FP8) {
          // the tile of codes goes to the staging slot; the converter warps widen it into ring slot `slot`
          ok = mbar_wait(B.st_empty(slot), par, s_abort);
          if (!ok) return;
          mbar_expect_tx(B.st_full(slot), S::kCodeBytes);
          tma_load_3d(sbase + S::kStage + slot * S::kCodeBytes, is_v ? &map_v : &map_k, 0, c.tile * kTileN, c.z, B.st_full(slot));
        } else {
          ok = mbar_wait(B.empty(slot), par, s_abort);
          if (!ok) return;
          mbar_expect_tx(B.full(slot), S::kTileBytes);
#pragma unroll
          for (int sl = 0; sl < S::kSlabs; ++sl)
            tma_load_3d(sbase + S::kRing + slot * S::kTileBytes + sl * S::kSlabBytes, is_v ? &map_v : &map_k, sl * 64, c.tile * kTileN, c.z,
                        B.full(slot));
        }
      };
      Cursor ck = {tp_lo - 1, 0, 0, 0, true, nullptr, 0}, cv = {tp_lo - 1, 0, 0, 0, true, nullptr, 0};
      advance(ck);
      advance(cv);
      for (int i = 0; i < 3; ++i, ++n) {   // K(0), K(1), K(2)
        if (ok && ck.valid) {
          load_tile(ck, false);
          advance(ck);
        }
      }
      while (ok && cv.valid) {
        load_tile(cv, true);      // V(g)
        ++n;
        advance(cv);
        if (ok && ck.valid) {     // K(g + 3)
          load_tile(ck, false);
          advance(ck);
        }
        ++n;
      }
    }
  } else if (FP8 && warp >= kWarpConvert) {
    // =========================================================================== fp8 -> fp16 converter (warps 11-14)
    // Thread r owns row r of every K / V tile: it reads the row's 128 codes from the staging slot (eight 16-byte chunks,
    // 128-byte swizzled as the copy laid them down), widens them, and writes the row's 256 bytes into the ring slot in
    // the swizzled two-slab layout the MMAs read.  Every e4m3 number is an fp16 number, subnormals included, so the
    // hardware conversion (two codes per instruction) is exact.  The MMAs of this form therefore run fp16 x fp16 (an
    // MMA takes one 16-bit type for both operands): the queries are converted as they are staged and P is written as
    // fp16.  The scales are applied elsewhere.
    if constexpr (FP8) {
      const int r0 = tid - 32 * kWarpConvert;
      uint32_t steps_total = 0;     // this CTA's steps over all its items
      for (int tp = tp_lo; tp < tp_hi; ++tp) {
        const WorkItem it = p.items[2 * tp + member];
        if (it.tile_end > it.tile_begin) steps_total += static_cast<uint32_t>(it.tile_end - it.tile_begin);
      }
      auto widen = [](uint32_t w, uint32_t& lo, uint32_t& hi) {    // four codes -> four fp16 numbers
        asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
            : "=r"(lo), "=r"(hi) : "r"(w));
      };
      // Entry n of the load sequence is K(n) for n < 3, V((n - 3) / 2) for odd n and K((n + 2) / 2) for even n after
      // that; the K entries of the last three steps do not exist (the producer skips them, the numbering keeps its gaps).
      bool ok = true;
      uint32_t slot = 0, par = 0;
      const uint32_t n_end = steps_total ? 2u * steps_total + 2u : 0u;
      for (uint32_t n = 0; n < n_end && ok; ++n, slot = (slot + 1 == kSlots ? 0 : slot + 1), par ^= (slot == 0 ? 1u : 0u)) {
        const uint32_t g = n < 3 ? n : ((n & 1u) ? (n - 3u) / 2u : (n + 2u) / 2u);
        if (g >= steps_total) continue;
        ok = mbar_wait_warp(B.st_full(slot), par, s_abort);
        if (!ok) break;
        ok = mbar_wait_warp(B.empty(slot), par ^ 1u, s_abort);    // the MMA that read the ring slot last has finished
        if (!ok) break;
#pragma unroll 1
        for (int r = r0; r < kTileN; r += 32 * kConvWarps) {
          const unsigned char* src = smem + S::kStage + slot * S::kCodeBytes + r * 128;
          unsigned char* dst = smem + S::kRing + slot * S::kTileBytes + r * 128;
          uint4 w[8];
#pragma unroll
          for (int c = 0; c < 8; ++c) w[c] = *reinterpret_cast<const uint4*>(src + ((c ^ (r & 7)) << 4));
#pragma unroll
          for (int c = 0; c < 8; ++c) {                            // codes 16c .. 16c + 15 of the row
            uint4 u, v;
            widen(w[c].x, u.x, u.y);
            widen(w[c].y, u.z, u.w);
            widen(w[c].z, v.x, v.y);
            widen(w[c].w, v.z, v.w);
            unsigned char* d = dst + (c >> 2) * S::kSlabBytes;     // 64 columns per slab: chunks 2c and 2c + 1 of the slab's row
            *reinterpret_cast<uint4*>(d + ((((2 * c) & 7) ^ (r & 7)) << 4)) = u;
            *reinterpret_cast<uint4*>(d + ((((2 * c + 1) & 7) ^ (r & 7)) << 4)) = v;
          }
        }
        fence_proxy_async();                                       // the MMAs read the slot through the async proxy
        mbar_arrive(B.full(slot));
        mbar_arrive(B.st_empty(slot));
      }
    }
  }

  // ---- teardown: everyone arrives here (normally or after an abort); release TMEM
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) report_status(p.status, EAGLE_ERR_TIMEOUT);
  if (warp == kWarpQK) {
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

// [B*Hkv, S_cap, D] bf16 viewed as a 3-D tensor (d, slot, sequence-head); box = 64 x box_rows x 1, 128-byte swizzle.
// A paged cache [num_pages, Hkv, page_size, D] is the same tensor with pages for sequences and page_size for S_cap;
// its box has min(page_size, 128) rows.
bool make_kv_map(CUtensorMap* map, const void* base, int D, int S_cap, long long bh, int box_rows = kTileN) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S_cap), static_cast<cuuint64_t>(bh)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(S_cap) * D * 2};
  const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A cache of fp8 codes [B*Hkv, S_cap, D] uint8: box = D x 128 rows x 1 (D = 128: one 128-byte swizzled row per slot).
bool make_code_map(CUtensorMap* map, const void* base, int D, int S_cap, long long bh, int rows = kTileN) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S_cap), static_cast<cuuint64_t>(bh)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S_cap) * D};
  const cuuint32_t box[3] = {static_cast<cuuint32_t>(D), static_cast<cuuint32_t>(rows), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q [B, T_max, Hq, D] bf16 viewed as (d, head, node, sequence); box = 64 x G x 128/G x 1: the 128 query rows of one
// (sequence, KV head, query tile) in (node, head-in-group) order.  Needs 128 % G == 0.
bool make_q_map(CUtensorMap* map, const void* base, int D, int Hq, int T_max, int B, int G) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(Hq), static_cast<cuuint64_t>(T_max),
                              static_cast<cuuint64_t>(B)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(Hq) * D * 2,
                                 static_cast<cuuint64_t>(T_max) * Hq * D * 2};
  const cuuint32_t box[4] = {64, static_cast<cuuint32_t>(G), static_cast<cuuint32_t>(kBlockM / G), 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int attn_tile_keys() { return kTileN; }

cudaError_t attn_prepare(int head_dim) {
  cudaError_t e;
  if (head_dim == 128) {
    e = cudaFuncSetAttribute(attn_kernel<128, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128, false>::kBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_kernel<128, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128, true>::kBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_kernel<128, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128, true>::kBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attn_kernel<128, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128, false>::kBytes);
  }
  e = cudaFuncSetAttribute(attn_kernel<64, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<64, false>::kBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_kernel<64, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<64, false>::kBytes);
}

// Returns cudaErrorInvalidValue when the tensor maps cannot be encoded.
cudaError_t launch_attn(const AttnParams& p_in, int num_ctas, cudaStream_t stream) {
  AttnParams p = p_in;
  CUtensorMap mk, mv, mq;
  const bool paged = p.page_size > 0, fp8 = p.k_scale != nullptr;
  if (fp8 && paged) {
    if (p.D != 128) return cudaErrorInvalidValue;
    const long long ph = static_cast<long long>(p.num_pages) * p.Hkv;
    const int rows = p.page_size < kTileN ? p.page_size : kTileN;
    if (!make_code_map(&mk, p.k, p.D, p.page_size, ph, rows) || !make_code_map(&mv, p.v, p.D, p.page_size, ph, rows)) return cudaErrorInvalidValue;
  } else if (fp8) {
    if (p.D != 128) return cudaErrorInvalidValue;
    const long long bh = static_cast<long long>(p.B) * p.Hkv;
    if (!make_code_map(&mk, p.k, p.D, p.S_cap, bh) || !make_code_map(&mv, p.v, p.D, p.S_cap, bh)) return cudaErrorInvalidValue;
  } else if (paged) {
    const long long ph = static_cast<long long>(p.num_pages) * p.Hkv;
    const int rows = p.page_size < kTileN ? p.page_size : kTileN;
    if (!make_kv_map(&mk, p.k, p.D, p.page_size, ph, rows) || !make_kv_map(&mv, p.v, p.D, p.page_size, ph, rows)) return cudaErrorInvalidValue;
  } else {
    const long long bh = static_cast<long long>(p.B) * p.Hkv;
    if (!make_kv_map(&mk, p.k, p.D, p.S_cap, bh) || !make_kv_map(&mv, p.v, p.D, p.S_cap, bh)) return cudaErrorInvalidValue;
  }
  p.q_tma = (kBlockM % p.G == 0 && !fp8) ? 1 : 0;   // (the fp8 form converts the queries to fp16 as it stages them)
  if (p.q_tma) {
    if (!make_q_map(&mq, p.q, p.D, p.Hq, p.T_max, p.B, p.G)) return cudaErrorInvalidValue;
  } else {
    mq = mk;   // unused by the kernel
  }
  if (fp8) {
    if (paged) attn_kernel<128, true, true><<<num_ctas, kThreadsFp8, Smem<128, true>::kBytes, stream>>>(p, mk, mv, mq);
    else attn_kernel<128, false, true><<<num_ctas, kThreadsFp8, Smem<128, true>::kBytes, stream>>>(p, mk, mv, mq);
  } else if (p.D == 128) {
    if (paged) attn_kernel<128, true, false><<<num_ctas, kThreads, Smem<128, false>::kBytes, stream>>>(p, mk, mv, mq);
    else attn_kernel<128, false, false><<<num_ctas, kThreads, Smem<128, false>::kBytes, stream>>>(p, mk, mv, mq);
  } else {
    if (paged) attn_kernel<64, true, false><<<num_ctas, kThreads, Smem<64, false>::kBytes, stream>>>(p, mk, mv, mq);
    else attn_kernel<64, false, false><<<num_ctas, kThreads, Smem<64, false>::kBytes, stream>>>(p, mk, mv, mq);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace eagle
