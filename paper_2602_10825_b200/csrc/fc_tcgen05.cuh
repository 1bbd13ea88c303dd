// Thin inline-PTX wrappers for the Blackwell (sm_100a) features the tensor-core kernels use:
// mbarriers, TMA tiled loads, tensor-memory allocation, tcgen05.mma / ld / st / commit, and the
// shared-memory and instruction descriptors tcgen05.mma takes.
#pragma once

#include <cuda.h>
#include <stdint.h>

namespace fc {
namespace sm100 {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// ---- mbarrier -------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Gives up once `limit_ns` of wall time have passed (checked every 32 failed polls; one poll
// may itself suspend the thread for a short, hardware-defined time) or as soon as another thread of the
// CTA has given up (*abort != 0); the caller then runs on without waiting, so control flow stays uniform
// and the kernel reaches its normal teardown.  Returns false if it gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile uint32_t* abort,
                                                  uint64_t limit_ns = 2000000000ull) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t n = 1;; ++n) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
    if ((n & 31u) == 0 && global_timer_ns() - t0 > limit_ns) break;
  }
  *abort = 1;
  return false;
}

// ---- TMA ------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// Four rows of a 2-D tensor (row indices r0..r3, starting at column c0) into four consecutive rows of a shared-memory
// tile: the tile::gather4 form of the tiled load.  The tensor map's box is one row high; the copy goes to this CTA only.
__device__ __forceinline__ void tma_gather4_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int r0, int r1,
                                               int r2, int r3) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---- tensor memory --------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t n_cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(n_cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t n_cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (quadrant base + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// ---- tcgen05.mma ----------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle.  Fields (bit positions): start address >> 4
// [0,14); leading-dimension byte offset >> 4 [16,30); stride-dimension byte offset >> 4 [32,46);
// descriptor version 1 at [46,48); swizzle mode 2 (128 B) at [61,64).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor for kind::f16 with bf16 operands and fp32 accumulation.
// D format fp32 = 1 at [4,6); A and B format bf16 = 1 at [7,10) and [10,13); A / B major at bits 15 / 16
// (0 = K-major, 1 = MN-major); N >> 3 at [17,23); M >> 4 at [24,29).
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int M, int N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on an mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

// Groups of MMAs issued as one block of instructions, every operand already in a register.  The issuing thread
// does not run ahead of the tensor pipe: what it executes between two MMAs of its own is time during which the
// pipe has nothing from it (measured: 64 clocks per 128x128x16 MMA back to back, plus 6 to 9 clocks for every
// instruction in between).  So descriptors are computed, and pinned in registers, before the wait that precedes a group.
template <int N>
__device__ __forceinline__ void pin(uint64_t (&d)[N]) {
  static_assert(N == 4 || N == 8, "group size");
  if constexpr (N == 8)
    asm volatile("" : "+l"(d[0]), "+l"(d[1]), "+l"(d[2]), "+l"(d[3]), "+l"(d[4]), "+l"(d[5]), "+l"(d[6]), "+l"(d[7]));
  else
    asm volatile("" : "+l"(d[0]), "+l"(d[1]), "+l"(d[2]), "+l"(d[3]));
}
__device__ __forceinline__ void pin(uint32_t (&d)[4]) {
  asm volatile("" : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]));
}
// D = A B over N k-steps, A and B in shared memory; the first k-step overwrites D
template <int N>
__device__ __forceinline__ void umma_ss_group(uint32_t d_tmem, const uint64_t (&a)[N], const uint64_t (&b)[N], uint32_t idesc) {
  if constexpr (N == 8) {
    asm volatile(
        "{\n"
        ".reg .pred f, t;\n"
        "setp.ne.b32 f, %0, %0;\n"
        "setp.eq.b32 t, %0, %0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %2, %10, %1, f;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %3, %11, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %4, %12, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %5, %13, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %6, %14, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %7, %15, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %8, %16, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %9, %17, %1, t;\n"
        "}\n"
        ::"r"(d_tmem), "r"(idesc), "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(a[4]), "l"(a[5]), "l"(a[6]), "l"(a[7]),
          "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "l"(b[4]), "l"(b[5]), "l"(b[6]), "l"(b[7])
        : "memory");
  } else {
    asm volatile(
        "{\n"
        ".reg .pred f, t;\n"
        "setp.ne.b32 f, %0, %0;\n"
        "setp.eq.b32 t, %0, %0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %2, %6, %1, f;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %3, %7, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %4, %8, %1, t;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %5, %9, %1, t;\n"
        "}\n"
        ::"r"(d_tmem), "r"(idesc), "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3])
        : "memory");
  }
}
// D (+)= A B over 4 k-steps, A in tensor memory; the first k-step accumulates only if `accumulate`
__device__ __forceinline__ void umma_ts_group(uint32_t d_tmem, const uint32_t (&a)[4], const uint64_t (&b)[4], uint32_t idesc,
                                              uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p, t;\n"
      "setp.ne.b32 p, %2, 0;\n"
      "setp.eq.b32 t, %0, %0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%3], %7, %1, p;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%4], %8, %1, t;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%5], %9, %1, t;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%6], %10, %1, t;\n"
      "}\n"
      ::"r"(d_tmem), "r"(idesc), "r"(accumulate), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "l"(b[0]), "l"(b[1]), "l"(b[2]),
        "l"(b[3])
      : "memory");
}

// ---- two-wide fp32 arithmetic and friends ------------------------------------------------------
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
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
// {lo, hi} -> packed bf16 pair, lo in the low half
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x for a pair of values on the fma pipe: x = n + r with n = round(x) (the low mantissa bits of x + 1.5 * 2^23)
// and r in [-0.5, 0.5]; 2^r by a cubic (relative error 7.5e-5, a thirtieth of a bf16 rounding step), 2^n by
// adding n to the exponent field.  x is clamped at -125 from below (the result is then 2^-125 instead of 0).
// PRECONDITION: x <= 127.  Above that the exponent field wraps and the result is garbage of either sign, so
// callers use this only where x is bounded by construction (a softmax argument after its reference maximum is
// known).
__device__ __forceinline__ void ex2_fma_pair(uint64_t x, float& p0, float& p1) {
  float x0, x1;
  unpack2(x, x0, x1);
  const uint64_t xc = pack2(fmaxf(x0, -125.f), fmaxf(x1, -125.f));
  const uint64_t t = add2(xc, pack2(12582912.f, 12582912.f));
  const uint64_t r = add2(xc, fma2(t, pack2(-1.f, -1.f), pack2(12582912.f, 12582912.f)));  // x - (t - magic)
  uint64_t q = fma2(pack2(0.0551716648f, 0.0551716648f), r, pack2(0.2426111251f, 0.2426111251f));
  q = fma2(q, r, pack2(0.6932609677f, 0.6932609677f));
  q = fma2(q, r, pack2(0.9999280572f, 0.9999280572f));
  float t0, t1, q0, q1;
  unpack2(t, t0, t1);
  unpack2(q, q0, q1);
  p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
  p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

}  // namespace sm100
}  // namespace fc
