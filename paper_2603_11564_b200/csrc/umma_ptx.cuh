// Inline-PTX helpers for the tensor-core scorer: mbarriers with bounded waits, TMA tile loads,
// tcgen05 MMA / tensor-memory loads and stores, and the descriptors they take.
#pragma once
#include <cuda.h>
#include <math_constants.h>
#include <stdint.h>

#include "dapq_internal.cuh"

namespace dapq {
namespace ptx {

constexpr long long kWaitLimit = 2000000000LL; // cycles (~1 s)

// ------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// The same test, but the thread may be suspended by the hardware for up to ~`ns` nanoseconds while the
// phase is incomplete (it resumes as soon as the phase completes): a waiting warp then costs the
// scheduler a few instructions per microsecond instead of a tight polling loop.
__device__ __forceinline__ bool mbar_try_suspend(uint32_t bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
  return ok != 0;
}
// Bounded wait of at most `limit` cycles.  Returns false if the CTA is aborting (this or another
// wait ran out): the caller then leaves its loop, and the CTA drains and returns normally.
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                                long long limit) {
  if (mbar_try(bar, parity)) return true;
  const long long start = clock64();
  while (true) {
    // (the clock is read before the suspended try, so that a limit of a few cycles gives up on the first wait
    // that is not satisfied at once, whatever the suspension hides)
    if (clock64() - start > limit) {
      *abort_flag = 1;
      atomicOr(status, kStatusTimeout);
      return false;
    }
    // (a burst of suspended tries between two looks at the flag and the clock: a waiting warp should cost the
    // schedulers as few instructions as possible, they are the epilogue's)
#pragma unroll 1
    for (int it = 0; it < 16; ++it)
      if (mbar_try_suspend(bar, parity, 20000u)) return true;
    if (*abort_flag) return false;
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  return mbar_wait_limit(bar, parity, abort_flag, status, kWaitLimit);
}
// Plain bounded wait that no abort cuts short: used to see copies and MMAs in flight complete before a
// CTA returns.
__device__ __forceinline__ void drain_wait(uint32_t bar, uint32_t parity, long long limit) {
  const long long start = clock64();
  while (!mbar_try(bar, parity) && clock64() - start < limit) {}
}
// Generic-proxy writes to shared memory (st.shared) become visible to the async proxy (TMA, tcgen05.mma
// operand reads) that is ordered after this fence.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row
// groups 1024 bytes apart (the layout a TMA box of 64 bf16 x rows with SWIZZLE_128B writes).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// The same for a K-major operand whose rows are 32 bytes (16 half-precision channels, one MMA k-step) with
// the 32-byte swizzle: 8-row groups 256 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_rows32(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(256 >> 4) << 32) | (1ull << 46) |
         (6ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, shape M x N.
__host__ __device__ constexpr uint32_t umma_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
// The same for fp16 x fp16 -> fp32 (operand format fields 0).
__host__ __device__ constexpr uint32_t umma_idesc_f16(int m, int n) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
// D (tensor memory) (+)= A (shared memory) B (shared memory)
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
// Wait for this thread's outstanding tensor-memory loads (16-register form, see tmem_ld_wait_for).
__device__ __forceinline__ void tmem_ld_wait_for16(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :: "memory");
}
// Wait for this thread's outstanding tensor-memory loads.  The registers of the load being
// waited for are passed through so that no use of them can be scheduled above the wait.
__device__ __forceinline__ void tmem_ld_wait_for(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                 "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :: "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x on the FMA / ALU pipes instead of the MUFU: round-to-nearest split x = n + f with the
// 1.5 * 2^23 trick, a degree-3 minimax polynomial for 2^f on [-0.5, 0.5] (relative error below
// 7.5e-5), and n added into the exponent field.  Inputs below -125 give 2^-125.  The scorer's
// epilogues owe one exponential per (query, key) pair and the MUFU pipe delivers only 16 per
// clock and SM, so a quarter of the column pairs of a piece takes this path.  Everything works
// on two values at once with the packed fp32 instructions of sm_100 (one FFMA2 / FADD2 per
// register pair): 2^x.x and 2^x.y on the MUFU, or both by the polynomial.
#ifndef DAPQ_POLY_PAIR_MASK
#define DAPQ_POLY_PAIR_MASK 0x8888u
#endif
constexpr uint32_t kPolyPairMask = DAPQ_POLY_PAIR_MASK;   // bit p: pair p of a 32-column piece takes the polynomial
__device__ __forceinline__ float2 ex2_pair_mufu(float2 x) { return make_float2(ex2(x.x), ex2(x.y)); }
// kSat: inputs above 128 give 2^128-ish values (> 1.7e38) instead of wrapping the exponent field, for callers
// that detect overflow by the size of the result.
template <bool kSat = false>
__device__ __forceinline__ float2 ex2_pair_poly(float2 x) {
  x.x = fmaxf(x.x, -125.f);
  x.y = fmaxf(x.y, -125.f);
  if (kSat) {
    x.x = fminf(x.x, 128.f);
    x.y = fminf(x.y, 128.f);
  }
  const float2 magic = make_float2(12582912.f, 12582912.f), neg_magic = make_float2(-12582912.f, -12582912.f);
  const float2 t = __fadd2_rn(x, magic);
  const float2 n = __fadd2_rn(t, neg_magic);
  const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
  float2 p = __ffma2_rn(make_float2(0.0551716648f, 0.0551716648f), f, make_float2(0.2426111251f, 0.2426111251f));
  p = __ffma2_rn(p, f, make_float2(0.6932609677f, 0.6932609677f));
  p = __ffma2_rn(p, f, make_float2(0.9999280572f, 0.9999280572f));
  return make_float2(__uint_as_float(__float_as_uint(p.x) + (__float_as_uint(t.x) << 23)),
                     __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(t.y) << 23)));
}

// Three-input maximum (one instruction on sm_100).
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// Barrier among the 16 epilogue warps only (the producer warps never join it).
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 1, 512;" ::: "memory"); }

// Descriptor of the operand `bytes` further on in shared memory (the start-address field is
// in 16-byte units in the low bits and never carries out of it for addresses below 256 KB).
__device__ __forceinline__ uint64_t desc_advance(uint64_t desc, int bytes) { return desc + (uint64_t)(bytes >> 4); }

}  // namespace ptx
}  // namespace dapq
