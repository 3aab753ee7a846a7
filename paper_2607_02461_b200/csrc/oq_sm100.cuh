// Thin wrappers around the sm_100a instructions both kernels use: mbarriers with bounded waits, the
// shared-memory matrix descriptor of tcgen05.mma, tensor-memory loads.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace oq {

constexpr long long WAIT_CYCLES = 4000000000ll;   // ~2 s: a wait that lasts longer reports and gives up

enum { WAIT_EMPTY = 1, WAIT_FULL = 2, WAIT_ACC_FULL = 3, WAIT_ACC_EMPTY = 4, WAIT_SELFTEST = 9 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  On expiry (or when another thread of the CTA / any CTA already gave up) it records
// `code` in the global status word, raises the CTA's abort flag and returns; callers carry on to the
// common tear-down so tensor memory is always released.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          int code, long long max_cycles = WAIT_CYCLES, unsigned sleep_ns = 32) {
  if (mbar_try(bar, parity)) return;
  const long long t0 = clock64();
  int polls = 0;
  while (!mbar_try(bar, parity)) {
    __nanosleep(sleep_ns);   // a waiting lane should not take issue slots from the warps it waits for
    if (*abort_flag) return;
    if ((++polls & 1023) == 0) {
      if (*reinterpret_cast<volatile int*>(status) != 0 || clock64() - t0 > max_cycles) {
        atomicCAS(status, 0, code);
        *abort_flag = 1;
        return;
      }
    }
  }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// 32 lanes x 32 consecutive fp32 columns of tensor memory: thread i of the warp gets lane base + i.
__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------------------
// Two-SM variant: a cluster of two CTAs computes one 256 x 256 tile with tcgen05.mma.cta_group::2.  Each
// CTA decodes its own 128 token rows of A and its own 128 feature rows of B (the tensor cores of both SMs
// read both halves of B, so every decoded byte of B is written once and used by 256 output rows), holds
// 128 x 256 fp32 accumulators, double-buffered in its 512 TMEM columns, and stores its own 128 rows of Y.
// CTA 0 of the pair issues the MMAs; "stage full" and "accumulator drained" arrivals from CTA 1 go to
// CTA 0's barriers through the cluster address window, "stage free" and "accumulator ready" come back to
// both CTAs with one multicast tcgen05.commit.  Dedicated epilogue warps overlap the epilogue of a tile
// with the main loop of the next one.

// The same for 16 consecutive columns, without waiting: the caller issues tcgen05.wait::ld before using r.
__device__ __forceinline__ void tmem_load16_nowait(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 32 lanes x 32 consecutive 32-bit columns of tensor memory: thread i of the warp writes lane base + i.
__device__ __forceinline__ void tmem_store32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

}  // namespace oq
