// mbarrier hand-over between producer and consumer warps, with bounded waits.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "m2rnn.h"

namespace m2rnn {

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// release.cta arrive: shared-memory writes made before it are visible to a thread whose wait
// on the completed phase succeeds
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Warp-collective bounded wait for the phase with the given parity.  Returns false for the
// whole warp if the limit runs out (about a second of SM clocks), never spins for ever.
// kSleepNs > 0: for waits that are expected to be long and whose end nobody is waiting for (a
// staging warp far ahead of its consumers): the polls of a tight loop would take issue slots
// from the warps that do the work.
// `limit` is in SM clocks; the kernels pass the default, the library's self-test a few thousand.
constexpr long long kWaitCycles = 1ll << 31;
template <uint32_t kSleepNs = 0>
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, long long limit = kWaitCycles) {
  bool ok = mbar_try_wait(bar, parity);
  if (!ok) {
    const long long t0 = clock64();
    uint32_t it = 0;
    for (;;) {
      if constexpr (kSleepNs > 0) __nanosleep(kSleepNs);
      else if (it > 64) __nanosleep(32);
      ok = mbar_try_wait(bar, parity);
      if (ok) break;
      // the clock is read every 32nd poll only: a poll is a handful of instructions, and polling
      // warps share issue slots with the warps that do the work
      if ((++it & 31u) == 0u && clock64() - t0 > limit) break;
    }
  }
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void report_timeout(int32_t *dev_status) {
  if (dev_status) atomicExch(dev_status, (int32_t)M2RNN_ERR_TIMEOUT);
}

// Explicit shared-window accesses by 32-bit shared address: a pointer selected at run time between
// stages may otherwise be treated as generic, which costs latency on every access of the hot loop.
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 lds64(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float lds32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, float4 v) {
  asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t addr, float2 v) {
  asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(addr), "f"(v.x), "f"(v.y) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t addr, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// 8 bf16 (one 16-byte load) widened to 8 floats in shared memory
__device__ __forceinline__ void store8_bf16_as_f32(float *dst, const uint4 raw) {
  float4 lo, hi;
  lo.x = __uint_as_float(raw.x << 16); lo.y = __uint_as_float(raw.x & 0xffff0000u);
  lo.z = __uint_as_float(raw.y << 16); lo.w = __uint_as_float(raw.y & 0xffff0000u);
  hi.x = __uint_as_float(raw.z << 16); hi.y = __uint_as_float(raw.z & 0xffff0000u);
  hi.z = __uint_as_float(raw.w << 16); hi.w = __uint_as_float(raw.w & 0xffff0000u);
  *reinterpret_cast<float4 *>(dst) = lo;
  *reinterpret_cast<float4 *>(dst + 4) = hi;
}

}  // namespace m2rnn
