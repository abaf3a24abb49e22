// Small device helpers shared by the two tensor-core backward kernels (routed sweep and local band).
#pragma once

#include <cuda_bf16.h>

#include "hga_sm100.cuh"

// Optional phase timers: a profiling harness defines these three macros; otherwise no-ops.
#ifndef HGA_TRACE_POINT
#define HGA_TRACE_DECL
#define HGA_TRACE_POINT(tag)
#define HGA_TRACE_DUMP
#endif

namespace hga {

// Bounded wait on an mbarrier phase.  Gives up after the time limit (sets the CTA's abort flag) or as
// soon as another thread of the CTA has given up; the caller then unwinds without touching TMEM.
__device__ __forceinline__ bool bwd_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
  if (sm100::mbar_test_wait(bar, parity)) return true;    // fast path: the phase is already over
  return sm100::mbar_wait_bounded(bar, parity, abort);
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

}  // namespace hga
