// Small device helpers shared by the two tensor-core backward kernels (routed sweep and local band).
#pragma once

#include <cuda_bf16.h>

#include "hga_sm100.cuh"
#include "hga_trace.cuh"

namespace hga {

// Bounded wait on an mbarrier phase.  Gives up after the time limit (sets the CTA's abort flag) or as
// soon as another thread of the CTA has given up; the caller then unwinds without touching TMEM.
//
// Diagnostic build (`python -m paper_2607_15105_b200.build --debug-waits`, i.e. -DHGA_DEBUG_WAIT; off by
// default): a wait that gives up records, per warp, its source line, parity and barrier address (the
// first failure since the last read); hga_debug_dump() copies the 64 ints out, and the status word carries
// the source line of the CTA's first failed wait in bits 8-27 and a kernel number in bits 28-30.  This is
// how a missed barrier phase shows which roles were waiting for what.
#ifdef HGA_DEBUG_WAIT
static __device__ int g_dbg_fail[64];     // [w] line | parity << 16, [16 + w] barrier address, [32 + w] block | blockDim << 16
#endif
__device__ __forceinline__ bool bwd_wait_(uint64_t* bar, uint32_t parity, volatile int* abort, int code) {
  if (sm100::mbar_test_wait(bar, parity)) return true;    // fast path: the phase is already over
  const bool fine = sm100::mbar_wait_bounded(bar, parity, abort, sm100::kWaitCycles, code);
#ifdef HGA_DEBUG_WAIT
  if (!fine && g_dbg_fail[threadIdx.x >> 5] == 0) {
    g_dbg_fail[threadIdx.x >> 5] = code | ((int)parity << 16);
    g_dbg_fail[32 + (threadIdx.x >> 5)] = (int)blockIdx.x | ((int)blockDim.x << 16);
    g_dbg_fail[16 + (threadIdx.x >> 5)] = (int)sm100::smem_u32(bar);
  }
#endif
  return fine;
}
#ifdef HGA_DEBUG_WAIT
#define bwd_wait(bar, parity, abort) bwd_wait_((bar), (parity), (abort), __LINE__)
#define HGA_ABORT_CODE(kernel, flag) (HGA_STATUS_WAIT_TIMEOUT | ((flag) << 8) | ((kernel) << 28))
#else
#define bwd_wait(bar, parity, abort) bwd_wait_((bar), (parity), (abort), 1)
#define HGA_ABORT_CODE(kernel, flag) HGA_STATUS_WAIT_TIMEOUT
#endif

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
