// Optional in-kernel timelines for the tensor-core kernels (off unless HGA_TRACE is defined).
//
// HGA_TRACE_POINT(tag) records (SM cycle counter, tag) for lane 0 of every warp of ONE chosen CTA of ONE
// chosen kernel (picked at run time through g_trace_threads = the kernel's block size and g_trace_blk = the
// block index); HGA_TRACE_DECL / HGA_TRACE_DUMP additionally record every CTA's SM id, start and end on
// the global timer.  The records go straight to global memory (the kernels have no shared memory to
// spare).  A point costs on the order of a hundred cycles, so a traced kernel is slower than the real
// one: read intervals, not totals.  The harness that sets the two selectors, runs the kernels on a
// configuration-3-shaped problem and prints the records is trace/hga_trace_harness.cu, built by
// `python -m paper_2607_15105_b200.build --trace`; the library itself is never built with HGA_TRACE.
#pragma once

#ifdef HGA_TRACE
#define HGA_TRACE_WARPS 16
#define HGA_TRACE_SLOTS 96
__device__ int g_trace_threads;
__device__ int g_trace_blk;
__device__ unsigned g_trace_log[HGA_TRACE_WARPS][HGA_TRACE_SLOTS];   // (cycles << 6) | tag
__device__ unsigned long long g_trace_cta[2048][3];                  // SM id, start, end (global timer, ns)
__device__ __forceinline__ unsigned long long hga_trace_gtimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ unsigned hga_trace_smid() {
  unsigned s;
  asm volatile("mov.u32 %0, %smid;" : "=r"(s));
  return s;
}
#define HGA_TRACE_DECL                                                                                  \
  int tr_n_ = 0;                                                                                        \
  const bool tr_on_ = (int)blockDim.x == g_trace_threads;                                               \
  if (tr_on_ && threadIdx.x == 0 && blockIdx.x < 2048) {                                                \
    g_trace_cta[blockIdx.x][0] = hga_trace_smid();                                                      \
    g_trace_cta[blockIdx.x][1] = hga_trace_gtimer();                                                    \
  }
#define HGA_TRACE_POINT(tag)                                                                            \
  do {                                                                                                  \
    if (tr_on_ && (threadIdx.x & 31) == 0 && (int)blockIdx.x == g_trace_blk) {                          \
      const int w_ = threadIdx.x >> 5;                                                                  \
      if (w_ < HGA_TRACE_WARPS && tr_n_ < HGA_TRACE_SLOTS)                                              \
        g_trace_log[w_][tr_n_++] = ((unsigned)clock64() << 6) | (tag);                                  \
    }                                                                                                   \
  } while (0)
#define HGA_TRACE_DUMP                                                                                  \
  do {                                                                                                  \
    if (tr_on_ && threadIdx.x == 0 && blockIdx.x < 2048) g_trace_cta[blockIdx.x][2] = hga_trace_gtimer(); \
  } while (0)
#else
#define HGA_TRACE_DECL
#define HGA_TRACE_POINT(tag)
#define HGA_TRACE_DUMP
#endif
