// hga_route_static: hga_route for callers that must not allocate device memory.
//
// hga_route needs a scratch buffer (the fp32 score of every candidate chunk of every item)
// that its caller allocates.  Some callers cannot do that: a plug-in that runs while the host
// framework's allocator is locked or has handed out all device memory, a latency-critical
// loop that must never enter cudaMalloc (it synchronises the whole device), a process whose
// device memory was budgeted to the last byte at start-up.  For them the scratch lives here,
// in a fixed array that is part of the library image: every GPU that has run this entry point
// holds HGA_ROUTE_STATIC_SCRATCH_BYTES of it until the process exits.  (CUDA loads a module's
// device data when something in the module is first used, so the array becomes resident with
// the address look-up of the first call on a device -- that first call is the one moment at
// which this entry point makes the driver reserve device memory.)
#include <mutex>

#include "hga_common.cuh"

namespace hga {

// The name below is only a host-side handle in host code; kernels are given the device
// address obtained with cudaGetSymbolAddress (once per device, with that device current).
static __device__ __align__(256) unsigned char g_route_scratch[HGA_ROUTE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static void* g_scratch_addr[kMaxDevices];
static std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device; set-up on first use.
static int scratch_on_current_device(void** out) {
  int dev = -1;
  int rc = record_cuda(cudaGetDevice(&dev));
  if (rc) return rc;
  if (dev < 0 || dev >= kMaxDevices) return HGA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    rc = record_cuda(cudaGetSymbolAddress(&p, g_route_scratch));
    if (rc) return rc;
    if (!p) return HGA_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return HGA_OK;
}

}  // namespace hga

using namespace hga;

extern "C" int hga_route_static(const hga_params* p, const void* Q, const void* chunk_sum,
                                const void* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                                int32_t* n_groups, void* stream) {
  Dims dm;
  int rc = resolve_params(p, dm);
  if (rc) return rc;
  if (!Q || !chunk_sum || !group_sum || !n_groups) return HGA_ERR_NULL;
  if (dm.kc > 0 && (!chunk_idx || !group_idx)) return HGA_ERR_NULL;
  auto misaligned = [](const void* x) { return (reinterpret_cast<uintptr_t>(x) & 15) != 0; };
  if (misaligned(Q) || misaligned(chunk_sum) || misaligned(group_sum)) return HGA_ERR_ALIGN;
  // the fixed array bounds the problem size: refuse anything larger, launch nothing (also where the
  // fused router below would not need the array, so that the limit does not depend on the shape)
  if (route_workspace_bytes(dm) > (size_t)HGA_ROUTE_STATIC_SCRATCH_BYTES) return HGA_ERR_WORKSPACE;
  void* scratch = nullptr;
  rc = scratch_on_current_device(&scratch);
  if (rc) return rc;
  // Shapes the fused tensor-core router takes keep every score on chip: it runs first, as in
  // hga_route, and the array stays untouched.  Other shapes go to the CUDA-core router below.
  if (route_sm100_supported(dm)) {
    rc = launch_route_sm100(dm, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, nullptr, nullptr,
                            (cudaStream_t)stream);
    if (rc != HGA_ERR_UNSUPPORTED) return rc;
  }
  // Every score the selection kernels read is written earlier in the same call, so nothing in
  // the array has to start at zero and the previous call's contents are simply overwritten.
  return launch_route_generic(dm, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, nullptr,
                              nullptr, scratch, (cudaStream_t)stream);
}
