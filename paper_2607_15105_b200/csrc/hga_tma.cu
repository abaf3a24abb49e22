// Host-side tensor-map encoding for the TMA loads of the tensor-core kernels.  The driver's
// encoder is looked up at run time, so the library has no link-time dependency on libcuda.
#include <cudaTypedefs.h>

#include <cstring>
#include <mutex>
#include <unordered_map>

#include "hga_common.cuh"
#include "hga_sm100.cuh"

namespace hga {

static PFN_cuTensorMapEncodeTiled_v12000 lookup_encoder() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q);
    if (e == cudaSuccess && q == cudaDriverEntryPointSuccess) fn = (PFN_cuTensorMapEncodeTiled_v12000)p;
    else (void)cudaGetLastError();
  });
  return fn;
}

// Encoded maps are cached: a training loop calls with the same pointers, sizes and strides step after
// step, and an encode costs more host time than the rest of a launch.  The key is everything the
// encoder sees (plus the device); the table is small and simply emptied when it fills up.
namespace {
struct MapKey {
  const void* base;
  int device, rank, swizzle;
  uint64_t dims[5], strides[4];
  uint32_t box[5];
  bool operator==(const MapKey& o) const { return memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    const uint64_t* w = reinterpret_cast<const uint64_t*>(&k);
    uint64_t h = 1469598103934665603ull;
    for (size_t i = 0; i < sizeof(MapKey) / 8; ++i) h = (h ^ w[i]) * 1099511628211ull;
    return (size_t)h;
  }
};
static_assert(sizeof(MapKey) % 8 == 0, "hashed as 64-bit words");
std::mutex g_map_mutex;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;
constexpr size_t kMaxCachedMaps = 512;
}  // namespace

int encode_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                           const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128) {
  auto enc = lookup_encoder();
  if (!enc) return -1;
  MapKey key;
  memset(&key, 0, sizeof key);
  key.base = base;
  key.rank = rank;
  key.swizzle = swizzle128;
  if (cudaGetDevice(&key.device) != cudaSuccess) return -1;
  for (int i = 0; i < rank; ++i) {
    key.dims[i] = dims[i];
    key.box[i] = box[i];
    if (i > 0) key.strides[i - 1] = strides_bytes[i - 1];
  }
  {
    std::lock_guard<std::mutex> lock(g_map_mutex);
    auto it = g_maps.find(key);
    if (it != g_maps.end()) { *out = it->second; return 0; }
  }
  cuuint64_t gdim[5];
  cuuint64_t gstr[4];
  cuuint32_t bx[5], estr[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bx[i] = box[i];
    estr[i] = 1;
    if (i > 0) gstr[i - 1] = strides_bytes[i - 1];
  }
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim,
                   gstr, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return (int)r;
  std::lock_guard<std::mutex> lock(g_map_mutex);
  if (g_maps.size() >= kMaxCachedMaps) g_maps.clear();
  g_maps.emplace(key, *out);
  return 0;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize [, maximal shared-memory carve-out]) once per (device,
// kernel, size): the attribute sticks, and the call is not free.
int ensure_dynamic_smem(const void* func, size_t bytes, bool max_carveout) {
  static std::mutex mu;
  static std::unordered_map<uint64_t, size_t> done;     // (device, function) -> largest size set
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda(e);
  const uint64_t key = (uint64_t)reinterpret_cast<uintptr_t>(func) * 64 + (uint64_t)dev;
  {
    std::lock_guard<std::mutex> lock(mu);
    auto it = done.find(key);
    if (it != done.end() && it->second >= bytes) return HGA_OK;
  }
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && max_carveout)
    e = cudaFuncSetAttribute(func, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return record_cuda(e);
  std::lock_guard<std::mutex> lock(mu);
  size_t& v = done[key];
  if (v < bytes) v = bytes;
  return HGA_OK;
}

}  // namespace hga
