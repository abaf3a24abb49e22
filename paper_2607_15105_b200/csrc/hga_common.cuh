// Internal definitions shared by the libhga translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hga.h"

namespace hga {

// Block score aggregator selected by hga_params.flags: 0 maximum, 1 mean, 2 log-sum-exp over the rows.
__host__ __device__ inline int score_agg_of(int flags) {
  return (flags & HGA_FLAG_SCORE_MEAN) ? 1 : (flags & HGA_FLAG_SCORE_LSE) ? 2 : 0;
}

// Internal flag (a bit of Dims.flags that hga.h does not define and the exported calls reject): launch
// the backward's kernels without programmatic serialization.  Set by hga_step_host, whose steps are bound
// by the host link: there the early-started CTAs only get in the way of the next (batch, kv head) pair's
// kernels.
constexpr int kFlagNoPdl = 1 << 30;

// Resolved problem description handed to kernels by value.
struct Dims {
  int B, Hq, Hkv, G, d;
  int L, S, H;          // total, active segment, history = L - S
  int c, g, Bq;         // chunk, group, query block
  int kc, kg, kge, per; // k_c, k_g, min(k_g, c/g), c/g
  int sink, local;
  int NQB, Nc, Ng;      // query blocks per sequence, chunks, groups
  int NcS, NgS;         // rows per (batch, kv head) in the chunk / group summary buffers (>= Nc, Ng)
  int width;            // group_idx entries per item = kc * kge
  int rows;             // G * Bq query rows per item
  int flags;
  float scale;          // softmax scale
  int64_t qs[3], ks[3], vs[3], os[3];  // element strides (batch, head, token)
};

// Window geometry of a query block (local start, sink end), see hga.h.
struct Window {
  int p0, ls, se;
};

__host__ __device__ inline Window window_of(const Dims& dm, int qb) {
  Window w;
  w.p0 = dm.H + qb * dm.Bq;
  int l = w.p0 - dm.local;
  w.ls = l <= 0 ? 0 : (l / dm.c) * dm.c;
  w.se = dm.sink < w.ls ? dm.sink : w.ls;
  return w;
}

__host__ __device__ inline void item_coords(const Dims& dm, int item, int& b, int& h, int& qb) {
  qb = item % dm.NQB;
  int bh = item / dm.NQB;
  h = bh % dm.Hkv;
  b = bh / dm.Hkv;
}

// Row layout of an item inside the tensor-core kernels: every query head's Bq rows are padded to
// whole octets (8 rows = one TMA box / swizzle atom), so row r of the item is (head r / bq_pad,
// token r % bq_pad) and rows with token >= Bq are padding.  Bq is a multiple of 8 except in
// generation-shaped problems (HGA_FLAG_DECODE), where bq_pad = 8 or 16 for 1..16 new tokens.
__host__ __device__ inline int bq_padded(const Dims& dm) { return (dm.Bq + 7) & ~7; }
__host__ __device__ inline int rows_padded(const Dims& dm) { return dm.G * bq_padded(dm); }

// Upper bound of routed tokens per item (sink + groups + local window + the block itself).
__host__ __device__ inline int max_routed_tokens(const Dims& dm) {
  return dm.sink + dm.width * dm.g + dm.local + dm.Bq + dm.c;
}

// cudaFuncSetAttribute(max dynamic shared memory [, maximal carve-out]) for `func`, cached per device (hga_tma.cu)
int ensure_dynamic_smem(const void* func, size_t bytes, bool max_carveout = false);

// Launch bookkeeping (hga_api.cu).
void count_launch(int family, int n = 1);   // family: HGA_KERNELS_*
int record_cuda(cudaError_t e);  // returns HGA_OK or HGA_ERR_CUDA and remembers the code

// Kernel launchers, one per translation unit.  All return an HGA status.
int launch_build_summaries(const Dims& dm, const void* K, int tok_begin, int tok_end,
                           void* chunk_sum, void* group_sum, cudaStream_t st);
int launch_route_generic(const Dims& dm, const void* Q, const void* chunk_sum,
                         const void* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                         int32_t* n_groups, float* chunk_scores, float* group_scores,
                         void* workspace, cudaStream_t st);
int launch_attn_fwd_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                            const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                            int32_t* status_word, cudaStream_t st);
int launch_attn_bwd_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                            const void* O, const float* LSE, const void* dO,
                            const int32_t* group_idx, const int32_t* n_groups, void* dQ, float* dK,
                            float* dV, float* delta_ws, int32_t* status_word, cudaStream_t st);

// tensor-core (tcgen05 / TMEM / TMA) kernels; *_supported says whether the shape qualifies
bool attn_fwd_sm100_supported(const Dims& dm);
int launch_attn_fwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V,
                          const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                          int32_t* status_word, cudaStream_t st);

bool route_sm100_supported(const Dims& dm);
int launch_route_sm100(const Dims& dm, const void* Q, const void* chunk_sum, const void* group_sum,
                       int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, float* chunk_scores,
                       float* group_scores, cudaStream_t st);
bool attn_bwd_sm100_supported(const Dims& dm);
int launch_attn_bwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const void* O,
                          const float* LSE, const void* dO, const int32_t* group_idx,
                          const int32_t* n_groups, void* dQ, float* dK, float* dV, int32_t* status_word,
                          cudaStream_t st);
// Key-major dK/dV of the local band (plain stores covering every active-segment row); launched by the above.
bool attn_bwd_band_sm100_supported(const Dims& dm);
int launch_attn_bwd_band_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const void* O,
                               const float* LSE, const void* dO, float* dK, float* dV, int32_t* status_word,
                               cudaStream_t st);

// Validates an hga_params block and fills the resolved description (hga_api.cu).
int resolve_params(const hga_params* p, Dims& dm);

size_t route_workspace_bytes(const Dims& dm);
size_t bwd_workspace_bytes(const Dims& dm);

// fp32 -> bf16 (round to nearest even): src holds n dK sums followed by n dV sums, n a multiple of 8; one
// launch for both tensors.  after_sweep: launched with programmatic serialization behind the tensor-core sweep
// (which releases it early in that mode), so that its launch overlaps the sweep's tail (hga_attn_generic.cu)
int launch_grads_to_bf16(const float* src, void* dst_k, void* dst_v, size_t n, bool after_sweep, cudaStream_t st);

}  // namespace hga
