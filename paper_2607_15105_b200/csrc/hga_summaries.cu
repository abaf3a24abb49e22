// hga_build_summaries: mean-key summaries of groups and chunks (Section 2.1).
//
// HBM streaming kernel: every key row of the range is read exactly once with 16-byte
// loads (a warp covers two 256-byte rows of d = 128), sums are carried in fp64 so the
// mean of up to 2^38-spread bf16 values is exact, and the result is rounded once to bf16.
// One CTA per (chunk, batch*kv_head): thread (u, v) sums group u's rows for the 8
// elements [8v, 8v+8); the chunk sum is the fixed-order sum of its group sums.
#include "hga_common.cuh"

namespace hga {

// Round a double to bf16, nearest-even, with a single rounding: truncate to fp32, fold
// everything lost into the last fp32 bit (round-to-odd), then let the fp32 -> bf16
// conversion round.  fp32 keeps 16 more bits than bf16, so no double rounding occurs.
__device__ inline uint16_t f64_to_bf16_once(double x) {
  float f = __double2float_rz(x);
  if ((double)f != x) f = __uint_as_float(__float_as_uint(f) | 1u);
  return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

template <int D>
__global__ void __launch_bounds__(1024)
k_build_summaries(const uint16_t* __restrict__ K, Dims dm, int chunk_begin,
                  uint16_t* __restrict__ chunk_sum, uint16_t* __restrict__ group_sum) {
  constexpr int VEC = D / 8;                  // threads across one row
  extern __shared__ double part[];            // [group slots][D]
  const int j = chunk_begin + blockIdx.x;     // chunk id
  const int bh = blockIdx.y;
  const int b = bh / dm.Hkv, h = bh % dm.Hkv;
  const int v = threadIdx.x % VEC;
  const int slot = threadIdx.x / VEC;
  const int slots = blockDim.x / VEC;
  const uint16_t* Kb = K + b * dm.ks[0] + h * dm.ks[1];

  double csum[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) csum[e] = 0.0;
  for (int u = slot; u < dm.per; u += slots) {
    double s[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) s[e] = 0.0;
    const int t0 = j * dm.c + u * dm.g;
    for (int t = t0; t < t0 + dm.g; ++t) {
      const uint4 raw = *reinterpret_cast<const uint4*>(Kb + (int64_t)t * dm.ks[2] + v * 8);
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        s[2 * e] += (double)__uint_as_float(w[e] << 16);
        s[2 * e + 1] += (double)__uint_as_float(w[e] & 0xffff0000u);
      }
    }
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      o[e] = (uint32_t)f64_to_bf16_once(s[2 * e] / (double)dm.g) |
             ((uint32_t)f64_to_bf16_once(s[2 * e + 1] / (double)dm.g) << 16);
      csum[2 * e] += s[2 * e];
      csum[2 * e + 1] += s[2 * e + 1];
    }
    const int64_t m = (int64_t)bh * dm.NgS + (int64_t)j * dm.per + u;
    *reinterpret_cast<uint4*>(group_sum + m * D + v * 8) = make_uint4(o[0], o[1], o[2], o[3]);
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) part[slot * D + v * 8 + e] = csum[e];
  __syncthreads();
  if (slot == 0) {
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      double a = 0.0, c2 = 0.0;
      for (int s2 = 0; s2 < slots; ++s2) {
        a += part[s2 * D + v * 8 + 2 * e];
        c2 += part[s2 * D + v * 8 + 2 * e + 1];
      }
      o[e] = (uint32_t)f64_to_bf16_once(a / (double)dm.c) |
             ((uint32_t)f64_to_bf16_once(c2 / (double)dm.c) << 16);
    }
    const int64_t jj = (int64_t)bh * dm.NcS + j;
    *reinterpret_cast<uint4*>(chunk_sum + jj * D + v * 8) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

int launch_build_summaries(const Dims& dm, const void* K, int tok_begin, int tok_end,
                           void* chunk_sum, void* group_sum, cudaStream_t st) {
  const int vec = dm.d / 8;
  int slots = dm.per;
  while (slots * vec > 1024) slots = (slots + 1) / 2;
  dim3 grid((tok_end - tok_begin) / dm.c, dm.B * dm.Hkv);
  dim3 block(slots * vec);
  size_t smem = (size_t)slots * dm.d * sizeof(double);
  auto Kp = (const uint16_t*)K;
  auto cs = (uint16_t*)chunk_sum;
  auto gs = (uint16_t*)group_sum;
  if (dm.d == 128)
    k_build_summaries<128><<<grid, block, smem, st>>>(Kp, dm, tok_begin / dm.c, cs, gs);
  else
    k_build_summaries<64><<<grid, block, smem, st>>>(Kp, dm, tok_begin / dm.c, cs, gs);
  count_launch(HGA_KERNELS_SUMMARIES);
  return record_cuda(cudaGetLastError());
}

}  // namespace hga
