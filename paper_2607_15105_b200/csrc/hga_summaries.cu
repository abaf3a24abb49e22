// hga_build_summaries: mean-key summaries of groups and chunks (Section 2.1).
//
// HBM streaming kernel: every key row of the range is read exactly once with 16-byte
// loads (a warp covers two 256-byte rows of d = 128), sums are carried in fp64 so the
// mean of up to 2^38-spread bf16 values is exact, and the result is rounded once to bf16.
// One CTA per (chunk, batch*kv_head), one warp per group; the chunk sum is the sum of its
// group sums (exact in fp64, so the order does not matter).
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

// One CTA per (chunk, batch*kv head), one warp per group (warps loop when a chunk has more groups than the
// CTA has warps).  A warp's 32 lanes cover 32 / (D/8) consecutive rows per load instruction, 16 bytes per
// lane, and request up to four such row sets before the first sum: the kernel is one round trip to memory
// deep, which is what bounds a 4 MB stream spread over the whole GPU.
template <int D>
__global__ void __launch_bounds__(512)
k_build_summaries(const uint16_t* __restrict__ K, Dims dm, int chunk_begin,
                  uint16_t* __restrict__ chunk_sum, uint16_t* __restrict__ group_sum) {
  constexpr int VEC = D / 8;                  // lanes across one row
  constexpr int RPI = 32 / VEC;               // rows per load instruction
  extern __shared__ double part[];            // [warps][D]: per-warp sums of the groups it handled
  const int j = chunk_begin + blockIdx.x;     // chunk id
  const int bh = blockIdx.y;
  const int b = bh / dm.Hkv, h = bh % dm.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  const int v = lane % VEC, sub = lane / VEC;
  const uint16_t* Kb = K + b * dm.ks[0] + h * dm.ks[1] + v * 8;

  double csum[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) csum[e] = 0.0;
  for (int u = warp; u < dm.per; u += n_warps) {
    double s[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) s[e] = 0.0;
    const int t0 = j * dm.c + u * dm.g;
    for (int r0 = 0; r0 < dm.g; r0 += 4 * RPI) {
      uint4 raw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = r0 + i * RPI + sub;
        raw[i] = r < dm.g ? *reinterpret_cast<const uint4*>(Kb + (int64_t)(t0 + r) * dm.ks[2]) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s[2 * e] += (double)__uint_as_float(w[e] << 16);
          s[2 * e + 1] += (double)__uint_as_float(w[e] & 0xffff0000u);
        }
      }
    }
    // the row sets of the warp's RPI lane groups: one exact sum per element (fp64 sums of bf16 values are exact)
#pragma unroll
    for (int off = VEC; off < 32; off <<= 1)
#pragma unroll
      for (int e = 0; e < 8; ++e) s[e] += __shfl_xor_sync(0xffffffffu, s[e], off);
    if (sub == 0) {
      uint32_t o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e)
        o[e] = (uint32_t)f64_to_bf16_once(s[2 * e] / (double)dm.g) |
               ((uint32_t)f64_to_bf16_once(s[2 * e + 1] / (double)dm.g) << 16);
      const int64_t m = (int64_t)bh * dm.NgS + (int64_t)j * dm.per + u;
      *reinterpret_cast<uint4*>(group_sum + m * D + v * 8) = make_uint4(o[0], o[1], o[2], o[3]);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) csum[e] += s[e];
  }
  if (sub == 0) {
#pragma unroll
    for (int e = 0; e < 8; ++e) part[warp * D + v * 8 + e] = csum[e];
  }
  __syncthreads();
  if (warp == 0 && sub == 0) {
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      double a = 0.0, c2 = 0.0;
      for (int s2 = 0; s2 < n_warps; ++s2) {
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
  const int n_warps = dm.per < 16 ? dm.per : 16;
  dim3 grid((tok_end - tok_begin) / dm.c, dm.B * dm.Hkv);
  dim3 block(n_warps * 32);
  size_t smem = (size_t)n_warps * dm.d * sizeof(double);
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
