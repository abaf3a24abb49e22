// Shape-generic CUDA-core kernels for routed exact-token attention (Section 2.1 item 3) and
// its backward under segment-wise TBPTT (Section 2.2).  One warp owns one query row (or,
// for dK/dV, one key row); a lane owns d/32 consecutive elements.  These kernels accept
// every shape hga_params allows and serve as the cross-check of the tensor-core kernels.
#include <cfloat>

#include "hga_common.cuh"

namespace hga {

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = kAttnThreads / 32;

template <int EPL>
struct Frag {
  float v[EPL];
};

// EPL consecutive bf16 -> fp32 (EPL = 2: one 32-bit load, EPL = 4: one 64-bit load)
template <int EPL>
__device__ inline Frag<EPL> load_frag(const uint16_t* p) {
  Frag<EPL> f;
  if constexpr (EPL == 2) {
    const uint32_t w = *reinterpret_cast<const uint32_t*>(p);
    f.v[0] = __uint_as_float(w << 16);
    f.v[1] = __uint_as_float(w & 0xffff0000u);
  } else {
    const uint2 w = *reinterpret_cast<const uint2*>(p);
    f.v[0] = __uint_as_float(w.x << 16);
    f.v[1] = __uint_as_float(w.x & 0xffff0000u);
    f.v[2] = __uint_as_float(w.y << 16);
    f.v[3] = __uint_as_float(w.y & 0xffff0000u);
  }
  return f;
}

template <int EPL>
__device__ inline void store_frag_bf16(uint16_t* p, const Frag<EPL>& f) {
  uint32_t w[EPL / 2];
#pragma unroll
  for (int i = 0; i < EPL / 2; ++i) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(f.v[2 * i], f.v[2 * i + 1]);
    w[i] = *reinterpret_cast<const uint32_t*>(&h);
  }
  if constexpr (EPL == 2) *reinterpret_cast<uint32_t*>(p) = w[0];
  else *reinterpret_cast<uint2*>(p) = make_uint2(w[0], w[1]);
}

template <int EPL>
__device__ inline float dot_frag(const Frag<EPL>& a, const Frag<EPL>& b) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < EPL; ++i) s = fmaf(a.v[i], b.v[i], s);
  return s;
}

__device__ inline float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// Builds the item's routed token list in shared memory: sink, valid groups, local window.
// Invalid group entries are skipped and reported.  Returns the number of tokens; s_meta[0]
// receives the number of valid groups.
__device__ int build_token_list(const Dims& dm, const Window& w, const int32_t* gi, int ng,
                                int* toks, int* s_meta, int32_t* status_word) {
  const int tid = threadIdx.x;
  // thread 0 validates sequentially (ascending, inside [se, ls)) and compacts group ids
  int* vg = toks + max_routed_tokens(dm);     // scratch for valid group ids, `width` entries
  if (tid == 0) {
    int n = 0, prev = -1, bad = 0;
    if (ng > dm.width) { ng = dm.width; bad = 1; }
    if (ng < 0) { ng = 0; bad = 1; }
    for (int i = 0; i < ng; ++i) {
      const int m = gi[i];
      const bool ok = m > prev && (int64_t)m * dm.g >= w.se && ((int64_t)m + 1) * dm.g <= w.ls;
      if (ok) { vg[n++] = m; prev = m; } else bad = 1;
    }
    s_meta[0] = n;
    if (bad && status_word) atomicOr(status_word, HGA_STATUS_BAD_INDEX);
  }
  __syncthreads();
  const int nvg = s_meta[0];
  const int n_far = w.se + nvg * dm.g;
  const int n_tok = n_far + (w.p0 + dm.Bq - w.ls);
  for (int i = tid; i < n_tok; i += blockDim.x) {
    int t;
    if (i < w.se) t = i;
    else if (i < n_far) t = vg[(i - w.se) / dm.g] * dm.g + (i - w.se) % dm.g;
    else t = w.ls + (i - n_far);
    toks[i] = t;
  }
  __syncthreads();
  return n_tok;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads)
k_attn_fwd_generic(const uint16_t* __restrict__ Q, const uint16_t* __restrict__ K,
                   const uint16_t* __restrict__ V, const int32_t* __restrict__ group_idx,
                   const int32_t* __restrict__ n_groups, Dims dm, uint16_t* __restrict__ O,
                   float* __restrict__ LSE, int32_t* status_word) {
  constexpr int EPL = D / 32;
  extern __shared__ int s_int[];
  __shared__ int s_meta[2];
  const int item = blockIdx.x;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);
  build_token_list(dm, w, group_idx + (int64_t)item * dm.width, n_groups[item], s_int, s_meta, status_word);
  const int n_far = w.se + s_meta[0] * dm.g;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint16_t* Kb = K + b * dm.ks[0] + h * dm.ks[1] + lane * EPL;
  const uint16_t* Vb = V + b * dm.vs[0] + h * dm.vs[1] + lane * EPL;
  for (int r = warp; r < dm.rows; r += kAttnWarps) {
    const int a = r / dm.Bq, t = r % dm.Bq;
    const int hq = h * dm.G + a, srow = qb * dm.Bq + t;
    const int pos = w.p0 + t;
    const int n_vis = n_far + (pos - w.ls + 1);
    const Frag<EPL> q = load_frag<EPL>(Q + b * dm.qs[0] + hq * dm.qs[1] + srow * dm.qs[2] + lane * EPL);
    float m = -FLT_MAX, l = 0.f;
    Frag<EPL> acc;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc.v[e] = 0.f;
    for (int i = 0; i < n_vis; i += 4) {
      float s[4];
      Frag<EPL> vv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int idx = i + u < n_vis ? i + u : n_vis - 1;
        const int64_t tok = s_int[idx];
        s[u] = dot_frag<EPL>(q, load_frag<EPL>(Kb + tok * dm.ks[2]));
        vv[u] = load_frag<EPL>(Vb + tok * dm.vs[2]);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) s[u] = warp_sum(s[u]) * dm.scale;
      float m_new = m;
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i + u < n_vis) m_new = fmaxf(m_new, s[u]);
      const float corr = __expf(m - m_new);
      l *= corr;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc.v[e] *= corr;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (i + u < n_vis) {
          const float p = __expf(s[u] - m_new);
          l += p;
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc.v[e] = fmaf(p, vv[u].v[e], acc.v[e]);
        }
      }
      m = m_new;
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc.v[e] *= inv;
    store_frag_bf16<EPL>(O + b * dm.os[0] + hq * dm.os[1] + srow * dm.os[2] + lane * EPL, acc);
    if (lane == 0) LSE[((int64_t)b * dm.Hq + hq) * dm.S + srow] = m + logf(l);
  }
}

// delta[row] = sum_e dO[row][e] * O[row][e]
template <int D>
__global__ void __launch_bounds__(kAttnThreads)
k_bwd_delta(const uint16_t* __restrict__ O, const uint16_t* __restrict__ dO, Dims dm,
            float* __restrict__ delta) {
  constexpr int EPL = D / 32;
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kAttnWarps + (threadIdx.x >> 5);
  const int64_t n_rows = (int64_t)dm.B * dm.Hq * dm.S;
  if (row >= n_rows) return;
  const int s = row % dm.S, hq = (row / dm.S) % dm.Hq, b = row / ((int64_t)dm.S * dm.Hq);
  const int64_t off = b * dm.os[0] + hq * dm.os[1] + s * dm.os[2] + lane * EPL;
  const float x = warp_sum(dot_frag<EPL>(load_frag<EPL>(O + off), load_frag<EPL>(dO + off)));
  if (lane == 0) delta[row] = x;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads)
k_bwd_dq_generic(const uint16_t* __restrict__ Q, const uint16_t* __restrict__ K,
                 const uint16_t* __restrict__ V, const uint16_t* __restrict__ dO,
                 const float* __restrict__ LSE, const float* __restrict__ delta,
                 const int32_t* __restrict__ group_idx, const int32_t* __restrict__ n_groups,
                 Dims dm, uint16_t* __restrict__ dQ, int32_t* status_word) {
  constexpr int EPL = D / 32;
  extern __shared__ int s_int[];
  __shared__ int s_meta[2];
  const int item = blockIdx.x;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);
  build_token_list(dm, w, group_idx + (int64_t)item * dm.width, n_groups[item], s_int, s_meta, status_word);
  const int n_far = w.se + s_meta[0] * dm.g;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint16_t* Kb = K + b * dm.ks[0] + h * dm.ks[1] + lane * EPL;
  const uint16_t* Vb = V + b * dm.vs[0] + h * dm.vs[1] + lane * EPL;
  for (int r = warp; r < dm.rows; r += kAttnWarps) {
    const int a = r / dm.Bq, t = r % dm.Bq;
    const int hq = h * dm.G + a, srow = qb * dm.Bq + t;
    const int n_vis = n_far + (w.p0 + t - w.ls + 1);
    const Frag<EPL> q = load_frag<EPL>(Q + b * dm.qs[0] + hq * dm.qs[1] + srow * dm.qs[2] + lane * EPL);
    const Frag<EPL> go = load_frag<EPL>(dO + b * dm.os[0] + hq * dm.os[1] + srow * dm.os[2] + lane * EPL);
    const int64_t row = ((int64_t)b * dm.Hq + hq) * dm.S + srow;
    const float lse = LSE[row], dl = delta[row];
    Frag<EPL> dq;
#pragma unroll
    for (int e = 0; e < EPL; ++e) dq.v[e] = 0.f;
    for (int i = 0; i < n_vis; i += 2) {
      float s[2], dp[2];
      Frag<EPL> kk[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int idx = i + u < n_vis ? i + u : n_vis - 1;
        const int64_t tok = s_int[idx];
        kk[u] = load_frag<EPL>(Kb + tok * dm.ks[2]);
        s[u] = dot_frag<EPL>(q, kk[u]);
        dp[u] = dot_frag<EPL>(go, load_frag<EPL>(Vb + tok * dm.vs[2]));
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        s[u] = warp_sum(s[u]);
        dp[u] = warp_sum(dp[u]);
        if (i + u < n_vis) {
          const float p = __expf(s[u] * dm.scale - lse);
          const float ds = p * (dp[u] - dl);
#pragma unroll
          for (int e = 0; e < EPL; ++e) dq.v[e] = fmaf(ds, kk[u].v[e], dq.v[e]);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) dq.v[e] *= dm.scale;
    store_frag_bf16<EPL>(dQ + b * dm.qs[0] + hq * dm.qs[1] + srow * dm.qs[2] + lane * EPL, dq);
  }
}

// dK/dV: one warp per routed ACTIVE key of the item (position >= H); history keys are
// detached constants (Section 2.2) and are skipped.  Partial sums over the item's rows stay
// in registers; one atomic add per element per (item, key) merges the query blocks.
template <int D>
__global__ void __launch_bounds__(kAttnThreads)
k_bwd_dkv_generic(const uint16_t* __restrict__ Q, const uint16_t* __restrict__ K,
                  const uint16_t* __restrict__ V, const uint16_t* __restrict__ dO,
                  const float* __restrict__ LSE, const float* __restrict__ delta,
                  const int32_t* __restrict__ group_idx, const int32_t* __restrict__ n_groups,
                  Dims dm, float* __restrict__ dK, float* __restrict__ dV) {
  constexpr int EPL = D / 32;
  extern __shared__ int s_int[];
  __shared__ int s_meta[2];
  const int item = blockIdx.x;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);
  const int n_tok = build_token_list(dm, w, group_idx + (int64_t)item * dm.width, n_groups[item],
                                     s_int, s_meta, nullptr);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint16_t* Qb = Q + b * dm.qs[0] + (int64_t)(h * dm.G) * dm.qs[1] + (int64_t)(qb * dm.Bq) * dm.qs[2] + lane * EPL;
  const uint16_t* dOb = dO + b * dm.os[0] + (int64_t)(h * dm.G) * dm.os[1] + (int64_t)(qb * dm.Bq) * dm.os[2] + lane * EPL;
  for (int i = warp; i < n_tok; i += kAttnWarps) {
    const int tok = s_int[i];
    if (tok < dm.H) continue;
    const Frag<EPL> kk = load_frag<EPL>(K + b * dm.ks[0] + h * dm.ks[1] + (int64_t)tok * dm.ks[2] + lane * EPL);
    const Frag<EPL> vv = load_frag<EPL>(V + b * dm.vs[0] + h * dm.vs[1] + (int64_t)tok * dm.vs[2] + lane * EPL);
    Frag<EPL> dk, dv;
#pragma unroll
    for (int e = 0; e < EPL; ++e) dk.v[e] = dv.v[e] = 0.f;
    const int t_first = tok > w.p0 ? tok - w.p0 : 0;    // causal: rows at or after the key
    for (int a = 0; a < dm.G; ++a) {
      const int64_t row0 = ((int64_t)b * dm.Hq + h * dm.G + a) * dm.S + qb * dm.Bq;
      for (int t = t_first; t < dm.Bq; ++t) {
        const Frag<EPL> q = load_frag<EPL>(Qb + a * dm.qs[1] + t * dm.qs[2]);
        const Frag<EPL> go = load_frag<EPL>(dOb + a * dm.os[1] + t * dm.os[2]);
        const float s = warp_sum(dot_frag<EPL>(q, kk));
        const float dp = warp_sum(dot_frag<EPL>(go, vv));
        const float p = __expf(s * dm.scale - LSE[row0 + t]);
        const float ds = p * (dp - delta[row0 + t]);
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          dk.v[e] = fmaf(ds, q.v[e], dk.v[e]);
          dv.v[e] = fmaf(p, go.v[e], dv.v[e]);
        }
      }
    }
    float* dKr = dK + (((int64_t)b * dm.Hkv + h) * dm.S + (tok - dm.H)) * D + lane * EPL;
    float* dVr = dV + (((int64_t)b * dm.Hkv + h) * dm.S + (tok - dm.H)) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      atomicAdd(dKr + e, dk.v[e] * dm.scale);
      atomicAdd(dVr + e, dv.v[e]);
    }
  }
}

static size_t token_smem_bytes(const Dims& dm) {
  return sizeof(int) * ((size_t)max_routed_tokens(dm) + dm.width + 4);
}

// dK/dV accumulators (fp32, adjacent: dV's follow dK's) -> the two bf16 outputs, eight elements per thread
__global__ void __launch_bounds__(256) k_grads_to_bf16(const float4* __restrict__ src, uint4* __restrict__ dst_k,
                                                       uint4* __restrict__ dst_v, size_t n8) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  // (a no-op unless launched with programmatic serialization: then the sums are complete only from here on)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (i >= 2 * n8) return;
  const float4 a = src[2 * i], b = src[2 * i + 1];
  const __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
  const __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
  uint4* dst = i < n8 ? dst_k + i : dst_v + (i - n8);
  *dst = make_uint4(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1),
                    *reinterpret_cast<const uint32_t*>(&h2), *reinterpret_cast<const uint32_t*>(&h3));
}

int launch_grads_to_bf16(const float* src, void* dst_k, void* dst_v, size_t n, bool after_sweep, cudaStream_t st) {
  const size_t n8 = n / 8;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((2 * n8 + 255) / 256));
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = after_sweep ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, k_grads_to_bf16, (const float4*)src, (uint4*)dst_k, (uint4*)dst_v, n8);
  count_launch(HGA_KERNELS_AUX);
  return record_cuda(e);
}

int launch_attn_fwd_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                            const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                            int32_t* status_word, cudaStream_t st) {
  const int items = dm.B * dm.Hkv * dm.NQB;
  const size_t smem = token_smem_bytes(dm);
  if (smem > 200 * 1024) return HGA_ERR_UNSUPPORTED;
  cudaError_t e;
  if (dm.d == 128) {
    e = cudaFuncSetAttribute(k_attn_fwd_generic<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return record_cuda(e);
    k_attn_fwd_generic<128><<<items, kAttnThreads, smem, st>>>(
        (const uint16_t*)Q, (const uint16_t*)K, (const uint16_t*)V, group_idx, n_groups, dm,
        (uint16_t*)O, LSE, status_word);
  } else {
    e = cudaFuncSetAttribute(k_attn_fwd_generic<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return record_cuda(e);
    k_attn_fwd_generic<64><<<items, kAttnThreads, smem, st>>>(
        (const uint16_t*)Q, (const uint16_t*)K, (const uint16_t*)V, group_idx, n_groups, dm,
        (uint16_t*)O, LSE, status_word);
  }
  count_launch(HGA_KERNELS_FWD_GENERIC);
  return record_cuda(cudaGetLastError());
}

template <int D>
static int bwd_generic(const Dims& dm, const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                       const uint16_t* O, const float* LSE, const uint16_t* dO,
                       const int32_t* group_idx, const int32_t* n_groups, uint16_t* dQ, float* dK,
                       float* dV, float* delta, int32_t* status_word, cudaStream_t st) {
  const int items = dm.B * dm.Hkv * dm.NQB;
  const size_t smem = token_smem_bytes(dm);
  if (smem > 200 * 1024) return HGA_ERR_UNSUPPORTED;
  cudaError_t e = cudaFuncSetAttribute(k_bwd_dq_generic<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_bwd_dkv_generic<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return record_cuda(e);
  const int64_t n_rows = (int64_t)dm.B * dm.Hq * dm.S;
  k_bwd_delta<D><<<(unsigned)((n_rows + kAttnWarps - 1) / kAttnWarps), kAttnThreads, 0, st>>>(O, dO, dm, delta);
  count_launch(HGA_KERNELS_BWD_GENERIC);
  int rc = record_cuda(cudaGetLastError());
  if (rc) return rc;
  k_bwd_dq_generic<D><<<items, kAttnThreads, smem, st>>>(Q, K, V, dO, LSE, delta, group_idx, n_groups, dm, dQ, status_word);
  count_launch(HGA_KERNELS_BWD_GENERIC);
  rc = record_cuda(cudaGetLastError());
  if (rc) return rc;
  k_bwd_dkv_generic<D><<<items, kAttnThreads, smem, st>>>(Q, K, V, dO, LSE, delta, group_idx, n_groups, dm, dK, dV);
  count_launch(HGA_KERNELS_BWD_GENERIC);
  return record_cuda(cudaGetLastError());
}

int launch_attn_bwd_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                            const void* O, const float* LSE, const void* dO,
                            const int32_t* group_idx, const int32_t* n_groups, void* dQ, float* dK,
                            float* dV, float* delta_ws, int32_t* status_word, cudaStream_t st) {
  if (dm.d == 128)
    return bwd_generic<128>(dm, (const uint16_t*)Q, (const uint16_t*)K, (const uint16_t*)V,
                            (const uint16_t*)O, LSE, (const uint16_t*)dO, group_idx, n_groups,
                            (uint16_t*)dQ, dK, dV, delta_ws, status_word, st);
  return bwd_generic<64>(dm, (const uint16_t*)Q, (const uint16_t*)K, (const uint16_t*)V,
                         (const uint16_t*)O, LSE, (const uint16_t*)dO, group_idx, n_groups,
                         (uint16_t*)dQ, dK, dV, delta_ws, status_word, st);
}

}  // namespace hga
