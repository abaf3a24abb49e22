// hga_route, shape-generic CUDA-core version (Section 2.1, items 1-2).
//
// Three kernels per call:
//   k_chunk_scores   scores[item][j] = max (or mean, or log-sum-exp: HGA_FLAG_SCORE_*) over the item's
//                    G*Bq rows of q . chunk_sum[j]
//   k_select_chunks  top-k_c of the candidate scores, ties to the lowest index
//   k_route_groups   scores of the opened chunks' group summaries, top-kg_eff per chunk (or, with
//                    HGA_FLAG_GLOBAL_GROUP_BUDGET, the best chunks*kg_eff groups over all of them)
// bf16 x bf16 products are exact in fp32; only the fp32 accumulation order differs from
// an exact evaluation (about 1e-6 relative).
#include <cfloat>

#include "hga_common.cuh"

namespace hga {

constexpr int kScoreTile = 64;    // summaries scored per CTA pass
constexpr int kRowTile = 32;      // query rows staged in shared memory per pass
constexpr int kScoreThreads = 256;

__device__ inline float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ inline float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Scores kScoreTile summaries against all rows of an item.  sum_rows[i] is the row id of the
// i-th summary inside `summ` (negative = unused slot).  Result: out[i] (shared memory).
// Thread (jj = tid % 64, part = tid / 64) handles summary jj for rows part, part+4, ...
template <int D>
__device__ void score_tile(const Dims& dm, const uint16_t* __restrict__ Qitem,
                           const uint16_t* __restrict__ summ, const int* sum_rows,
                           float* s_sum /*[64][D+1]*/, float* s_q /*[kRowTile][D]*/,
                           float* s_red /*[4][64]*/, float* out /*[64]*/) {
  const int tid = threadIdx.x;
  // stage the summaries as fp32, padded rows (conflict-free column reads)
  for (int i = tid; i < kScoreTile * (D / 2); i += kScoreThreads) {
    const int r = i / (D / 2), e2 = i % (D / 2);
    const int row = sum_rows[r];
    uint32_t w = 0;
    if (row >= 0) w = *reinterpret_cast<const uint32_t*>(summ + (int64_t)row * D + 2 * e2);
    s_sum[r * (D + 1) + 2 * e2] = bf16_lo(w);
    s_sum[r * (D + 1) + 2 * e2 + 1] = bf16_hi(w);
  }
  const int jj = tid % kScoreTile, part = tid / kScoreTile;
  const int agg = score_agg_of(dm.flags);
  float best = -FLT_MAX, sum = 0.f;       // log-sum-exp keeps (running maximum, sum of exp(dot - maximum))
  for (int r0 = 0; r0 < dm.rows; r0 += kRowTile) {
    __syncthreads();
    for (int i = tid; i < kRowTile * (D / 2); i += kScoreThreads) {
      const int r = r0 + i / (D / 2), e2 = i % (D / 2);
      uint32_t w = 0;
      if (r < dm.rows) {
        const int a = r / dm.Bq, t = r % dm.Bq;
        w = *reinterpret_cast<const uint32_t*>(Qitem + a * dm.qs[1] + t * dm.qs[2] + 2 * e2);
      }
      s_q[(i / (D / 2)) * D + 2 * e2] = bf16_lo(w);
      s_q[(i / (D / 2)) * D + 2 * e2 + 1] = bf16_hi(w);
    }
    __syncthreads();
    const float* sv = s_sum + jj * (D + 1);
    for (int r = part; r < kRowTile && r0 + r < dm.rows; r += kScoreThreads / kScoreTile) {
      const float* qv = s_q + r * D;
      float acc = 0.f;
#pragma unroll 16
      for (int e = 0; e < D; ++e) acc = fmaf(qv[e], sv[e], acc);
      if (agg == 0) {
        best = fmaxf(best, acc);
      } else if (agg == 1) {
        sum += acc;
      } else {
        if (acc > best) { sum *= expf(best - acc); best = acc; }
        sum += expf(acc - best);
      }
    }
  }
  constexpr int kParts = kScoreThreads / kScoreTile;
  s_red[part * kScoreTile + jj] = agg == 1 ? sum : best;
  __syncthreads();
  float m = 0.f;
  if (tid < kScoreTile) {
    m = s_red[tid];
    for (int q = 1; q < kParts; ++q) m = agg == 1 ? m + s_red[q * kScoreTile + tid] : fmaxf(m, s_red[q * kScoreTile + tid]);
    if (agg == 1) m *= 1.f / (float)dm.rows;
    if (agg != 2) out[tid] = m;
  }
  if (agg == 2) {
    // second round: every part's sum rescaled to the common maximum
    const float mj = fmaxf(fmaxf(s_red[jj], s_red[kScoreTile + jj]), fmaxf(s_red[2 * kScoreTile + jj], s_red[3 * kScoreTile + jj]));
    static_assert(kParts == 4, "four row parts per summary");
    __syncthreads();
    s_red[part * kScoreTile + jj] = sum * expf(best - mj);
    __syncthreads();
    if (tid < kScoreTile) {
      float s = 0.f;
      for (int q = 0; q < kParts; ++q) s += s_red[q * kScoreTile + tid];
      out[tid] = m + logf(s);
    }
  }
  __syncthreads();
}

template <int D>
__global__ void __launch_bounds__(kScoreThreads)
k_chunk_scores(const uint16_t* __restrict__ Q, const uint16_t* __restrict__ chunk_sum, Dims dm,
               float* __restrict__ scores /*[items][Nc]*/) {
  extern __shared__ float smem[];
  float* s_sum = smem;
  float* s_q = s_sum + kScoreTile * (D + 1);
  float* s_red = s_q + kRowTile * D;
  float* s_out = s_red + kScoreThreads;
  int* s_rows = reinterpret_cast<int*>(s_out + kScoreTile);
  const int item = blockIdx.y;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);
  const int j0 = w.se / dm.c, n_cand = (w.ls - w.se) / dm.c;
  const int base = blockIdx.x * kScoreTile;
  if (base >= n_cand) return;
  const int bh = b * dm.Hkv + h;
  if (threadIdx.x < kScoreTile) {
    const int i = base + threadIdx.x;
    s_rows[threadIdx.x] = i < n_cand ? j0 + i : -1;
  }
  __syncthreads();
  const uint16_t* Qitem = Q + b * dm.qs[0] + (int64_t)(h * dm.G) * dm.qs[1] + (int64_t)(qb * dm.Bq) * dm.qs[2];
  score_tile<D>(dm, Qitem, chunk_sum + (int64_t)bh * dm.NcS * D, s_rows, s_sum, s_q, s_red, s_out);
  if (threadIdx.x < kScoreTile && base + threadIdx.x < n_cand)
    scores[(int64_t)item * dm.Nc + j0 + base + threadIdx.x] = s_out[threadIdx.x];
}

// Monotone map float -> uint32 (larger float => larger key).
__device__ inline uint32_t orderable(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// key = (score, lowest index wins): larger is better
__device__ inline unsigned long long pack_key(float score, int idx) {
  return ((unsigned long long)orderable(score) << 32) | (uint32_t)(0x7fffffff - idx);
}

__global__ void __launch_bounds__(256)
k_select_chunks(const float* __restrict__ scores, Dims dm, int32_t* __restrict__ chunk_idx,
                float* __restrict__ chunk_scores_out) {
  __shared__ unsigned long long s_warp[8];
  __shared__ int s_sel[1024];
  __shared__ int s_nsel;
  const int item = blockIdx.x;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);
  const int j0 = w.se / dm.c, n_cand = (w.ls - w.se) / dm.c;
  const float* sc = scores + (int64_t)item * dm.Nc;
  const int k = dm.kc < n_cand ? dm.kc : n_cand;
  const int tid = threadIdx.x;
  if (chunk_scores_out) {
    float* o = chunk_scores_out + (int64_t)item * dm.Nc;
    for (int j = tid; j < dm.Nc; j += blockDim.x)
      o[j] = (j >= j0 && j < j0 + n_cand) ? sc[j] : -INFINITY;
  }
  if (tid == 0) s_nsel = 0;
  __syncthreads();
  for (int r = 0; r < k; ++r) {
    unsigned long long best = 0;
    const int nsel = s_nsel;
    for (int i = tid; i < n_cand; i += blockDim.x) {
      const int j = j0 + i;
      bool taken = false;
      for (int q = 0; q < nsel; ++q) taken |= (s_sel[q] == j);
      if (!taken) {
        const unsigned long long key = pack_key(sc[j], j);
        best = key > best ? key : best;
      }
    }
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
      best = other > best ? other : best;
    }
    if ((tid & 31) == 0) s_warp[tid >> 5] = best;
    __syncthreads();
    if (tid == 0) {
      for (int q = 1; q < (int)(blockDim.x >> 5); ++q) best = s_warp[q] > best ? s_warp[q] : best;
      s_sel[s_nsel] = 0x7fffffff - (int)(uint32_t)(best & 0xffffffffu);
      s_nsel = s_nsel + 1;
    }
    __syncthreads();
  }
  if (tid == 0) {
    // ascending order (k is small)
    for (int i = 1; i < k; ++i) {
      const int v = s_sel[i];
      int q = i - 1;
      while (q >= 0 && s_sel[q] > v) { s_sel[q + 1] = s_sel[q]; --q; }
      s_sel[q + 1] = v;
    }
  }
  __syncthreads();
  for (int i = tid; i < dm.kc; i += blockDim.x) chunk_idx[(int64_t)item * dm.kc + i] = i < k ? s_sel[i] : -1;
}

template <int D>
__global__ void __launch_bounds__(kScoreThreads)
k_route_groups(const uint16_t* __restrict__ Q, const uint16_t* __restrict__ group_sum, Dims dm,
               const int32_t* __restrict__ chunk_idx, int32_t* __restrict__ group_idx,
               int32_t* __restrict__ n_groups, float* __restrict__ group_scores_out,
               float* __restrict__ gscratch /* [items][kc * per], global budget only */) {
  extern __shared__ float smem[];
  float* s_sum = smem;
  float* s_q = s_sum + kScoreTile * (D + 1);
  float* s_red = s_q + kRowTile * D;
  float* s_out = s_red + kScoreThreads;
  int* s_rows = reinterpret_cast<int*>(s_out + kScoreTile);
  __shared__ int s_count;
  __shared__ unsigned long long s_flags[64];          // global budget: bit i = slot i selected (<= 4096 slots)
  const bool global_budget = (dm.flags & HGA_FLAG_GLOBAL_GROUP_BUDGET) != 0;
  const int item = blockIdx.x;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const int bh = b * dm.Hkv + h;
  const int tid = threadIdx.x;
  const int32_t* ci = chunk_idx + (int64_t)item * dm.kc;
  int32_t* gi = group_idx + (int64_t)item * dm.width;
  const uint16_t* Qitem = Q + b * dm.qs[0] + (int64_t)(h * dm.G) * dm.qs[1] + (int64_t)(qb * dm.Bq) * dm.qs[2];
  int nsel = 0;
  while (nsel < dm.kc && ci[nsel] >= 0) ++nsel;
  const int total = nsel * dm.per;          // opened group summaries, chunk-major
  if (tid == 0) s_count = 0;
  for (int i = tid; i < dm.width; i += blockDim.x) gi[i] = -1;
  if (group_scores_out)
    for (int i = tid; i < dm.kc * dm.per; i += blockDim.x)
      group_scores_out[(int64_t)item * dm.kc * dm.per + i] = -INFINITY;
  __syncthreads();
  const int chunks_per_tile = kScoreTile / dm.per;   // per <= 64 by validation
  for (int base = 0; base < total; base += chunks_per_tile * dm.per) {
    if (tid < kScoreTile) {
      const int i = base + tid;
      s_rows[tid] = (tid < chunks_per_tile * dm.per && i < total)
                        ? ci[i / dm.per] * dm.per + (i % dm.per) : -1;
    }
    __syncthreads();
    score_tile<D>(dm, Qitem, group_sum + (int64_t)bh * dm.NgS * D, s_rows, s_sum, s_q, s_red, s_out);
    if (group_scores_out && tid < chunks_per_tile * dm.per && base + tid < total)
      group_scores_out[(int64_t)item * dm.kc * dm.per + base + tid] = s_out[tid];
    if (global_budget) {
      // keep the scores: the selection runs over all opened chunks at the end
      if (tid < chunks_per_tile * dm.per && base + tid < total)
        gscratch[(int64_t)item * dm.kc * dm.per + base + tid] = s_out[tid];
    } else if (tid == 0) {
      // one thread per opened chunk of this tile: top-kg_eff of its `per` groups.  Chunks are
      // handled in ascending order by thread 0 so the output list is ascending.
      int n = s_count;
      for (int cc = 0; cc < chunks_per_tile && base + cc * dm.per < total; ++cc) {
        const float* v = s_out + cc * dm.per;
        unsigned long long picked = 0;     // bit u set = group u selected (per <= 64)
        for (int r = 0; r < dm.kge; ++r) {
          int bu = -1;
          for (int u = 0; u < dm.per; ++u)
            if (!((picked >> u) & 1ull) && (bu < 0 || v[u] > v[bu])) bu = u;
          picked |= 1ull << bu;
        }
        const int m0 = ci[(base / dm.per) + cc] * dm.per;
        for (int u = 0; u < dm.per; ++u)
          if ((picked >> u) & 1ull) gi[n++] = m0 + u;
      }
      s_count = n;
    }
    __syncthreads();
  }
  if (global_budget) {
    // slot i (chunk-major = ascending group id) is selected when fewer than nsel * kg_eff slots beat
    // it (higher score, or equal score and lower id); its output place is the number of selected
    // slots below it
    const float* v = gscratch + (int64_t)item * dm.kc * dm.per;
    const int want = nsel * dm.kge;
    if (tid < 64) s_flags[tid] = 0;
    __syncthreads();                        // also orders the score writes above before the reads below
    for (int i = tid; i < total; i += blockDim.x) {
      const float mine = v[i];
      int beat = 0;
      for (int q = 0; q < total; ++q) beat += v[q] > mine || (v[q] == mine && q < i);
      if (beat < want) atomicOr(&s_flags[i >> 6], 1ull << (i & 63));
    }
    __syncthreads();
    for (int i = tid; i < total; i += blockDim.x)
      if ((s_flags[i >> 6] >> (i & 63)) & 1ull) {
        int pos = __popcll(s_flags[i >> 6] & ((1ull << (i & 63)) - 1));
        for (int q = 0; q < (i >> 6); ++q) pos += __popcll(s_flags[q]);
        gi[pos] = ci[i / dm.per] * dm.per + i % dm.per;
      }
    if (tid == 0) n_groups[item] = want;
    return;
  }
  if (tid == 0) n_groups[item] = s_count;
}

static size_t score_smem_bytes(int D) {
  return sizeof(float) * (kScoreTile * (D + 1) + kRowTile * D + kScoreThreads + kScoreTile) +
         sizeof(int) * kScoreTile;
}

int launch_route_generic(const Dims& dm, const void* Q, const void* chunk_sum,
                         const void* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                         int32_t* n_groups, float* chunk_scores, float* group_scores,
                         void* workspace, cudaStream_t st) {
  const int items = dm.B * dm.Hkv * dm.NQB;
  float* scores = (float*)workspace;
  float* gscratch = scores + (size_t)items * dm.Nc;      // behind the chunk scores (global group budget only)
  auto Qp = (const uint16_t*)Q;
  auto cs = (const uint16_t*)chunk_sum;
  auto gs = (const uint16_t*)group_sum;
  const size_t smem = score_smem_bytes(dm.d);
  // the widest candidate range is the last query block's
  const Window wl = window_of(dm, dm.NQB - 1);
  const int max_cand = (wl.ls - wl.se) / dm.c;
  cudaError_t e;
  if (dm.d == 128) {
    e = cudaFuncSetAttribute(k_chunk_scores<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_route_groups<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  } else {
    e = cudaFuncSetAttribute(k_chunk_scores<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_route_groups<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  }
  if (e != cudaSuccess) return record_cuda(e);
  if (max_cand > 0 && dm.kc > 0) {
    dim3 grid((max_cand + kScoreTile - 1) / kScoreTile, items);
    if (dm.d == 128)
      k_chunk_scores<128><<<grid, kScoreThreads, smem, st>>>(Qp, cs, dm, scores);
    else
      k_chunk_scores<64><<<grid, kScoreThreads, smem, st>>>(Qp, cs, dm, scores);
    count_launch(HGA_KERNELS_ROUTE_GENERIC);
    int rc = record_cuda(cudaGetLastError());
    if (rc) return rc;
  } else if (chunk_scores) {
    // nothing to score: the optional output is still defined (-inf everywhere) by k_select_chunks
  }
  k_select_chunks<<<items, 256, 0, st>>>(scores, dm, chunk_idx, chunk_scores);
  count_launch(HGA_KERNELS_ROUTE_GENERIC);
  int rc = record_cuda(cudaGetLastError());
  if (rc) return rc;
  if (dm.d == 128)
    k_route_groups<128><<<items, kScoreThreads, smem, st>>>(Qp, gs, dm, chunk_idx, group_idx, n_groups, group_scores, gscratch);
  else
    k_route_groups<64><<<items, kScoreThreads, smem, st>>>(Qp, gs, dm, chunk_idx, group_idx, n_groups, group_scores, gscratch);
  count_launch(HGA_KERNELS_ROUTE_GENERIC);
  return record_cuda(cudaGetLastError());
}

}  // namespace hga
