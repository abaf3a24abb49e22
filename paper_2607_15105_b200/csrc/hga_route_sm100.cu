// hga_route for sm_100a: chunk selection and group selection (Section 2.1 items 1-2) as one
// fused tcgen05 kernel per item (b, kv head, query block).
//
// Scores are the max (or mean / log-sum-exp, HGA_FLAG_SCORE_*) over the item's G*Bq query rows of q . summary.  The GEMM puts 128 summaries
// on the MMA M dimension (= TMEM lanes) and up to 256 query rows on N (= TMEM columns), so the
// maximum over rows is an in-thread reduction over the columns a thread reads back with
// tcgen05.ld: thread = summary.
//   phase 1  candidate chunk summaries, 128 per tile, streamed by TMA (octets of 8 rows)
//   select   k_c rounds of block arg-max on packed (orderable score, ~index) keys: highest score,
//            ties to the lowest index; the winners are then ordered ascending
//   phase 2  the opened chunks' group summaries (c/g = 8 or 16 consecutive rows per chunk, i.e.
//            one or two octets each) gathered by TMA, same GEMM, then top-kg_eff inside each chunk
// bf16 x bf16 products are exact in fp32; only the accumulation order differs from an exact sum.
#include <cfloat>

#include "hga_common.cuh"
#include "hga_sm100.cuh"

namespace hga {

using namespace sm100;

constexpr int kRtThreads = 320;     // warp 0 producer, warp 1 MMA, warps 2-5 readers, 6-9 help in select
// One summary-tile stage and one accumulator per CTA: an item has only a few tiles, so there is
// little to pipeline inside a CTA; the smaller footprint (under half of the shared memory and of
// TMEM) lets two CTAs share an SM, and the serial phases of one item overlap the GEMMs of another.
constexpr int kRtStages = 1;
constexpr int kRtAccs = 1;
constexpr int kRtTmemCols = 256 * kRtAccs;

template <int D>
struct RouteSmem {
  static constexpr int kTile = 128 * D * 2;
  alignas(1024) uint8_t a[kRtStages][kTile];   // summary tiles (A operand)
  uint64_t q_full, a_full[kRtStages], a_empty[kRtStages], acc_full[kRtAccs], acc_free[kRtAccs];
  uint32_t tmem_base;
  volatile int abort;
  int n_sel;
  unsigned long long warp_best[kRtThreads / 32];
  int sel[1024];          // selected chunk ids, first in selection order, then ascending
  int sorted[1024];
  // dynamic tail: Q rows (B operand, 1024-aligned), keys[n_cand_max] u64, gscore[kc*per] f32
};

__device__ __forceinline__ bool rt_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
  return mbar_wait_bounded(bar, parity, abort);
}

__device__ __forceinline__ uint32_t rt_orderable(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int D>
__global__ void __launch_bounds__(kRtThreads, 2)
k_route_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_cs,
              const __grid_constant__ CUtensorMap map_gs, Dims dm, int32_t* __restrict__ chunk_idx,
              int32_t* __restrict__ group_idx, int32_t* __restrict__ n_groups,
              float* __restrict__ chunk_scores, float* __restrict__ group_scores, int q_bytes,
              int max_cand) {
  constexpr int kOctBytes = 8 * D * 2;
  extern __shared__ uint8_t smem_raw[];
  RouteSmem<D>& sm = *reinterpret_cast<RouteSmem<D>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(&sm + 1) + 1023) & ~uintptr_t(1023));
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(q_smem + q_bytes);
  float* gscore = reinterpret_cast<float*>(keys + max_cand + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int item = blockIdx.x;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);
  const int j0 = w.se / dm.c, n_cand = (w.ls - w.se) / dm.c;
  // query rows on N: every head's Bq rows padded to whole octets, the total padded to a multiple of 32
  // (padding columns hold whatever shared memory held and are masked when the columns are reduced)
  const int bq_pad = bq_padded(dm), rows_pad = rows_padded(dm);
  const int n_cols = (rows_pad + 31) & ~31;
  const bool all_rows_real = n_cols == dm.rows;
  const int n_halves = n_cols > 256 ? n_cols / 256 : 1;
  const int rows_half = n_cols / n_halves;                   // N of one MMA: <= 256, multiple of 32
  const int k_sel = dm.kc < n_cand ? dm.kc : n_cand;
  const int opc = dm.per / 8;                                // octets per opened chunk
  const int n_ct = (n_cand + 127) / 128;                     // chunk tiles
  const int n_gt = (k_sel * dm.per + 127) / 128;             // group tiles
  volatile int* abort = &sm.abort;
  const int agg = score_agg_of(dm.flags);
  constexpr float kLog2e = 1.4426950408889634f;

  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kRtStages; ++s) { mbar_init(&sm.a_full[s], 1); mbar_init(&sm.a_empty[s], 1); }
    for (int s = 0; s < kRtAccs; ++s) { mbar_init(&sm.acc_full[s], 1); mbar_init(&sm.acc_free[s], 128); }
    sm.abort = 0;
    sm.n_sel = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, kRtTmemCols);
    tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&map_q); prefetch_tensormap(&map_cs); prefetch_tensormap(&map_gs);
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_base;

  // One GEMM phase: tiles [t_begin, t_begin + n_tiles) in the global tile numbering (which
  // drives barrier parities); `phase2` selects the octet source.
  auto run_phase = [&](int t_begin, int n_tiles, bool phase2) {
    if (warp == 0) {
      // ---------------------------------------------------------------- producer
      if (!phase2) {
        if (lane == 0) mbar_arrive_expect_tx(&sm.q_full, (uint32_t)(rows_pad / 8) * kOctBytes);
        __syncwarp();
        for (int o = lane; o < rows_pad / 8; o += 32) {
          const int r = 8 * o, a = r / bq_pad, t = r % bq_pad;    // rows past the segment arrive as zeros
          tma_load_5d(q_smem + o * kOctBytes, &map_q, &sm.q_full, 0, qb * dm.Bq + t, 0, h * dm.G + a, b);
        }
      }
      bool ok = true;
      for (int t = 0; t < n_tiles; ++t) {
        const int tg = t_begin + t, s = tg % kRtStages, use = tg / kRtStages;
        if (lane == 0 && use > 0) ok = rt_wait(&sm.a_empty[s], (use - 1) & 1, abort);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(&sm.a_full[s], RouteSmem<D>::kTile);
        __syncwarp();
        if (lane < 16) {
          int row;
          if (!phase2) {
            row = j0 + 128 * t + 8 * lane;                    // rows past the table read as zeros
            tma_load_5d(sm.a[s] + lane * kOctBytes, &map_cs, &sm.a_full[s], 0, row, 0, h, b);
          } else {
            const int oc = 16 * t + lane, r = oc / opc;
            row = r < k_sel ? sm.sorted[r] * dm.per + 8 * (oc % opc) : dm.Ng;
            tma_load_5d(sm.a[s] + lane * kOctBytes, &map_gs, &sm.a_full[s], 0, row, 0, h, b);
          }
        }
      }
    } else if (warp == 1) {
      // ---------------------------------------------------------------- MMA issuer
      if (lane == 0) {
        const uint32_t idesc = idesc_bf16_f32(128, rows_half, 0, 0);
        bool ok = phase2 ? true : rt_wait(&sm.q_full, 0, abort);
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int tg = t_begin + t, s = tg % kRtStages;
          ok = rt_wait(&sm.a_full[s], (tg / kRtStages) & 1, abort);
          for (int hf = 0; hf < n_halves && ok; ++hf) {
            const int step = tg * n_halves + hf, buf = step % kRtAccs, use = step / kRtAccs;
            if (use > 0) ok = rt_wait(&sm.acc_free[buf], (use - 1) & 1, abort);
            if (!ok) break;
            tc_fence_after_sync();
            const uint64_t ad = smem_desc_sw128(smem_u32(sm.a[s]), 16, kOctBytes);
            const uint64_t bd = smem_desc_sw128(
                smem_u32(q_smem) + (uint32_t)hf * (uint32_t)(rows_half / 8) * kOctBytes, 16, kOctBytes);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t off = (kk >> 2) * 1024 + (kk & 3) * 32;
              mma_ss(tmem + buf * 256, desc_advance(ad, off), desc_advance(bd, off), idesc, kk > 0);
            }
            mma_commit(&sm.acc_full[buf]);
          }
          if (ok) mma_commit(&sm.a_empty[s]);
        }
      }
    } else if (warp < 6) {
      // ---------------------------------------------------------------- readers: thread = summary
      const int quarter = warp & 3;
      const int row = quarter * 32 + lane;
      const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
      bool ok = true;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int tg = t_begin + t;
        float best = -FLT_MAX, sum = 0.f;    // log-sum-exp: (running maximum, sum of exp(dot - maximum))
        for (int hf = 0; hf < n_halves; ++hf) {
          const int step = tg * n_halves + hf, buf = step % kRtAccs;
          ok = __all_sync(0xffffffffu, rt_wait(&sm.acc_full[buf], (step / kRtAccs) & 1, abort));
          if (!ok) break;
          tc_fence_after_sync();
          for (int c = 0; c < rows_half; c += 32) {
            uint32_t x[32];
            tmem_ld32(lane_base + buf * 256 + c, x);
            tmem_wait_ld();
            if (!all_rows_real) {
              // padding columns become the neutral element of the reduction
              const float neutral = agg == 1 ? 0.f : -INFINITY;
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const int col = hf * rows_half + c + i;
                if (col >= rows_pad || col % bq_pad >= dm.Bq) x[i] = __float_as_uint(neutral);
              }
            }
            if (agg == 0) {
#pragma unroll
              for (int i = 0; i < 32; ++i) best = fmaxf(best, __uint_as_float(x[i]));
            } else if (agg == 1) {
#pragma unroll
              for (int i = 0; i < 32; ++i) sum += __uint_as_float(x[i]);
            } else {
              float cm = -FLT_MAX;
#pragma unroll
              for (int i = 0; i < 32; ++i) cm = fmaxf(cm, __uint_as_float(x[i]));
              if (cm > best) { sum *= exp2f((best - cm) * kLog2e); best = cm; }
#pragma unroll
              for (int i = 0; i < 32; ++i) sum += exp2f((__uint_as_float(x[i]) - best) * kLog2e);
            }
          }
          tc_fence_before_sync();
          mbar_arrive(&sm.acc_free[buf]);
        }
        if (!ok) break;
        if (agg == 1) best = sum * (1.f / (float)dm.rows);
        else if (agg == 2) best += logf(sum);
        const int i = 128 * t + row;
        if (!phase2) {
          if (i < n_cand) keys[i] = ((unsigned long long)rt_orderable(best) << 32) | (uint32_t)(0x7fffffff - (j0 + i));
          if (chunk_scores && i < n_cand) chunk_scores[(int64_t)item * dm.Nc + j0 + i] = best;
        } else {
          if (i < k_sel * dm.per) gscore[i] = best;
        }
      }
    }
  };

  // optional output: -inf outside the candidate range
  if (chunk_scores)
    for (int j = tid; j < dm.Nc; j += kRtThreads)
      if (j < j0 || j >= j0 + n_cand) chunk_scores[(int64_t)item * dm.Nc + j] = -INFINITY;
  if (group_scores)
    for (int i = tid; i < dm.kc * dm.per; i += kRtThreads)
      group_scores[(int64_t)item * dm.kc * dm.per + i] = -INFINITY;

  if (k_sel > 0) run_phase(0, n_ct, false);
  __syncwarp();          // the roles diverge inside a warp: reconverge before the block barrier
  __syncthreads();

  // ---------------------------------------------------------------------- chunk top-k
  if (!sm.abort) {
    if (n_cand <= 2 * kRtThreads) {
      // Few candidates: rank every key by counting the larger ones (keys are distinct, the index
      // is part of the key), no rounds and no block-wide arg-max.  A candidate is selected when
      // fewer than k_sel keys beat it; its place in the ascending output is the number of selected
      // candidates with a lower index.
      unsigned long long* flags = reinterpret_cast<unsigned long long*>(sm.sel);   // bit i: candidate i selected
      for (int i = tid; i < (n_cand + 63) / 64; i += kRtThreads) flags[i] = 0;
      __syncthreads();
      for (int i = tid; i < n_cand; i += kRtThreads) {
        const unsigned long long mine = keys[i];
        int beat = 0;
        for (int q = 0; q < n_cand; ++q) beat += keys[q] > mine;
        if (beat < k_sel) atomicOr(&flags[i >> 6], 1ull << (i & 63));
      }
      __syncthreads();
      for (int i = tid; i < n_cand; i += kRtThreads) {
        if ((flags[i >> 6] >> (i & 63)) & 1ull) {
          int pos = __popcll(flags[i >> 6] & ((1ull << (i & 63)) - 1));
          for (int q = 0; q < (i >> 6); ++q) pos += __popcll(flags[q]);
          sm.sorted[pos] = j0 + i;
        }
      }
      __syncthreads();
    } else {
      for (int r = 0; r < k_sel; ++r) {
        unsigned long long best = 0;
        for (int i = tid; i < n_cand; i += kRtThreads) best = keys[i] > best ? keys[i] : best;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
          best = other > best ? other : best;
        }
        if (lane == 0) sm.warp_best[warp] = best;
        __syncthreads();
        if (tid == 0) {
          for (int q = 1; q < kRtThreads / 32; ++q) best = sm.warp_best[q] > best ? sm.warp_best[q] : best;
          const int j = 0x7fffffff - (int)(uint32_t)(best & 0xffffffffu);
          sm.sel[r] = j;
          keys[j - j0] = 0;                                  // taken
        }
        __syncthreads();
      }
      // ascending order by counting ranks (indices are distinct)
      for (int i = tid; i < k_sel; i += kRtThreads) {
        const int v = sm.sel[i];
        int rank = 0;
        for (int q = 0; q < k_sel; ++q) rank += sm.sel[q] < v;
        sm.sorted[rank] = v;
      }
      __syncthreads();
    }
    for (int i = tid; i < dm.kc; i += kRtThreads)
      chunk_idx[(int64_t)item * dm.kc + i] = i < k_sel ? sm.sorted[i] : -1;
  }
  __syncthreads();

  // ---------------------------------------------------------------------- groups of the opened chunks
  if (k_sel > 0 && !sm.abort) run_phase(n_ct, n_gt, true);
  __syncwarp();
  __syncthreads();
  if (!sm.abort) {
    int32_t* gi = group_idx + (int64_t)item * dm.width;
    if (dm.flags & HGA_FLAG_GLOBAL_GROUP_BUDGET) {
      // One budget over all opened chunks: slot i (chunk-major, i.e. ascending group id) is selected
      // when fewer than k_sel * kg_eff slots beat it (higher score, or equal score and lower id); its
      // place in the ascending output is the number of selected slots below it.
      const int total = k_sel * dm.per, want = k_sel * dm.kge;
      unsigned long long* flags = reinterpret_cast<unsigned long long*>(sm.sel);   // 4096 bits
      for (int i = tid; i < (total + 63) / 64; i += kRtThreads) flags[i] = 0;
      __syncthreads();
      for (int i = tid; i < total; i += kRtThreads) {
        const float mine = gscore[i];
        int beat = 0;
        for (int q = 0; q < total; ++q) beat += gscore[q] > mine || (gscore[q] == mine && q < i);
        if (beat < want) atomicOr(&flags[i >> 6], 1ull << (i & 63));
        if (group_scores) group_scores[(int64_t)item * dm.kc * dm.per + i] = mine;
      }
      __syncthreads();
      for (int i = tid; i < total; i += kRtThreads)
        if ((flags[i >> 6] >> (i & 63)) & 1ull) {
          int pos = __popcll(flags[i >> 6] & ((1ull << (i & 63)) - 1));
          for (int q = 0; q < (i >> 6); ++q) pos += __popcll(flags[q]);
          gi[pos] = sm.sorted[i / dm.per] * dm.per + i % dm.per;
        }
    } else
    for (int r = tid; r < dm.kc; r += kRtThreads) {
      if (r < k_sel) {
        const float* v = gscore + r * dm.per;
        unsigned long long picked = 0;
        for (int q = 0; q < dm.kge; ++q) {
          int bu = -1;
          for (int u = 0; u < dm.per; ++u)
            if (!((picked >> u) & 1ull) && (bu < 0 || v[u] > v[bu])) bu = u;     // first wins ties
          picked |= 1ull << bu;
        }
        int n = r * dm.kge;
        for (int u = 0; u < dm.per; ++u)
          if ((picked >> u) & 1ull) gi[n++] = sm.sorted[r] * dm.per + u;
        if (group_scores)
          for (int u = 0; u < dm.per; ++u)
            group_scores[(int64_t)item * dm.kc * dm.per + r * dm.per + u] = v[u];
      }
    }
    for (int i = k_sel * dm.kge + tid; i < dm.width; i += kRtThreads) gi[i] = -1;
    if (tid == 0) n_groups[item] = k_sel * dm.kge;
  }

  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, kRtTmemCols);
  }
}

static size_t route_sm100_smem(const Dims& dm, int max_cand) {
  const size_t q_bytes = (size_t)((rows_padded(dm) + 31) & ~31) * dm.d * 2;
  const size_t base = dm.d == 128 ? sizeof(RouteSmem<128>) : sizeof(RouteSmem<64>);
  return base + 1024 + q_bytes + 1024 + sizeof(unsigned long long) * (max_cand + 2) +
         sizeof(float) * ((size_t)dm.kc * dm.per + 8);
}

static int route_max_cand(const Dims& dm) {
  const Window wl = window_of(dm, dm.NQB - 1);
  return (wl.ls - wl.se) / dm.c;
}

bool route_sm100_supported(const Dims& dm) {
  if (dm.flags & HGA_FLAG_GENERIC_KERNELS) return false;
  const int n_cols = (rows_padded(dm) + 31) & ~31;
  if (n_cols > 256 && (n_cols % 256 != 0 || n_cols != dm.rows)) return false;
  if (dm.per != 8 && dm.per != 16) return false;            // opened chunk = 1 or 2 octets of summaries
  if (dm.kc > 1024) return false;
  if ((dm.flags & HGA_FLAG_GLOBAL_GROUP_BUDGET) && dm.kc * dm.per > 4096) return false;   // bitmap in sel[]
  return route_sm100_smem(dm, route_max_cand(dm)) <= 227 * 1024;
}

template <int D>
static int launch_route(const Dims& dm, const void* Q, const void* chunk_sum, const void* group_sum,
                        int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, float* chunk_scores,
                        float* group_scores, cudaStream_t st) {
  CUtensorMap mq, mc, mg;
  const uint32_t box[5] = {64, 8, (uint32_t)(D / 64), 1, 1};
  const uint64_t dq[5] = {64, (uint64_t)dm.S, (uint64_t)(D / 64), (uint64_t)dm.Hq, (uint64_t)dm.B};
  const uint64_t dc[5] = {64, (uint64_t)dm.Nc, (uint64_t)(D / 64), (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t dg[5] = {64, (uint64_t)dm.Ng, (uint64_t)(D / 64), (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t sq[4] = {(uint64_t)dm.qs[2] * 2, 128, (uint64_t)dm.qs[1] * 2, (uint64_t)dm.qs[0] * 2};
  const uint64_t sc[4] = {(uint64_t)D * 2, 128, (uint64_t)dm.NcS * D * 2, (uint64_t)dm.Hkv * dm.NcS * D * 2};
  const uint64_t sg[4] = {(uint64_t)D * 2, 128, (uint64_t)dm.NgS * D * 2, (uint64_t)dm.Hkv * dm.NgS * D * 2};
  if (encode_tensor_map_bf16(&mq, Q, 5, dq, sq, box, true) ||
      encode_tensor_map_bf16(&mc, chunk_sum, 5, dc, sc, box, true) ||
      encode_tensor_map_bf16(&mg, group_sum, 5, dg, sg, box, true))
    return HGA_ERR_UNSUPPORTED;
  const int max_cand = route_max_cand(dm);
  const size_t smem = route_sm100_smem(dm, max_cand);
  cudaError_t e = cudaFuncSetAttribute(k_route_sm100<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return record_cuda(e);
  // two CTAs per SM need the largest shared-memory carve-out
  e = cudaFuncSetAttribute(k_route_sm100<D>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
  if (e != cudaSuccess) return record_cuda(e);
  const int items = dm.B * dm.Hkv * dm.NQB;
  k_route_sm100<D><<<items, kRtThreads, smem, st>>>(mq, mc, mg, dm, chunk_idx, group_idx, n_groups, chunk_scores,
                                                   group_scores, ((rows_padded(dm) + 31) & ~31) * D * 2, max_cand);
  count_launch();
  return record_cuda(cudaGetLastError());
}

int launch_route_sm100(const Dims& dm, const void* Q, const void* chunk_sum, const void* group_sum,
                       int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, float* chunk_scores,
                       float* group_scores, cudaStream_t st) {
  if (dm.d == 128)
    return launch_route<128>(dm, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, chunk_scores,
                             group_scores, st);
  return launch_route<64>(dm, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, chunk_scores,
                          group_scores, st);
}

}  // namespace hga
