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
// Training shapes (up to 256 query rows on N): one summary-tile stage and one accumulator per CTA.  An
// item has only a few tiles, so there is little to pipeline inside a CTA; the smaller footprint (under
// half of the shared memory and of TMEM) lets two CTAs share an SM, and the serial phases of one item
// overlap the GEMMs of another.  Generation shapes (at most 128 padded query rows) leave room for a
// two-stage ring and two 128-column accumulators in the same footprint, so the summary tiles of an
// item stream from HBM back to back.
constexpr int kRtTmemCols = 256;

template <int D, int STAGES, int ACCS>
struct RouteSmem {
  static constexpr int kTile = 128 * D * 2;
  alignas(1024) uint8_t a[STAGES][kTile];   // summary tiles (A operand)
  uint64_t q_full, a_full[STAGES], a_empty[STAGES], acc_full[ACCS], acc_free[ACCS];
  uint64_t drain;              // give-up path only: completes when the tensor pipe has run dry
  uint32_t tmem_base;
  volatile int abort;
  int n_sel;
  unsigned long long warp_best[kRtThreads / 32];
  alignas(16) int sel[1024];   // selection bitmaps and 32-bit scores, or chunk ids in selection order
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

template <int D, int STAGES, int ACCS>
__global__ void __launch_bounds__(kRtThreads, 2)
k_route_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_ct,
              const __grid_constant__ CUtensorMap map_gs, Dims dm, int32_t* __restrict__ chunk_idx,
              int32_t* __restrict__ group_idx, int32_t* __restrict__ n_groups,
              float* __restrict__ chunk_scores, float* __restrict__ group_scores, int q_bytes,
              int max_cand) {
  constexpr int kOctBytes = 8 * D * 2;
  extern __shared__ uint8_t smem_raw[];
  using Smem = RouteSmem<D, STAGES, ACCS>;
  constexpr uint32_t kAccCols = kRtTmemCols / ACCS;   // TMEM columns per accumulator
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(&sm + 1) + 1023) & ~uintptr_t(1023));
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(q_smem + q_bytes);
  float* gscore = reinterpret_cast<float*>(keys + max_cand + 2);
  uint32_t* okeys = reinterpret_cast<uint32_t*>(sm.sel) + 64;   // orderable scores alone, when candidates <= 640

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
  uint32_t col_mask = 0;                                       // bit i: column i of a block of 32 is a real query row
  for (int i = 0; i < 32; ++i) col_mask |= (uint32_t)((i % bq_pad) < dm.Bq) << i;

  // Copies one 128-row summary tile into its ring stage; all lanes of warp 0.  The candidate chunks are
  // consecutive rows of the summary table, so a tile of them is 64-row x one-panel boxes (8 KB each: two or four
  // per tile, laid out [panel][128 rows][128 B]); the opened chunks' group summaries are gathered octet by octet
  // (16 boxes, [octet][panel][8 rows][128 B]).  A box costs the issuing warp on the order of a hundred cycles.
  int tiles_issued = 0;                 // warp 0's count of summary tiles whose copies were started
  auto issue_tile = [&](int tg, int t, bool phase2) {
    const int s = tg % STAGES;
    tiles_issued = tg + 1;
    if (lane == 0) mbar_arrive_expect_tx(&sm.a_full[s], Smem::kTile);
    __syncwarp();
    if (!phase2) {
      if (lane < 2 * (D / 64)) {
        const int half = lane & 1, panel = lane >> 1;
        const int row = j0 + 128 * t + 64 * half;             // rows past the table read as zeros
        tma_load_5d(sm.a[s] + panel * 16384 + half * 8192, &map_ct, &sm.a_full[s], 0, row, panel, h, b);
      }
    } else if (lane < 16) {
      const int oc = 16 * t + lane, r = oc / opc;
      const int row = r < k_sel ? sm.sorted[r] * dm.per + 8 * (oc % opc) : dm.Ng;
      tma_load_5d(sm.a[s] + lane * kOctBytes, &map_gs, &sm.a_full[s], 0, row, 0, h, b);
    }
  };
  const int n_pre = k_sel > 0 ? (n_ct < STAGES ? n_ct : STAGES) : 0;   // chunk tiles copied ahead of the CTA barrier

  if (warp == 0) {
    if (lane == 0) {
      mbar_init(&sm.q_full, 1);
      for (int s = 0; s < STAGES; ++s) { mbar_init(&sm.a_full[s], 1); mbar_init(&sm.a_empty[s], 1); }
      for (int s = 0; s < ACCS; ++s) { mbar_init(&sm.acc_full[s], 1); mbar_init(&sm.acc_free[s], 128); }
      mbar_init(&sm.drain, 1);
      sm.abort = 0;
      sm.n_sel = 0;
      fence_barrier_init();
      prefetch_tensormap(&map_q); prefetch_tensormap(&map_ct); prefetch_tensormap(&map_gs);
    }
    __syncwarp();
    // the first chunk tiles depend on nothing: their copies start before the CTA meets
    for (int t = 0; t < n_pre; ++t) issue_tile(t, t, false);
    if (lane == 0 && k_sel > 0) mbar_arrive_expect_tx(&sm.q_full, (uint32_t)(rows_pad / 8) * kOctBytes);
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, kRtTmemCols);
    tmem_relinquish();
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_base;

  // One GEMM phase: tiles [t_begin, t_begin + n_tiles) in the global tile numbering (which
  // drives barrier parities); `phase2` selects the octet source.
  auto run_phase = [&](int t_begin, int n_tiles, bool phase2) {
    if (!phase2 && warp >= 2 && lane < 4) {
      // The item's query rows, one octet box per lane.  Issuing a box costs its warp a few hundred
      // cycles and warps issue in parallel, so the boxes are spread over the eight non-producer warps.
      for (int o = (warp - 2) * 4 + lane; o < rows_pad / 8; o += 32) {
        const int r = 8 * o, a = r / bq_pad, t = r % bq_pad;    // rows past the segment arrive as zeros
        tma_load_5d(q_smem + o * kOctBytes, &map_q, &sm.q_full, 0, qb * dm.Bq + t, 0, h * dm.G + a, b);
      }
    }
    if (phase2 && warp >= 2 && lane < 2) {
      // First tile of the opened chunks' group summaries, again spread over the eight warps (two
      // octet boxes each).  Its ring stage is known to be free: every tile of the first phase has been
      // read back, so no barrier needs to be observed; warp 0 announces the bytes.
      const int s = t_begin % STAGES;
      const int oc = (warp - 2) * 2 + lane, r = oc / opc;
      const int row = r < k_sel ? sm.sorted[r] * dm.per + 8 * (oc % opc) : dm.Ng;
      tma_load_5d(sm.a[s] + oc * kOctBytes, &map_gs, &sm.a_full[s], 0, row, 0, h, b);
    }
    __syncwarp();
    if (warp == 0) {
      // ---------------------------------------------------------------- producer
      bool ok = true;
      if (phase2) {
        tiles_issued = t_begin + 1;        // (its boxes come from the other warps, see above)
        if (lane == 0) mbar_arrive_expect_tx(&sm.a_full[t_begin % STAGES], Smem::kTile);
      }
      for (int t = phase2 ? 1 : n_pre; t < n_tiles; ++t) {
        const int tg = t_begin + t, s = tg % STAGES, use = tg / STAGES;
        if (lane == 0 && use > 0) ok = rt_wait(&sm.a_empty[s], (use - 1) & 1, abort);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        issue_tile(tg, t, phase2);
      }
    } else if (warp == 1) {
      // ---------------------------------------------------------------- MMA issuer
      // The whole warp runs this branch converged (waits included) and one elected lane issues: see mma_ss_w.
      {
        auto mma_wait = [&](uint64_t* bar, uint32_t parity, volatile int* ab) {
          return __all_sync(0xffffffffu, rt_wait(bar, parity, ab));
        };
        const uint32_t idesc = idesc_bf16_f32(128, rows_half, 0, 0);
        bool ok = phase2 ? true : mma_wait(&sm.q_full, 0, abort);
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int tg = t_begin + t, s = tg % STAGES;
          ok = mma_wait(&sm.a_full[s], (tg / STAGES) & 1, abort);
          for (int hf = 0; hf < n_halves && ok; ++hf) {
            const int step = tg * n_halves + hf, buf = step % ACCS, use = step / ACCS;
            if (use > 0) ok = mma_wait(&sm.acc_free[buf], (use - 1) & 1, abort);
            if (!ok) break;
            tc_fence_after_sync();
            // A: the summary tile -- 8-row groups 1024 B apart and panels 16 KB apart for the chunk tiles,
            // octets (8 rows x all panels) for the gathered group tiles; B: the query rows, octets
            const uint64_t ad = smem_desc_sw128(smem_u32(sm.a[s]), 16, phase2 ? kOctBytes : 1024);
            const uint32_t a_panel = phase2 ? 1024u : 16384u;
            const uint64_t bd = smem_desc_sw128(
                smem_u32(q_smem) + (uint32_t)hf * (uint32_t)(rows_half / 8) * kOctBytes, 16, kOctBytes);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t a_off = (kk >> 2) * a_panel + (kk & 3) * 32, b_off = (kk >> 2) * 1024 + (kk & 3) * 32;
              mma_ss_w(tmem + buf * kAccCols, desc_advance(ad, a_off), desc_advance(bd, b_off), idesc, kk > 0);
            }
            mma_commit_w(&sm.acc_full[buf]);
          }
          if (ok) mma_commit_w(&sm.a_empty[s]);
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
          const int step = tg * n_halves + hf, buf = step % ACCS;
          ok = __all_sync(0xffffffffu, rt_wait(&sm.acc_full[buf], (step / ACCS) & 1, abort));
          if (!ok) break;
          tc_fence_after_sync();
          for (int c = 0; c < rows_half; c += 32) {
            uint32_t x[32];
            tmem_ld32(lane_base + buf * kAccCols + c, x);
            tmem_wait_ld();
            if (!all_rows_real) {
              // padding columns become the neutral element of the reduction (bq_pad divides 32, so the
              // pattern of real columns repeats in every block of 32; only the last block can be cut)
              const float neutral = agg == 1 ? 0.f : -INFINITY;
              const int left = rows_pad - (hf * rows_half + c);
              const uint32_t m = left >= 32 ? col_mask : (col_mask & ((1u << (left > 0 ? left : 0)) - 1u));
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (!((m >> i) & 1u)) x[i] = __float_as_uint(neutral);
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
          if (i < n_cand) {
            keys[i] = ((unsigned long long)rt_orderable(best) << 32) | (uint32_t)(0x7fffffff - (j0 + i));
            if (n_cand <= 2 * kRtThreads) okeys[i] = rt_orderable(best);
          }
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
      // The count runs on the 32-bit orderable scores alone (four per 16-byte load).  Equal scores
      // then share a rank; that only matters when a tie straddles the k-th place, which shows as a
      // selection of the wrong size and is redone on the full 64-bit keys (ties to the lowest index).
      uint32_t* flags = reinterpret_cast<uint32_t*>(sm.sel);      // bit i: candidate i selected (20 words at most)
      auto rank_select = [&](bool exact) {
        for (int base = 0; base < n_cand; base += kRtThreads) {   // warp-uniform trip count (ballots below)
          const int i = base + tid;
          bool sel = false;
          if (i < n_cand) {
            int beat = 0, q = 0;
            if (!exact) {
              const uint32_t mine = okeys[i];
              const uint4* k4 = reinterpret_cast<const uint4*>(okeys);
#pragma unroll 4
              for (; q + 4 <= n_cand; q += 4) {
                const uint4 kk = k4[q >> 2];
                beat += (int)(kk.x > mine) + (int)(kk.y > mine) + (int)(kk.z > mine) + (int)(kk.w > mine);
              }
              for (; q < n_cand; ++q) beat += okeys[q] > mine;
            } else {
              const unsigned long long mine = keys[i];
              const ulonglong2* k2 = reinterpret_cast<const ulonglong2*>(keys);
#pragma unroll 4
              for (; q + 2 <= n_cand; q += 2) {
                const ulonglong2 kk = k2[q >> 1];
                beat += (int)(kk.x > mine) + (int)(kk.y > mine);
              }
              if (q < n_cand) beat += keys[q] > mine;
            }
            sel = beat < k_sel;
          }
          const uint32_t word = __ballot_sync(0xffffffffu, sel);
          if (lane == 0 && base + warp * 32 < n_cand) flags[(base + warp * 32) >> 5] = word;
        }
      };
      rank_select(false);
      __syncthreads();
      int n_picked = 0;
      for (int q = 0; q < (n_cand + 31) / 32; ++q) n_picked += __popc(flags[q]);
      if (n_picked != k_sel) {          // same value in every thread
        __syncthreads();
        rank_select(true);
        __syncthreads();
      }
      for (int i = tid; i < n_cand; i += kRtThreads) {
        if ((flags[i >> 5] >> (i & 31)) & 1u) {
          int pos = __popc(flags[i >> 5] & ((1u << (i & 31)) - 1u));
          for (int q = 0; q < (i >> 5); ++q) pos += __popc(flags[q]);
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
    const bool global_budget = (dm.flags & HGA_FLAG_GLOBAL_GROUP_BUDGET) != 0;
    if (k_sel * dm.per <= 4096) {
      // One thread per slot (opened chunk, group), slots in chunk-major order = ascending group id.
      // A slot is selected when fewer than `want` slots of its scope beat it (higher score, or equal
      // score and lower id); the scope is its own chunk (want = kg_eff) or, with one budget over all
      // opened chunks, every slot (want = k_sel * kg_eff).  Its place in the ascending output is the
      // number of selected slots below it.
      const int total = k_sel * dm.per;
      uint32_t* flags = reinterpret_cast<uint32_t*>(sm.sel);      // 4096 bits
      const int want = global_budget ? k_sel * dm.kge : dm.kge;
      for (int base = 0; base < total; base += kRtThreads) {      // warp-uniform trip count (ballots below)
        const int i = base + tid;
        bool sel = false;
        if (i < total) {
          const float mine = gscore[i];
          const int lo = global_budget ? 0 : i - i % dm.per, hi = global_budget ? total : lo + dm.per;
          int beat = 0;
#pragma unroll 8
          for (int q = lo; q < hi; ++q) beat += gscore[q] > mine || (gscore[q] == mine && q < i);
          sel = beat < want;
          if (group_scores) group_scores[(int64_t)item * dm.kc * dm.per + i] = mine;
        }
        const uint32_t word = __ballot_sync(0xffffffffu, sel);
        if (lane == 0 && base + warp * 32 < total) flags[(base + warp * 32) >> 5] = word;
      }
      __syncthreads();
      for (int i = tid; i < total; i += kRtThreads)
        if ((flags[i >> 5] >> (i & 31)) & 1u) {
          int pos = __popc(flags[i >> 5] & ((1u << (i & 31)) - 1u));
          for (int q = 0; q < (i >> 5); ++q) pos += __popc(flags[q]);
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

  if (sm.abort) {
    // A bounded wait gave up: the item's routing is marked invalid (the attention calls report a negative
    // count and use no routed groups for that item), and the copies still in flight get a bounded time to land
    // before the CTA's shared memory is released.
    if (tid == 0) n_groups[item] = -1;
    if (warp == 0 && lane == 0) {        // (tiles_issued is warp 0's own count)
      if (k_sel > 0) mbar_wait(&sm.q_full, 0);
      for (int tg = tiles_issued > STAGES ? tiles_issued - STAGES : 0; tg < tiles_issued; ++tg)
        mbar_wait(&sm.a_full[tg % STAGES], (tg / STAGES) & 1);
    }
    if (warp == 1) {
      // GEMMs the warp's issuing lane started may still be writing tensor memory: a commit completes once
      // every earlier MMA of that lane has, so wait for one (bounded) before the columns are given back
      mma_commit_w(&sm.drain);
      mbar_wait(&sm.drain, 0);
    }
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, kRtTmemCols);
  }
}

// Generation shapes (few query rows) take the pipelined instantiation.
static bool route_pipelined(const Dims& dm) { return ((rows_padded(dm) + 31) & ~31) <= 128; }

static size_t route_sm100_smem(const Dims& dm, int max_cand) {
  const size_t q_bytes = (size_t)((rows_padded(dm) + 31) & ~31) * dm.d * 2;
  const size_t base = route_pipelined(dm) ? (dm.d == 128 ? sizeof(RouteSmem<128, 2, 2>) : sizeof(RouteSmem<64, 2, 2>))
                                          : (dm.d == 128 ? sizeof(RouteSmem<128, 1, 1>) : sizeof(RouteSmem<64, 1, 1>));
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
  if (n_cols != dm.rows && 32 % bq_padded(dm) != 0) return false;   // the padding mask repeats every 32 columns
  if (dm.per != 8 && dm.per != 16) return false;            // opened chunk = 1 or 2 octets of summaries
  if (dm.kc > 1024) return false;
  if ((dm.flags & HGA_FLAG_GLOBAL_GROUP_BUDGET) && dm.kc * dm.per > 4096) return false;   // bitmap in sel[]
  return route_sm100_smem(dm, route_max_cand(dm)) <= 227 * 1024;
}

template <int D, int STAGES, int ACCS>
static int launch_route(const Dims& dm, const void* Q, const void* chunk_sum, const void* group_sum,
                        int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, float* chunk_scores,
                        float* group_scores, cudaStream_t st) {
  CUtensorMap mq, mc, mg;
  const uint32_t box[5] = {64, 8, (uint32_t)(D / 64), 1, 1};
  const uint32_t box_ct[5] = {64, 64, 1, 1, 1};            // half a chunk tile, one panel
  const uint64_t dq[5] = {64, (uint64_t)dm.S, (uint64_t)(D / 64), (uint64_t)dm.Hq, (uint64_t)dm.B};
  const uint64_t dc[5] = {64, (uint64_t)dm.Nc, (uint64_t)(D / 64), (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t dg[5] = {64, (uint64_t)dm.Ng, (uint64_t)(D / 64), (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t sq[4] = {(uint64_t)dm.qs[2] * 2, 128, (uint64_t)dm.qs[1] * 2, (uint64_t)dm.qs[0] * 2};
  const uint64_t sc[4] = {(uint64_t)D * 2, 128, (uint64_t)dm.NcS * D * 2, (uint64_t)dm.Hkv * dm.NcS * D * 2};
  const uint64_t sg[4] = {(uint64_t)D * 2, 128, (uint64_t)dm.NgS * D * 2, (uint64_t)dm.Hkv * dm.NgS * D * 2};
  if (encode_tensor_map_bf16(&mq, Q, 5, dq, sq, box, true) ||
      encode_tensor_map_bf16(&mc, chunk_sum, 5, dc, sc, box_ct, true) ||
      encode_tensor_map_bf16(&mg, group_sum, 5, dg, sg, box, true))
    return HGA_ERR_UNSUPPORTED;
  const int max_cand = route_max_cand(dm);
  const size_t smem = route_sm100_smem(dm, max_cand);
  // two CTAs per SM need the largest shared-memory carve-out
  const int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(&k_route_sm100<D, STAGES, ACCS>), smem, true);
  if (rc) return rc;
  const int items = dm.B * dm.Hkv * dm.NQB;
  k_route_sm100<D, STAGES, ACCS><<<items, kRtThreads, smem, st>>>(mq, mc, mg, dm, chunk_idx, group_idx, n_groups, chunk_scores,
                                                   group_scores, ((rows_padded(dm) + 31) & ~31) * D * 2, max_cand);
  count_launch(HGA_KERNELS_ROUTE_TENSOR);
  return record_cuda(cudaGetLastError());
}

int launch_route_sm100(const Dims& dm, const void* Q, const void* chunk_sum, const void* group_sum,
                       int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, float* chunk_scores,
                       float* group_scores, cudaStream_t st) {
#define HGA_ROUTE_ARGS dm, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, chunk_scores, group_scores, st
  if (route_pipelined(dm))
    return dm.d == 128 ? launch_route<128, 2, 2>(HGA_ROUTE_ARGS) : launch_route<64, 2, 2>(HGA_ROUTE_ARGS);
  return dm.d == 128 ? launch_route<128, 1, 1>(HGA_ROUTE_ARGS) : launch_route<64, 1, 1>(HGA_ROUTE_ARGS);
#undef HGA_ROUTE_ARGS
}

}  // namespace hga
