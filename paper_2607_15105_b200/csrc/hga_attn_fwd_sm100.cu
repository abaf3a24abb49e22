// hga_attn_fwd for sm_100a: routed exact-token attention as a TMA-gather-fed tcgen05 / TMEM
// flash-style kernel (Section 2.1 item 3).
//
// Work unit (one CTA): one 128-row M-tile of one item (b, kv head, query block) swept over the
// item's routed key set.  A CTA takes half of an SM's resources (96 KB of shared memory, 256
// TMEM columns, 192 threads), so two CTAs -- usually the two M-tiles of one item, which then
// share their K/V gather through L2 -- run on an SM at once: one CTA's exp2 overlaps the other's
// GEMMs, and one CTA's set-up and epilogue overlap the other's main loop.
// Keys are addressed in "octets" (8 consecutive tokens = one 8-row 128-byte-swizzle atom per
// 64-element panel): sink, each selected group and the local window are runs of octets, and a
// 64-key tile is 8 octets fetched by 8 TMA boxes (one lane each) for K and 8 for V, on separate
// 2-stage rings.  Octets past the end of the list load an out-of-range row and arrive as zeros.
//
// Warp roles (256 threads; warps are allocated in fours, and two CTAs of 8 warps leave 128
// registers per thread):
//   warp 0      octet table, Q load, K tile ring (boxes 0-3 of a tile; warp 7: boxes 4-7)    warp 6   V tile ring
//   warp 1      MMA issuer (one thread): S = Q K^T (smem x smem), O += P V (P from TMEM)
//   warps 2-5   softmax, one thread per row (thread owns TMEM lane = row), then the epilogue
// K and V have independent producers: K(j+2) is wanted as soon as S(j) has been issued, V(j+1)
// only after PV(j-1), and neither may wait for the other.
// TMEM (256 columns): S[2] (64 columns each, double buffered) | O.  P (bf16) is written over the
// S buffer it came from.  Because S is double buffered, S of tile j+1 is computed while the rows
// of tile j are in their exp2.
// The running maximum is only raised when it grows by more than 2^8 (rescaling O is then done
// by the row's own thread, after the PV of the previous tile has completed), so rescales are rare.
#include "hga_common.cuh"
#include "hga_octets.cuh"
#include "hga_sm100.cuh"
#include "hga_trace.cuh"

namespace hga {

using namespace sm100;

constexpr int kFwdThreads = 256;
constexpr int kStages = 2;
constexpr int kFT = 64;                      // keys per tile
constexpr float kRescaleThreshold = 8.0f;   // log2 units: the reference is raised when the maximum outgrows it by this much

template <int D>
struct FwdSmem {
  static constexpr int kQBytes = 128 * D * 2;
  static constexpr int kTileBytes = kFT * D * 2;
  alignas(1024) uint8_t q[kQBytes];
  alignas(1024) uint8_t k[kStages][kTileBytes];
  alignas(1024) uint8_t v[kStages][kTileBytes];
  uint64_t q_full;
  uint64_t k_full[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[2], p_full[2], tail_done, o_done;
  uint32_t tmem_base;
  int n_oct;
  volatile int abort;
  int oct_row[1];   // really max_routed_tokens/8 entries (dynamic shared memory follows)
};

__device__ __forceinline__ bool wait_or_abort_(uint64_t* bar, uint32_t parity, volatile int* abort, int code) {
  return mbar_wait_bounded(bar, parity, abort, kWaitCycles, code);
}
#ifdef HGA_DEBUG_WAIT
#define wait_or_abort(bar, parity, abort) wait_or_abort_((bar), (parity), (abort), __LINE__)
#define HGA_FWD_ABORT_CODE(flag) (HGA_STATUS_WAIT_TIMEOUT | ((flag) << 8) | (1 << 28))
#else
#define wait_or_abort(bar, parity, abort) wait_or_abort_((bar), (parity), (abort), 1)
#define HGA_FWD_ABORT_CODE(flag) HGA_STATUS_WAIT_TIMEOUT
#endif

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 2)
k_attn_fwd_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ group_idx,
                 const int32_t* __restrict__ n_groups, Dims dm, uint16_t* __restrict__ O,
                 float* __restrict__ LSE, int32_t* status_word) {
  constexpr int kOctBytes = 8 * D * 2;            // one octet of rows, all panels
  constexpr int kQBytes = 128 * D * 2;
  constexpr int kTileBytes = kFT * D * 2;
  constexpr uint32_t kSbo = kOctBytes;            // byte distance between 8-row groups
  constexpr uint32_t kColO = 128;                 // TMEM: S[buf] at buf*64, O at 128
  constexpr uint32_t kTmemCols = 256;
  extern __shared__ uint8_t smem_raw[];
  FwdSmem<D>& sm = *reinterpret_cast<FwdSmem<D>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  HGA_TRACE_DECL;
  // rows of the item: every head's Bq rows padded to whole octets (padding rows compute garbage
  // in their own TMEM lanes and are never stored)
  const int bq_pad = bq_padded(dm), rows_pad = rows_padded(dm);
  const int n_mt_item = (rows_pad + 127) / 128;
  // Launch order: late query blocks first -- where the history is short they see the most keys, so the
  // cheapest CTAs are the ones that fill the last wave.
  const int unit = blockIdx.x / n_mt_item, n_bh = dm.B * dm.Hkv;
  const int item = (unit % n_bh) * dm.NQB + (dm.NQB - 1 - unit / n_bh);
  const int mt0 = blockIdx.x % n_mt_item;               // this CTA's M-tile inside the item
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);

  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], 1);
      mbar_init(&sm.v_full[s], 1); mbar_init(&sm.v_empty[s], 1);
    }
    for (int u = 0; u < 2; ++u) { mbar_init(&sm.s_full[u], 1); mbar_init(&sm.p_full[u], 128); }
    mbar_init(&sm.tail_done, 1);
    mbar_init(&sm.o_done, 1);
    sm.abort = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  if (warp == 0) {
    // Q does not depend on the routing: start its copy first (tid 0 initialised the barriers above)
    if (lane == 0) {
      prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
    }
    const int q_oct = min(16, rows_pad / 8 - 16 * mt0);   // octets of real rows in this M-tile
    if (lane == 0) mbar_arrive_expect_tx(&sm.q_full, (uint32_t)q_oct * kOctBytes);
    __syncwarp();
    if (lane < q_oct) {
      const int r = mt0 * 128 + 8 * lane;              // first row of the octet inside the item
      const int a = r / bq_pad, t = r % bq_pad;        // token rows past the segment arrive as zeros
      tma_load_5d(sm.q + lane * kOctBytes, &map_q, &sm.q_full, 0, qb * dm.Bq + t, 0, h * dm.G + a, b);
    }
    bool bad;
    const int n = build_octet_table(dm, w, group_idx + (int64_t)item * dm.width, n_groups + item, sm.oct_row, &bad);
    if (lane == 0) {
      sm.n_oct = n;
      if (bad && status_word) atomicOr(status_word, HGA_STATUS_BAD_INDEX);
    }
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tmem = sm.tmem_base;
  const int n_oct = sm.n_oct;
  // exact key count: only the last octet of the local window can be partial
  const int n_keys = n_oct * 8 - ((8 - ((w.p0 + dm.Bq - w.ls) & 7)) & 7);
  const int n_tiles = (n_oct + 7) / 8;
  volatile int* abort = &sm.abort;
  HGA_TRACE_POINT(1);

  if (warp == 0 || warp == 6 || warp == 7) {
    // ------------------------------------------------------------------ producers: warps 0 and 7 K, warp 6 V
    // K boxes are split between warps 0 and 7 (a box costs its issuing warp a few hundred cycles)
    const bool is_k = warp != 6;
    const int first = warp == 7 ? 4 : 0, count = is_k ? 4 : 8;   // this warp's octets of a tile
    uint64_t* full = is_k ? sm.k_full : sm.v_full;
    // a K stage is free as soon as S of its tile is complete: that is s_full of the same index (the K
    // ring and the S buffers both have two slots), which saves the MMA thread one commit per tile
    static_assert(kStages == 2, "K ring and S buffers are indexed alike");
    uint64_t* empty = is_k ? sm.s_full : sm.v_empty;
    uint8_t* ring = is_k ? sm.k[0] : sm.v[0];
    const CUtensorMap* map = is_k ? &map_k : &map_v;
    bool ok = true;
    int issued = 0;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const int s = j % kStages, use = j / kStages;
      if (lane == 0 && use > 0) ok = wait_or_abort(&empty[s], (use - 1) & 1, abort);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0 && warp != 7) mbar_arrive_expect_tx(&full[s], kTileBytes);
      __syncwarp();
      if (lane < count) {
        const int o = 8 * j + first + lane;
        const int row = o < n_oct ? sm.oct_row[o] : dm.L;   // past the list: out of range -> zeros
        tma_load_5d(ring + s * kTileBytes + (first + lane) * kOctBytes, map, &full[s], 0, row, 0, h, b);
      }
      issued = j + 1;
      HGA_TRACE_POINT(2);
    }
    if (*abort && lane == 0 && warp != 7) {
      // giving up: let the copies still in flight land before shared memory is released
      if (is_k) mbar_wait(&sm.q_full, 0);
      for (int j = issued > kStages ? issued - kStages : 0; j < issued; ++j)
        mbar_wait(&full[j % kStages], (j / kStages) & 1);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs this branch converged (waits included) and one elected lane issues: see mma_ss_w.
    {
      auto mma_wait = [&](uint64_t* bar, uint32_t parity, volatile int* ab) {
        return __all_sync(0xffffffffu, wait_or_abort(bar, parity, ab));
      };
      constexpr uint32_t idesc_s = idesc_bf16_f32(128, kFT, 0, 0);
      constexpr uint32_t idesc_o = idesc_bf16_f32(128, D, 0, 1);
      // Descriptors are built once; inside the loops an MMA costs two integer adds (the lone
      // issuing thread is latency-bound, and a K=16 step is only 64 tensor-pipe cycles).
      const uint64_t q_desc = smem_desc_sw128(smem_u32(sm.q), 16, kSbo);
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, kSbo);       // K-major B of S = Q K^T
      const uint64_t v_desc0 = smem_desc_sw128(smem_u32(sm.v[0]), 1024, kSbo);     // MN-major B of O += P V
      const uint32_t o_acc = tmem + kColO;
      // S(j) into buffer j&1; the K stage is released behind it
      auto issue_s = [&](int j) {
        const uint64_t kd = desc_advance(k_desc0, (uint32_t)(j % kStages) * kTileBytes);
        const uint32_t d_addr = tmem + (j & 1) * 64;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * 1024 + (kk & 3) * 32;   // panel, then 32-byte K step
          mma_ss_w(d_addr, desc_advance(q_desc, off), desc_advance(kd, off), idesc_s, kk > 0);
        }
        mma_commit_w(&sm.s_full[j & 1]);           // also releases the K stage (see the K producer)
      };
      bool ok = mma_wait(&sm.q_full, 0, abort);
      for (int j = 0; j < 2 && j < n_tiles && ok; ++j) {      // prologue: S two tiles ahead
        ok = mma_wait(&sm.k_full[j % kStages], (j / kStages) & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        issue_s(j);
      }
      HGA_TRACE_POINT(3);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int sv = j % kStages;
        const bool more = j + 2 < n_tiles;
        ok = mma_wait(&sm.v_full[sv], (j / kStages) & 1, abort);
        HGA_TRACE_POINT(6);
        if (ok) ok = mma_wait(&sm.p_full[j & 1], (j >> 1) & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        HGA_TRACE_POINT(5);
        const uint64_t vd = desc_advance(v_desc0, (uint32_t)sv * kTileBytes);
        const uint32_t p_addr = tmem + (j & 1) * 64;
#pragma unroll
        for (int kk = 0; kk < kFT / 16; ++kk)     // 16 keys per step: 2 octets in smem, 8 TMEM columns of P
          mma_ts_w(o_acc, p_addr + kk * 8, desc_advance(vd, kk * 2 * kOctBytes), idesc_o, (j > 0 || kk > 0));
        mma_commit_w(&sm.v_empty[sv]);
        if (j + 2 == n_tiles) mma_commit_w(&sm.tail_done);   // PV of the last-but-one tile (see rescale)
        if (j + 1 == n_tiles) mma_commit_w(&sm.o_done);
        HGA_TRACE_POINT(7);
        if (more) {                                // S(j+2) reuses the buffer P(j) sat in: ordered after PV(j)
          ok = mma_wait(&sm.k_full[(j + 2) % kStages], ((j + 2) / kStages) & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
          issue_s(j + 2);
        }
        HGA_TRACE_POINT(8);
      }
    }
  } else if (warp >= 2 && warp < 6) {
    // ------------------------------------------------------------------ softmax + epilogue
    {
      const int quarter = warp & 3;                       // TMEM lanes this warp may touch
      const int row_in_tile = quarter * 32 + lane;
      const int r = mt0 * 128 + row_in_tile;              // row inside the item
      const int a = r / bq_pad, t = r % bq_pad;
      const bool real_row = r < rows_pad && t < dm.Bq;
      // a warp whose 32 lanes are all padding (generation shapes) only keeps the barriers moving
      const bool warp_real = __any_sync(0xffffffffu, real_row);
      const int limit = n_keys - dm.Bq + t + 1;           // visible key slots (causal inside the block)
      const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
      const uint32_t o_addr = lane_base + kColO;
      const float sl2 = dm.scale * 1.4426950408889634f;   // softmax scale in log2 units
      // m_used: the reference the exponentials of a row are taken against (log2 units).  Only the FIRST tile
      // is read twice (true maximum, then exponentials).  Later tiles are read once: p = 2^(x - m_used) with
      // the reference as it stands, the tile's own maximum being found in the same pass.  A tile whose maximum
      // outgrows the reference by more than the threshold (rare after the first tiles) raises the reference to
      // that maximum (O, l rescaled) and takes its exponentials again -- S is still intact then, because P is
      // only written once the tile is known to be in range.  The result is the one a maximum pass per tile
      // would give: the reference is raised at the same tiles to the same values.
      float m_used = -INFINITY, l = 0.f, l_mma = 0.f;
      const uint64_t sl2_2 = pack_f32x2(sl2, sl2);
      bool ok = true;
      // O *= corr (per row); O must hold exactly the sum up to tile j-1, i.e. PV(j-1) must have completed.
      // The issuer queues S(j+1) directly behind PV(j-1), so that S being ready proves it; the last tile
      // has no S(j+1) and uses a barrier committed behind PV(n-2) instead.
      auto rescale_o = [&](int j, float corr) {
        bool fine;
        if (j + 1 < n_tiles)
          fine = __all_sync(0xffffffffu, wait_or_abort(&sm.s_full[(j + 1) & 1], ((j + 1) >> 1) & 1, abort));
        else
          fine = __all_sync(0xffffffffu, wait_or_abort(&sm.tail_done, 0, abort));
        if (!fine) return false;
        tc_fence_after_sync();
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t y[32];
          tmem_ld32(o_addr + c * 32, y);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) y[i] = __float_as_uint(__uint_as_float(y[i]) * corr);
          tmem_st32(o_addr + c * 32, y);
        }
        return true;
      };
      for (int j = 0; j < n_tiles; ++j) {
        const uint32_t s_addr = lane_base + (j & 1) * 64;
        ok = __all_sync(0xffffffffu, wait_or_abort(&sm.s_full[j & 1], (j >> 1) & 1, abort));
        if (!ok) break;                                   // warp-uniform
        if (!warp_real) {
          // S(j) complete implies that the previous use of this P barrier is over: arriving now is safe
          mbar_arrive(&sm.p_full[j & 1]);
          continue;
        }
        tc_fence_after_sync();
        HGA_TRACE_POINT(11);     // waiting for S
        const int vis = limit - kFT * j;                  // visible columns of this tile (may be <= 0)
        // scaled maximum of the tile's visible columns (a pass of its own: first tile and fall-back only)
        auto tile_max = [&]() {
          float mxs[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t x[32];
            tmem_ld32(s_addr + 32 * c, x);
            tmem_wait_ld();
            if (vis >= kFT) {
#pragma unroll
              for (int i = 0; i < 32; ++i) mxs[i & 3] = fmaxf(mxs[i & 3], __uint_as_float(x[i]));
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (32 * c + i < vis) mxs[i & 3] = fmaxf(mxs[i & 3], __uint_as_float(x[i]));
            }
          }
          return fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])) * sl2;
        };
        // raises the reference of the rows that ask for it to `to` and rescales their sums and O
        auto raise_to = [&](bool raise, float to) {
          float corr = 1.f;
          if (raise) {
            corr = fast_exp2(m_used - to);                // 0 when m_used is -inf
            m_used = to;
            l *= corr;
            l_mma *= corr;
          }
          if (j > 0 && __any_sync(0xffffffffu, raise)) return rescale_o(j, corr);
          return true;
        };
        if (j == 0) {
          ok = raise_to(true, tile_max());
          if (!ok) break;
        }
        HGA_TRACE_POINT(13);
        // p = 2^(x - m); P (bf16) is written over S once the whole tile is known to be in range.  l sums the
        // exact probabilities (for LSE), l_mma the rounded ones the MMA really applies: normalising O by THEIR
        // sum makes the rounding of a dominant weight cancel.  Two columns per step on packed fp32 pairs.
        uint32_t pk[32];
        float t_l, t_r, t_max;
        auto exp_pass = [&]() {
          const float neg_m = -m_used;
          const uint64_t neg_m2 = pack_f32x2(neg_m, neg_m);
          uint64_t lsum = pack_f32x2(0.f, 0.f), rsum = pack_f32x2(0.f, 0.f);
          float mxa = -INFINITY, mxb = -INFINITY;
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t x[32];
            tmem_ld32(s_addr + 32 * c, x);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float x0 = __uint_as_float(x[2 * i]), x1 = __uint_as_float(x[2 * i + 1]);
              float a0, a1;
              unpack_f32x2(fma_f32x2(pack_f32x2(x0, x1), sl2_2, neg_m2), a0, a1);
              float p0 = fast_exp2(a0), p1 = fast_exp2(a1);
              if (vis < kFT) {                            // diagonal / ragged tile only
                if (32 * c + 2 * i >= vis) { p0 = 0.f; a0 = -INFINITY; }
                if (32 * c + 2 * i + 1 >= vis) { p1 = 0.f; a1 = -INFINITY; }
              }
              if (i & 1) mxb = fmaxf(mxb, fmaxf(a0, a1)); else mxa = fmaxf(mxa, fmaxf(a0, a1));
              lsum = add_f32x2(lsum, pack_f32x2(p0, p1));
              const __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
              pk[16 * c + i] = *reinterpret_cast<const uint32_t*>(&hh);
              rsum = add_f32x2(rsum, pack_f32x2(__uint_as_float(pk[16 * c + i] << 16), __uint_as_float(pk[16 * c + i] & 0xffff0000u)));
            }
          }
          float la, lb, ra, rb;
          unpack_f32x2(lsum, la, lb);
          unpack_f32x2(rsum, ra, rb);
          t_l = la + lb;
          t_r = ra + rb;
          t_max = fmaxf(mxa, mxb);                        // largest exponent argument = tile maximum - m_used
        };
        exp_pass();
        if (__any_sync(0xffffffffu, t_max > kRescaleThreshold)) {
          // the tile's maximum outgrows the reference: raise it to that maximum and take the exponentials again
          ok = raise_to(t_max > kRescaleThreshold, m_used + t_max);
          if (!ok) break;
          exp_pass();
        }
        {
          uint32_t out[16];
#pragma unroll
          for (int c = 0; c < 2; ++c) {
#pragma unroll
            for (int i = 0; i < 16; ++i) out[i] = pk[16 * c + i];
            tmem_st16(s_addr + c * 16, out);
          }
        }
        l += t_l;
        l_mma += t_r;
        HGA_TRACE_POINT(14);
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&sm.p_full[j & 1]);
        HGA_TRACE_POINT(15);
      }
      if (ok) ok = __all_sync(0xffffffffu, wait_or_abort(&sm.o_done, 0, abort));
      HGA_TRACE_POINT(20);
      if (ok && warp_real) {
        // every lane takes part in the TMEM loads (warp-wide instructions); only real rows are stored
        tc_fence_after_sync();
        const float inv = 1.f / l_mma;
        const int hq = h * dm.G + a, srow = qb * dm.Bq + t;
        uint16_t* orow = O + b * dm.os[0] + hq * dm.os[1] + (int64_t)srow * dm.os[2];
#pragma unroll
        for (int c2 = 0; c2 < D / 64; ++c2) {
          uint32_t y[2][32];
          tmem_ld32(o_addr + c2 * 64, y[0]);
          tmem_ld32(o_addr + c2 * 64 + 32, y[1]);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(y[c][2 * i]) * inv,
                                                               __uint_as_float(y[c][2 * i + 1]) * inv);
              pk[i] = *reinterpret_cast<const uint32_t*>(&hh);
            }
            uint4* dst = reinterpret_cast<uint4*>(orow + c2 * 64 + c * 32);
            if (real_row) {
#pragma unroll
              for (int i = 0; i < 4; ++i) dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
            }
          }
        }
        if (real_row) LSE[((int64_t)b * dm.Hq + hq) * dm.S + srow] = (m_used + log2f(l)) * 0.6931471805599453f;
        HGA_TRACE_POINT(21);
      }
    }
  }

  // common exit: every role has either finished or given up; tensor memory is released
  HGA_TRACE_POINT(30);
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  HGA_TRACE_POINT(31);
  HGA_TRACE_DUMP;
  if (tid == 0 && sm.abort && status_word) atomicOr(status_word, HGA_FWD_ABORT_CODE(sm.abort));
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}

bool attn_fwd_sm100_supported(const Dims& dm) {
  if (dm.flags & HGA_FLAG_GENERIC_KERNELS) return false;
  const int rows_pad = rows_padded(dm);
  if (rows_pad > 128 && (rows_pad % 128 != 0 || rows_pad != dm.rows)) return false;
  if (rows_pad < 128 && !(dm.flags & HGA_FLAG_DECODE)) return false;   // small training shapes stay on the generic kernel
  if (dm.g % 8 != 0) return false;
  return true;
}

template <int D>
static int launch_fwd(const Dims& dm, const void* Q, const void* K, const void* V,
                      const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                      int32_t* status_word, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  const uint32_t box[5] = {64, 8, (uint32_t)(D / 64), 1, 1};
  const uint64_t dq[5] = {64, (uint64_t)dm.S, (uint64_t)(D / 64), (uint64_t)dm.Hq, (uint64_t)dm.B};
  const uint64_t dk[5] = {64, (uint64_t)dm.L, (uint64_t)(D / 64), (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t sq[4] = {(uint64_t)dm.qs[2] * 2, 128, (uint64_t)dm.qs[1] * 2, (uint64_t)dm.qs[0] * 2};
  const uint64_t sk[4] = {(uint64_t)dm.ks[2] * 2, 128, (uint64_t)dm.ks[1] * 2, (uint64_t)dm.ks[0] * 2};
  const uint64_t sv[4] = {(uint64_t)dm.vs[2] * 2, 128, (uint64_t)dm.vs[1] * 2, (uint64_t)dm.vs[0] * 2};
  if (encode_tensor_map_bf16(&mq, Q, 5, dq, sq, box, true) ||
      encode_tensor_map_bf16(&mk, K, 5, dk, sk, box, true) ||
      encode_tensor_map_bf16(&mv, V, 5, dk, sv, box, true))
    return HGA_ERR_UNSUPPORTED;
  const size_t smem = sizeof(FwdSmem<D>) + sizeof(int) * (max_routed_tokens(dm) / 8 + 8) + 1024;
  if (smem > 113 * 1024) return HGA_ERR_UNSUPPORTED;      // two CTAs per SM
  // two CTAs per SM need the largest shared-memory carve-out
  const int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(&k_attn_fwd_sm100<D>), smem, true);
  if (rc) return rc;
  const int units = dm.B * dm.Hkv * dm.NQB * ((rows_padded(dm) + 127) / 128);
  k_attn_fwd_sm100<D><<<units, kFwdThreads, smem, st>>>(mq, mk, mv, group_idx, n_groups, dm, (uint16_t*)O, LSE,
                                                       status_word);
  count_launch(HGA_KERNELS_FWD_TENSOR);
  return record_cuda(cudaGetLastError());
}

int launch_attn_fwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V,
                          const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                          int32_t* status_word, cudaStream_t st) {
  if (dm.d == 128) return launch_fwd<128>(dm, Q, K, V, group_idx, n_groups, O, LSE, status_word, st);
  return launch_fwd<64>(dm, Q, K, V, group_idx, n_groups, O, LSE, status_word, st);
}

}  // namespace hga
