// Key-major backward of the local band for sm_100a (head_dim 128): dK and dV of the keys that query
// blocks see through their local window or their own causal block (Section 2.1: the dense part of
// the routed set; Section 2.2: only keys of the active segment receive gradients).
//
// Every key of the active segment lies in the band of a few consecutive query blocks (its own
// block and the ones whose local window still reaches it).  Summing those contributions with
// atomics from the query-major sweep costs one red.add per element per contributing M-tile; here
// one CTA owns a 128-key tile instead, loops over every 128-row M-tile of every query block whose
// band touches the tile, accumulates dK and dV in tensor memory and writes the tile once with plain
// stores.  The query-major sweep (k_attn_bwd_sm100) then adds only the contributions of keys
// selected through routing (and of sink keys inside the active segment), and computes dQ.
//
// The GEMMs are the TRANSPOSED ones, so that P and dS never pass through shared memory:
//   S^T  = K Q^T,  dP^T = V dO^T         (M = 128 keys, N = 64 query rows, K = head_dim)   smem x smem
//   P^T  = 2^(S^T*c - LSE*log2e),  dS^T = scale * P^T o (dP^T - delta)    one thread per KEY (TMEM lane),
//          written back as bf16 over the columns just read
//   dV  += P^T dO,  dK += dS^T Q         (M = 128 keys, N = head_dim, K = 64 query rows)   A from TMEM
// An M-tile (128 query rows) is taken in two HALF-STEPS of 64 rows that alternate between two 128-column
// regions of tensor memory, so that the GEMMs of one half-step run while the key threads work on the other
// (with one 256-column region per M-tile the tensor pipe idled through the key threads' work and vice versa).
// delta = rowsum(dO o O) of the M-tile's rows is computed here, by four otherwise idle warps (one
// thread per query row, from the O and dO tiles in shared memory; the O tile arrives by TMA one step
// ahead), so the backward needs no separate pass over O and dO.
//
// Work unit (one CTA): (batch, kv head, 128-key tile of the active segment); keys past the end of the
// segment arrive as zeros, are masked by causality and are not stored.
// Warp roles (448 threads): warp 0 producer (K, V once; Q, dO tiles through a two-stage ring, O tiles one at a time),
// warp 1 MMA issuer, warps 2-5 and 6-9 one thread per key (warpgroup w: query rows 32w .. 32w+31 of
// every half-step), warps 10-13 row statistics (LSE, delta).
// TMEM (512 columns): two regions of [S^T / P^T (64) | dP^T / dS^T (64)], then dV and dK, 128 columns each.
#include "hga_bwd_sm100.cuh"
#include "hga_common.cuh"
#include "hga_sm100.cuh"

namespace hga {

using namespace sm100;

namespace {

constexpr int kBandThreads = 448;
constexpr int kD = 128;
constexpr int kKeys = 128;                       // keys per CTA
constexpr int kTile = 128 * kD * 2;              // bytes of one K, V, Q or dO tile: [panel][128 rows][128 B]

struct BandSmem {
  alignas(1024) uint8_t k[kTile];
  alignas(1024) uint8_t v[kTile];
  alignas(1024) uint8_t q[2][kTile];
  alignas(1024) uint8_t dO[2][kTile];
  alignas(1024) uint8_t o[kTile];                // (q, dO and o, contiguous, also stage the dV / dK tiles on their way out)
  alignas(16) float nlse[128];                   // per query row of the current M-tile: -LSE * log2(e)
  alignas(16) float nds[128];                    //                                      -delta * scale
  uint64_t kv_full, qdo_full[2][2], qdo_empty[2][2], o_full, o_empty;   // Q/dO: [ring stage][half of the M-tile's rows]
  // per half of the M-tile (= per region of tensor memory), so that every barrier completes once per step and
  // each completion depends on its waiter having seen the previous one
  uint64_t stat_full[2], sdp_full[2], pds_full[2], acc_done, drain;
  uint32_t tmem_base;
  volatile int abort;
};

// query block of step m, and the first query row (inside the item) of its M-tile
struct Step {
  int qb, r0;
};

}  // namespace

__global__ void __launch_bounds__(kBandThreads, 1)
k_attn_bwd_band_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                      const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const __grid_constant__ CUtensorMap map_o, const float* __restrict__ LSE, Dims dm,
                      float* __restrict__ dK, float* __restrict__ dV, int32_t* status_word) {
  constexpr uint32_t kColS = 0, kColDP = 64, kRegion = 128, kColDV = 256, kColDK = 384;   // (S^T, dP^T: inside a region)
  extern __shared__ uint8_t smem_raw[];
  BandSmem& sm = *reinterpret_cast<BandSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  HGA_TRACE_DECL;
  const int tiles_per_seq = (dm.S + kKeys - 1) / kKeys;
  const int kt = blockIdx.x % tiles_per_seq;
  const int bh = blockIdx.x / tiles_per_seq;
  const int h = bh % dm.Hkv, b = bh / dm.Hkv;
  const int k0 = dm.H + kt * kKeys;               // first key position of the tile
  const int k_end = min(k0 + kKeys, dm.L);        // one past its last real key
  // query blocks whose band [ls, p0 + Bq) touches the tile: from the block that holds the tile's first
  // key, while the local window still starts before the tile's end
  const int qb_first = (kt * kKeys) / dm.Bq;
  int n_qb = 1;
  while (qb_first + n_qb < dm.NQB && window_of(dm, qb_first + n_qb).ls < k_end) ++n_qb;
  const int n_mt = dm.rows / 128;
  const int n_steps = n_qb * n_mt;
  auto step_of = [&](int m) { return Step{qb_first + m / n_mt, (m % n_mt) * 128}; };

  if (tid == 0) {
    mbar_init(&sm.kv_full, 1);
    for (int s = 0; s < 4; ++s) {
      mbar_init(&sm.qdo_full[s >> 1][s & 1], 1); mbar_init(&sm.qdo_empty[s >> 1][s & 1], 1);
    }
    mbar_init(&sm.o_full, 1); mbar_init(&sm.o_empty, 128);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.stat_full[s], 64); mbar_init(&sm.sdp_full[s], 1); mbar_init(&sm.pds_full[s], 256);
    }
    mbar_init(&sm.acc_done, 1); mbar_init(&sm.drain, 1);
    sm.abort = 0;
    fence_barrier_init();
    // the copies of the K and V tile, of the first two steps' Q and dO and of the first O tile are issued by
    // twelve warps at once right after the block barrier below; their byte counts are announced here
    mbar_arrive_expect_tx(&sm.kv_full, 2 * kTile);
    mbar_arrive_expect_tx(&sm.o_full, kTile);
    for (int s = 0; s < (n_steps > 1 ? 4 : 2); ++s) mbar_arrive_expect_tx(&sm.qdo_full[s >> 1][s & 1], kTile);
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  // the sweep, next in the stream, may start on SMs this grid leaves idle (it waits for this grid only
  // before it adds to dK/dV)
  if (tid == 0) pdl_launch_dependents();

  const uint32_t tmem = sm.tmem_base;
  volatile int* abort = &sm.abort;
  HGA_TRACE_POINT(1);

  // A copy is latency-bound per box and costs its issuing warp a few hundred cycles, so every tile travels as
  // four boxes of 64 rows x one 64-element panel (8 KB each); the 28 boxes a CTA starts with go out from
  // twelve warps in parallel, in the order they are needed: K, V, the first half-step's Q and dO rows, the
  // second half-step's, the first O tile, then the second step's Q and dO.
  auto qdo_coords = [&](int m, int half, int& row, int& head) {
    const Step sp = step_of(m);
    const int r = sp.r0 + 64 * half;
    row = sp.qb * dm.Bq + r % dm.Bq;
    head = h * dm.G + r / dm.Bq;
  };
  if (warp >= 2 && lane == 0) {
    for (int i = warp - 2; i < (n_steps > 1 ? 28 : 20); i += 12) {
      int row, head;
      // All CTAs start at once and HBM is the bottleneck of these first microseconds: what the first
      // half-step needs (the first twelve boxes) goes out alone, the rest once that has arrived
      if (i >= 12 && !(bwd_wait(&sm.kv_full, 0, abort) && bwd_wait(&sm.qdo_full[0][0], 0, abort))) break;
      if (i < 8) {                                   // K, V: (half, panel) = (i & 1, (i >> 1) & 1)
        const int half = i & 1, panel = (i >> 1) & 1;
        const uint32_t off = (uint32_t)panel * 16384 + (uint32_t)half * 8192;
        tma_load_5d((i < 4 ? sm.k : sm.v) + off, i < 4 ? &map_k : &map_v, &sm.kv_full, 0, k0 + 64 * half, panel, h, b);
      } else if (i < 16) {                           // step 0: half (i - 8) / 4, then Q panel 0, 1, dO panel 0, 1
        const int half = (i - 8) >> 2, panel = i & 1, is_do = (i >> 1) & 1;
        const uint32_t off = (uint32_t)panel * 16384 + (uint32_t)half * 8192;
        qdo_coords(0, half, row, head);
        tma_load_5d((is_do ? sm.dO[0] : sm.q[0]) + off, is_do ? &map_do : &map_q, &sm.qdo_full[0][half], 0, row, panel, head, b);
      } else if (i < 20) {                           // O tile of step 0
        const int half = i & 1, panel = (i >> 1) & 1;
        const uint32_t off = (uint32_t)panel * 16384 + (uint32_t)half * 8192;
        qdo_coords(0, half, row, head);
        tma_load_5d(sm.o + off, &map_o, &sm.o_full, 0, row, panel, head, b);
      } else {                                       // step 1, as step 0
        const int half = (i - 20) >> 2, panel = i & 1, is_do = (i >> 1) & 1;
        const uint32_t off = (uint32_t)panel * 16384 + (uint32_t)half * 8192;
        qdo_coords(1, half, row, head);
        tma_load_5d((is_do ? sm.dO[1] : sm.q[1]) + off, is_do ? &map_do : &map_q, &sm.qdo_full[1][half], 0, row, panel, head, b);
      }
    }
  }
  __syncwarp();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (Q and dO from the third step on)
    if (lane == 0) {
      prefetch_tensormap(&map_q); prefetch_tensormap(&map_do);
    }
    bool ok = true;
    int issued = n_steps > 1 ? 4 : 2;                // half-steps whose copies have been issued
    for (int m = 2; m < n_steps && ok; ++m) {
      const int st = m & 1;
      // one half of the rows (Q panel 0, 1, dO panel 0, 1: lanes 0-3) at a time: a half is free again as soon
      // as the GEMMs of its half-step two steps ago are done
      for (int hf = 0; hf < 2 && ok; ++hf) {
        if (lane == 0) ok = bwd_wait(&sm.qdo_empty[st][hf], ((m >> 1) - 1) & 1, abort);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(&sm.qdo_full[st][hf], kTile);
        __syncwarp();
        if (lane < 4) {
          const int panel = lane & 1, is_do = lane >> 1;
          const uint32_t off = (uint32_t)panel * 16384 + (uint32_t)hf * 8192;
          int row, head;
          qdo_coords(m, hf, row, head);
          tma_load_5d((is_do ? sm.dO[st] : sm.q[st]) + off, is_do ? &map_do : &map_q, &sm.qdo_full[st][hf], 0, row, panel, head, b);
        }
        issued = 2 * m + hf + 1;
        HGA_TRACE_POINT(2);
      }
    }
    if (*abort && lane == 0) {
      // giving up: let the copies still in flight land before shared memory is released
      mbar_wait(&sm.kv_full, 0);
      for (int hs = issued > 4 ? issued - 4 : 0; hs < issued; ++hs)
        mbar_wait(&sm.qdo_full[(hs >> 1) & 1][hs & 1], (hs >> 2) & 1);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs this branch converged (waits included) and one elected lane issues: see mma_ss_w.
    {
      auto mma_wait = [&](uint64_t* bar, uint32_t parity, volatile int* ab) {
        return __all_sync(0xffffffffu, bwd_wait(bar, parity, ab));
      };
      constexpr uint32_t idesc_t = idesc_bf16_f32(128, 64, 0, 0);      // keys x 64 rows: A, B K-major (head_dim runs along K)
      constexpr uint32_t idesc_g = idesc_bf16_f32(128, kD, 0, 1);      // keys x head_dim: A from TMEM, B MN-major
      // every tile is [panel][128 rows][128 B]: K-major with 8-row groups 1024 B apart and the second
      // panel 16 KB on; MN-major (head_dim along N, rows along K) with panels 16 KB and 8-row groups 1024 B apart.
      // The rows of half-step hf start 64 * 128 B = 8 KB into each panel.
      const uint64_t k_k = smem_desc_sw128(smem_u32(sm.k), 16, 1024);
      const uint64_t v_k = smem_desc_sw128(smem_u32(sm.v), 16, 1024);
      const uint64_t q_k0 = smem_desc_sw128(smem_u32(sm.q[0]), 16, 1024);
      const uint64_t do_k0 = smem_desc_sw128(smem_u32(sm.dO[0]), 16, 1024);
      const uint64_t q_mn0 = smem_desc_sw128(smem_u32(sm.q[0]), 16384, 1024);
      const uint64_t do_mn0 = smem_desc_sw128(smem_u32(sm.dO[0]), 16384, 1024);
      // acc (keys x 64 rows) = a (K or V tile) x b^T (64 rows of the Q or dO tile), both K-major
      auto issue_t = [&](uint32_t acc, uint64_t a, uint64_t bq) {
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint32_t off = (kk >> 2) * 16384 + (kk & 3) * 32;       // panel, then 32-byte K step
          mma_ss_w(acc, desc_advance(a, off), desc_advance(bq, off), idesc_t, kk > 0);
        }
      };
      // acc (keys x head_dim) += a (keys x 64 rows, bf16 in TMEM: rows 0-31 at columns 0-15, rows 32-63 at
      // columns 32-47 of its S^T or dP^T part) x b (64 rows of the Q or dO tile: rows along K, 16 per instruction)
      auto issue_g = [&](uint32_t acc, uint32_t a_tmem, uint64_t bmn, bool accumulate) {
#pragma unroll
        for (int kk = 0; kk < 64 / 16; ++kk)
          mma_ts_w(acc, a_tmem + (kk < 2 ? 8 * kk : 32 + 8 * (kk - 2)), desc_advance(bmn, kk * 2048), idesc_g,
                   (accumulate || kk > 0));
      };
      // S^T and dP^T of half-step hf of the M-tile in ring stage st, into region hf
      auto issue_sdp = [&](uint32_t st, uint32_t hf) {
        const uint32_t region = tmem + hf * kRegion, off = st * kTile + hf * 8192;
        issue_t(region + kColS, k_k, desc_advance(q_k0, off));
        issue_t(region + kColDP, v_k, desc_advance(do_k0, off));
        mma_commit_w(&sm.sdp_full[hf]);
      };
      const int n_half = 2 * n_steps;
      bool ok = mma_wait(&sm.kv_full, 0, abort);
      for (uint32_t hf = 0; hf < 2 && ok; ++hf) {
        ok = mma_wait(&sm.qdo_full[0][hf], 0, abort);
        if (!ok) break;
        tc_fence_after_sync();
        issue_sdp(0, hf);
      }
      HGA_TRACE_POINT(3);
      for (int hs = 0; hs < n_half && ok; ++hs) {
        const int m = hs >> 1;
        const uint32_t st = (uint32_t)(m & 1), hf = (uint32_t)(hs & 1);
        ok = mma_wait(&sm.pds_full[hf], m & 1, abort);           // P^T and dS^T of this half-step are in TMEM
        if (!ok) break;
        tc_fence_after_sync();
        HGA_TRACE_POINT(5);
        const uint32_t region = tmem + hf * kRegion, off = st * kTile + hf * 8192;
        issue_g(tmem + kColDV, region + kColS, desc_advance(do_mn0, off), hs > 0);
        issue_g(tmem + kColDK, region + kColDP, desc_advance(q_mn0, off), hs > 0);
        mma_commit_w(&sm.qdo_empty[st][hf]);                     // these 64 rows of Q and dO are consumed
        if (hs + 2 < n_half) {
          // the same half of the next M-tile reuses this region: the in-order tensor pipe runs its GEMMs after
          // the two above, which read P^T and dS^T from it
          const uint32_t st_n = st ^ 1u;
          ok = mma_wait(&sm.qdo_full[st_n][hf], ((m + 1) >> 1) & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
          issue_sdp(st_n, hf);
        }
        HGA_TRACE_POINT(7);
      }
      if (ok) mma_commit_w(&sm.acc_done);
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------------ one thread per key
    const int wg = (warp - 2) >> 2;                  // query rows 32*wg .. 32*wg+31 of every half-step
    const int quarter = warp & 3;                    // TMEM lanes this warp may touch
    const int key = quarter * 32 + lane;
    const int kp = k0 + key;                         // absolute position of this thread's key
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    const float sl2 = dm.scale * 1.4426950408889634f;
    const uint64_t sl2_2 = pack_f32x2(sl2, sl2), scale_2 = pack_f32x2(dm.scale, dm.scale);
    bool ok = true;
    for (int hs = 0; hs < 2 * n_steps; ++hs) {
      const int m = hs >> 1, hf = hs & 1;
      const Step sp = step_of(m);
      const Window w = window_of(dm, sp.qb);
      // the warpgroup's 32 columns are 32 consecutive positions of one query head (Bq is a multiple of 64);
      // column i is visible to this key iff the key is inside the block's band and not after the query
      const int r_first = 64 * hf + 32 * wg;         // first of those rows inside the M-tile
      const int qp0 = w.p0 + (sp.r0 + r_first) % dm.Bq;
      const int imin = (kp < w.ls || kp >= k_end) ? 32 : kp - qp0;       // first visible column (may be <= 0)
      const bool none = __all_sync(0xffffffffu, imin >= 32);
      const bool masked = __any_sync(0xffffffffu, imin > 0);
      const uint32_t nlse_a = smem_u32(&sm.nlse[r_first]), nds_a = smem_u32(&sm.nds[r_first]);
      const uint32_t s_addr = lane_base + hf * kRegion + kColS + 32 * wg;
      const uint32_t dp_addr = lane_base + hf * kRegion + kColDP + 32 * wg;
      uint32_t pk[16];                               // P of this key against 32 query rows, packed bf16
      ok = __all_sync(0xffffffffu, bwd_wait(&sm.sdp_full[hf], m & 1, abort));
      if (ok) ok = __all_sync(0xffffffffu, bwd_wait(&sm.stat_full[hf], m & 1, abort));
      if (!ok) break;
      tc_fence_after_sync();
      HGA_TRACE_POINT(11);
      if (none) {
        // no key of this warp is visible to any of the 32 rows: zeros, no exponentials
#pragma unroll
        for (int i = 0; i < 16; ++i) pk[i] = 0u;
      } else {
        uint32_t x[32];
        tmem_ld32(s_addr, x);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          uint32_t n0, n1, n2, n3;                   // -LSE*log2e of four consecutive columns
          ld_shared_v4(nlse_a + (2 * i) * 4, n0, n1, n2, n3);
          float a0, a1, a2, a3;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(x[2 * i]), __uint_as_float(x[2 * i + 1])), sl2_2,
                                 pack_f32x2(__uint_as_float(n0), __uint_as_float(n1))), a0, a1);
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(x[2 * i + 2]), __uint_as_float(x[2 * i + 3])), sl2_2,
                                 pack_f32x2(__uint_as_float(n2), __uint_as_float(n3))), a2, a3);
          float p0 = fast_exp2(a0), p1 = fast_exp2(a1), p2 = fast_exp2(a2), p3 = fast_exp2(a3);
          if (masked) {
            const int col = 2 * i;
            if (col < imin) p0 = 0.f;
            if (col + 1 < imin) p1 = 0.f;
            if (col + 2 < imin) p2 = 0.f;
            if (col + 3 < imin) p3 = 0.f;
          }
          pk[i] = pack_bf16(p0, p1);
          pk[i + 1] = pack_bf16(p2, p3);
        }
      }
      tmem_st16(s_addr, pk);                         // P^T (bf16) over the first 16 of the S^T columns just read
      HGA_TRACE_POINT(13);
      {
        uint32_t out[16];
        if (!none) {
          uint32_t x[32];
          tmem_ld32(dp_addr, x);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            uint32_t n0, n1, n2, n3;                 // -delta*scale of four consecutive columns
            ld_shared_v4(nds_a + (2 * i) * 4, n0, n1, n2, n3);
            const uint32_t pa = pk[i], pb = pk[i + 1];
            const uint64_t g0 = fma_f32x2(pack_f32x2(__uint_as_float(x[2 * i]), __uint_as_float(x[2 * i + 1])), scale_2,
                                          pack_f32x2(__uint_as_float(n0), __uint_as_float(n1)));
            const uint64_t g1 = fma_f32x2(pack_f32x2(__uint_as_float(x[2 * i + 2]), __uint_as_float(x[2 * i + 3])), scale_2,
                                          pack_f32x2(__uint_as_float(n2), __uint_as_float(n3)));
            float d0, d1, d2, d3;
            unpack_f32x2(mul_f32x2(pack_f32x2(__uint_as_float(pa << 16), __uint_as_float(pa & 0xffff0000u)), g0), d0, d1);
            unpack_f32x2(mul_f32x2(pack_f32x2(__uint_as_float(pb << 16), __uint_as_float(pb & 0xffff0000u)), g1), d2, d3);
            out[i] = pack_bf16(d0, d1);
            out[i + 1] = pack_bf16(d2, d3);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) out[i] = 0u;
        }
        tmem_st16(dp_addr, out);                     // dS^T (bf16) over the first 16 of the dP^T columns just read
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(&sm.pds_full[hf]);
      HGA_TRACE_POINT(14);
    }
    if (ok) ok = __all_sync(0xffffffffu, bwd_wait(&sm.acc_done, 0, abort));
    HGA_TRACE_POINT(20);
    if (ok) {
      // epilogue: thread = key row; warpgroup 0 sends dV, warpgroup 1 dK.  A row (512 bytes) goes through
      // shared memory (the Q / dO / O tiles, free now: every GEMM and every copy into them is complete) and
      // leaves as one bulk copy, or one bulk add with the accumulate flag; rows are 528 bytes apart so that
      // the 16-byte stores of a quarter warp fall into different banks
      tc_fence_after_sync();
      constexpr uint32_t kRowPitch = kD * 4 + 16;
      static_assert(2 * 128 * kRowPitch <= 5 * kTile, "staging area: q, dO and o tiles");
      const int srow = kt * kKeys + key;
      float* dst = (wg == 0 ? dV : dK) + ((int64_t)(b * dm.Hkv + h) * dm.S + srow) * kD;
      const uint32_t col = wg == 0 ? kColDV : kColDK;
      const uint32_t stage = smem_u32(sm.q[0]) + (uint32_t)(wg * 128 + key) * kRowPitch;
#pragma unroll
      for (int c = 0; c < kD / 32; ++c) {
        uint32_t x[32];
        tmem_ld32(lane_base + col + 32 * c, x);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) st_shared_v4(stage + (uint32_t)(32 * c + 4 * i) * 4, x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
      }
      fence_proxy_async_smem();
      if (srow < dm.S) {
        if (dm.flags & HGA_FLAG_BWD_ACCUMULATE) bulk_reduce_add_f32(dst, stage, kD * 4);
        else bulk_store(dst, stage, kD * 4);
        tma_store_commit();
        tma_store_wait_read();
      }
    }
  } else {
    // ------------------------------------------------------------------ row statistics, one thread per query row
    const int j = (warp - 10) * 32 + lane;           // row of the M-tile
    const uint32_t key7 = (uint32_t)(j & 7);
    auto lse_of = [&](int m) {
      const Step sp = step_of(m);
      const int r = sp.r0 + j;
      return LSE[((int64_t)b * dm.Hq + h * dm.G + r / dm.Bq) * dm.S + sp.qb * dm.Bq + r % dm.Bq];
    };
    float lse_next = lse_of(0);
    bool ok = true;
    int o_issued = 1;                                // O tiles whose copies have been issued
    for (int m = 0; m < n_steps; ++m) {
      const int st = m & 1;
      const float lse = lse_next;
      if (m + 1 < n_steps) lse_next = lse_of(m + 1);
      ok = __all_sync(0xffffffffu, bwd_wait(&sm.qdo_full[st][j >> 6], (m >> 1) & 1, abort));   // (this row's half of dO)
      HGA_TRACE_POINT(11);
      if (ok) ok = __all_sync(0xffffffffu, bwd_wait(&sm.o_full, m & 1, abort));
      if (!ok) break;
      HGA_TRACE_POINT(13);
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const uint32_t do_line = smem_u32(sm.dO[st]) + (uint32_t)j * 128, o_line = smem_u32(sm.o) + (uint32_t)j * 128;
#pragma unroll
      for (int i = 0; i < 16; ++i) {                 // 16-byte chunk i of the row: panel i / 8, chunk i % 8 (XOR-swizzled)
        const uint32_t off = (uint32_t)(i >> 3) * 16384 + (((uint32_t)(i & 7) ^ key7) * 16);
        uint32_t xs[4], ys[4];
        ld_shared_v4(o_line + off, xs[0], xs[1], xs[2], xs[3]);
        ld_shared_v4(do_line + off, ys[0], ys[1], ys[2], ys[3]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          acc[e] = fmaf(__uint_as_float(xs[e] << 16), __uint_as_float(ys[e] << 16), acc[e]);
          acc[e] = fmaf(__uint_as_float(xs[e] & 0xffff0000u), __uint_as_float(ys[e] & 0xffff0000u), acc[e]);
        }
      }
      mbar_arrive(&sm.o_empty);                      // the O tile may be overwritten by the next step's
      if (warp == 13 && m + 1 < n_steps) {
        // ... which this warp -- the one whose rows of dO arrive last -- fetches as soon as all four
        // statistics warps have read this one
        if (lane == 0) ok = bwd_wait(&sm.o_empty, m & 1, abort);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(&sm.o_full, kTile);
        __syncwarp();
        if (lane < 4) {
          const int half = lane & 1, panel = lane >> 1;
          int row, head;
          qdo_coords(m + 1, half, row, head);
          tma_load_5d(sm.o + (uint32_t)panel * 16384 + (uint32_t)half * 8192, &map_o, &sm.o_full, 0, row, panel, head, b);
        }
        o_issued = m + 2;
      }
      const float delta = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      HGA_TRACE_POINT(15);
      // the key threads read the previous step's statistics of this half until they hand its P^T and dS^T over
      if (m > 0) ok = __all_sync(0xffffffffu, bwd_wait(&sm.pds_full[j >> 6], (m - 1) & 1, abort));
      if (!ok) break;
      sm.nlse[j] = -lse * 1.4426950408889634f;
      sm.nds[j] = -delta * dm.scale;
      mbar_arrive(&sm.stat_full[j >> 6]);
      HGA_TRACE_POINT(14);
    }
    // giving up: let the O copy still in flight land before shared memory is released
    if (*abort && warp == 13 && lane == 0) mbar_wait(&sm.o_full, (o_issued - 1) & 1);
  }
  HGA_TRACE_POINT(30);

  // every warp reconverges before the block barrier (a barrier reached by part of a warp would
  // count that warp as arrived)
  __syncwarp();
  if (warp == 1 && sm.abort) {
    // giving up: GEMMs already issued may still be writing tensor memory; wait (bounded) until the
    // tensor pipe has run dry before the columns are given back
    mma_commit_w(&sm.drain);
    mbar_wait(&sm.drain, 0);
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  HGA_TRACE_DUMP;
  if (tid == 0 && sm.abort && status_word) atomicOr(status_word, HGA_ABORT_CODE(2, sm.abort));
  if (warp == 1) tmem_dealloc(tmem, 512);
}

bool attn_bwd_band_sm100_supported(const Dims& dm) {
  if (dm.flags & HGA_FLAG_GENERIC_KERNELS) return false;
  return dm.d == 128 && dm.rows % 128 == 0 && dm.Bq % 64 == 0;
}

int launch_attn_bwd_band_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const void* O,
                               const float* LSE, const void* dO, float* dK, float* dV, int32_t* status_word,
                               cudaStream_t st) {
  CUtensorMap mq, mdo, mk, mv, mo;
  const uint32_t box[5] = {64, 64, 1, 1, 1};
  const uint64_t dq[5] = {64, (uint64_t)dm.S, 2, (uint64_t)dm.Hq, (uint64_t)dm.B};
  const uint64_t dk[5] = {64, (uint64_t)dm.L, 2, (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t sq[4] = {(uint64_t)dm.qs[2] * 2, 128, (uint64_t)dm.qs[1] * 2, (uint64_t)dm.qs[0] * 2};
  const uint64_t so[4] = {(uint64_t)dm.os[2] * 2, 128, (uint64_t)dm.os[1] * 2, (uint64_t)dm.os[0] * 2};
  const uint64_t sk[4] = {(uint64_t)dm.ks[2] * 2, 128, (uint64_t)dm.ks[1] * 2, (uint64_t)dm.ks[0] * 2};
  const uint64_t sv[4] = {(uint64_t)dm.vs[2] * 2, 128, (uint64_t)dm.vs[1] * 2, (uint64_t)dm.vs[0] * 2};
  if (encode_tensor_map_bf16(&mq, Q, 5, dq, sq, box, true) ||
      encode_tensor_map_bf16(&mdo, dO, 5, dq, so, box, true) ||
      encode_tensor_map_bf16(&mo, O, 5, dq, so, box, true) ||
      encode_tensor_map_bf16(&mk, K, 5, dk, sk, box, true) ||
      encode_tensor_map_bf16(&mv, V, 5, dk, sv, box, true))
    return HGA_ERR_UNSUPPORTED;
  const size_t smem = sizeof(BandSmem) + 1024;
  const int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(&k_attn_bwd_band_sm100), smem);
  if (rc) return rc;
  const int units = dm.B * dm.Hkv * ((dm.S + kKeys - 1) / kKeys);
  k_attn_bwd_band_sm100<<<units, kBandThreads, smem, st>>>(mq, mdo, mk, mv, mo, LSE, dm, dK, dV, status_word);
  count_launch(HGA_KERNELS_BWD_TENSOR);
  return record_cuda(cudaGetLastError());
}

}  // namespace hga
