// hga_attn_bwd for sm_100a (head_dim 128): backward of routed exact-token attention with the
// routing frozen (Section 2.1, last paragraph) and history K/V detached (Section 2.2).
//
// Work unit (one CTA): one 128-row M-tile of one item, swept over the item's routed keys, which
// TMA gathers in 64-key tiles (8 octets) exactly as in the forward kernel.  Two kinds of steps:
//
//  * dK/dV steps (one 64-key tile each): tiles that hold keys whose dK/dV this kernel must add,
//    i.e. keys of the active segment that lie before the local band: selected through routing, or
//    sink keys (the local band is written by the key-major kernel k_attn_bwd_band_sm100, which
//    runs first and stores every row of dK/dV).  They come first:
//      S = Q K^T, dP = dO V^T -> TMEM;  P, dS by one thread per row -> shared memory;
//      dQ += dS K;  dV^T = dO^T P, dK^T = Q^T dS (M = head_dim, N = 64 keys, K = 128 rows) -> TMEM,
//    then four reduction warps add the transposed tiles to global memory (a warp's 32 lanes hold 32
//    consecutive elements of one key row: one coalesced 128-byte red.global.add.f32 request).
//
//  * all other steps run on PAIRS of tiles (128 keys), because a tcgen05.mma with N = 64 runs at
//    little more than half the rate of one with N = 128:
//      S(u)  = Q K^T   (N = 128: two adjacent ring stages are one B operand)  -> TMEM region
//      dP(u) = dO V^T                                                          -> TMEM region
//      phase 1 of the row threads: P = 2^(S*c - LSE*log2e), kept as packed bf16 in registers;
//      phase 2: dS = scale * P o (dP - delta), written as bf16 over the dP columns already read;
//      dQ += dS K      (A = dS from TMEM, B = the two K stages, MN-major).
//    Three 128-column TMEM regions rotate: S(u+1) is issued while the row threads still work on
//    step u, dP(u+1) goes into S(u)'s region as soon as they are done with it, and dQ(u) follows; so
//    the exp2 of step u+1 overlaps the dP GEMM of step u+1, and the tensor pipe never waits for the
//    row threads except for that one hand-off.  The in-order tensor pipe makes the other hazards
//    (dQ(u) reads dS before S(u+2) overwrites it) free of barriers.
//
// Warp roles (512 threads): warp 0 copies K tiles and runs up to three pairs ahead, warps 14 and 15
// copy V tiles (half of each tile; in the paired steps V has room for two pairs -- its own two stages and
// the P / dS tiles, idle by then -- each refilled as soon as the dP GEMM that read it is done: with one
// pair only, the copy's latency sat between consecutive dP GEMMs), warp 1 MMA issuer, warps 2-5 and 6-9
// one thread per query row (warpgroup 0: first tile of a pair and all dK/dV steps; warpgroup 1:
// second tile of a pair; both write the dQ epilogue), warps 10-13 dK/dV reduction.
// Every barrier hand-off costs the MMA thread a few hundred cycles and every tcgen05.commit about a
// hundred, so a paired step has one full barrier per operand and pair, and the dP commit doubles as
// the V stages' release.
// TMEM (512 columns): region 0 | region 2 (aliased by dV^T, dK^T during the dK/dV steps) | dQ |
// region 1.  Shared memory: Q, dO (32 KB each), K ring of six 16 KB stages, V ring of two, P and dS
// (16 KB each, used by the dK/dV steps only).
// delta = rowsum(dO o O) of the CTA's 128 rows is computed during set-up by the row threads themselves
// (the O row from global memory, the dO row from the tile in shared memory; the two warpgroups take
// one 64-element half each), so no pass over O and dO precedes the kernel.
#include "hga_bwd_sm100.cuh"
#include "hga_common.cuh"
#include "hga_octets.cuh"
#include "hga_sm100.cuh"

#include <cstddef>

namespace hga {

using namespace sm100;

constexpr int kBwdThreads = 512;                // 16 warps: 128 registers per thread
constexpr int kBwdKStages = 6;                  // K ring: three pairs (a K tile is held until its dQ GEMM)
constexpr int kBwdVStages = 2;                  // V ring of the dK/dV steps; the paired steps add the P / dS tiles as a second pair
constexpr int kBwdD = 128;
constexpr int kKT = 64;                         // keys per tile
constexpr int kOct = 8 * kBwdD * 2;             // bytes of one octet of K/V/Q/dO rows (2 panels)
constexpr int kKvTile = kKT * kBwdD * 2;        // bytes of one K or V tile
constexpr int kPdsTile = 128 * kKT * 2;         // bytes of one P or dS tile

struct BwdSmem {
  alignas(1024) uint8_t q[128 * kBwdD * 2];
  alignas(1024) uint8_t dO[128 * kBwdD * 2];
  alignas(1024) uint8_t k[kBwdKStages][kKvTile];
  alignas(1024) uint8_t v[kBwdVStages][kKvTile];
  alignas(1024) uint8_t p[kPdsTile];            // [16 row octets][8 rows][128 B], 128-byte swizzle
  alignas(1024) uint8_t ds[kPdsTile];           // (P and dS pass through shared memory only for dK/dV tiles)
  uint64_t q_full, k_full[kBwdKStages], k_empty[kBwdKStages];   // (dK/dV steps: even stages hold K tiles, odd ones V tiles)
  uint64_t sdp_full, pds_full, dkv_full, dkv_free;      // dK/dV steps
  uint64_t s_full[2], dp_full[4], ds_full[2], s_read[2];   // paired steps (S(u+1) is committed before step u is over: two barriers;
                                                        // dP: four, so that a copy item taken ahead of time cannot mistake an older phase)
  uint64_t phase_a_done;                                // every GEMM of the dK/dV steps is complete
  uint64_t kp_full[kBwdKStages / 2], kp_empty[kBwdKStages], vp_full[2];    // paired steps: one barrier per pair of stages
                                                        // (kp_empty: indexed by pair number mod 6, see dp_full)
  uint64_t dq_done, dq_staged;
  uint32_t tmem_base;
  int n_oct, dkv_lo, n_dkv;    // tiles [dkv_lo, dkv_lo + n_dkv) are processed as dK/dV steps
  volatile int abort;
  int oct_row[1];
};

static_assert(kPdsTile == kKvTile && offsetof(BwdSmem, ds) == offsetof(BwdSmem, p) + kKvTile,
              "the P and dS tiles double as one pair of V stages");

__global__ void __launch_bounds__(kBwdThreads, 1)
k_attn_bwd_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                 const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                 const __grid_constant__ CUtensorMap map_dq, const uint16_t* __restrict__ O,
                 const float* __restrict__ LSE, const int32_t* __restrict__ group_idx,
                 const int32_t* __restrict__ n_groups, Dims dm,
                 float* __restrict__ dK, float* __restrict__ dV, int32_t* status_word) {
  constexpr int D = kBwdD;
  // TMEM columns.  Regions 0, 1, 2 rotate through the roles S / dP+dS of the paired steps; a dK/dV
  // step keeps S (64 columns) and dP (64) in region 0 and dV^T, dK^T in region 1.
  constexpr uint32_t kColDQ = 256;
  constexpr uint32_t kColDV = 128, kColDK = 192;
  // (region 2 is the one that aliases dV^T/dK^T: the paired steps reach it last)
  auto region = [](int r) -> uint32_t { return r == 0 ? 0u : (r == 1 ? 384u : 128u); };
  extern __shared__ uint8_t smem_raw[];
  BwdSmem& sm = *reinterpret_cast<BwdSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  HGA_TRACE_DECL;
  const int n_mt_item = dm.rows / 128;
  // Launch order: late query blocks first.  They have the most routed keys inside the active segment (the
  // expensive dK/dV steps), early ones none, so the cheapest CTAs are the ones that fill the last wave.
  const int unit = blockIdx.x / n_mt_item, n_bh = dm.B * dm.Hkv;
  const int item = (unit % n_bh) * dm.NQB + (dm.NQB - 1 - unit / n_bh);
  const int mt = blockIdx.x % n_mt_item;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);

  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kBwdKStages; ++s) { mbar_init(&sm.k_full[s], (s & 1) ? 2 : 1); mbar_init(&sm.k_empty[s], 1); }   // (two V producers)
    mbar_init(&sm.sdp_full, 1); mbar_init(&sm.pds_full, 256);
    mbar_init(&sm.dkv_full, 1); mbar_init(&sm.dkv_free, 128);
    mbar_init(&sm.s_full[0], 1); mbar_init(&sm.s_full[1], 1);
    // (two barriers each, used alternately: S(u+1) and dP(u+1) are issued before the MMA warp waits for the row
    // threads' arrivals of pair u, so the row threads may finish pair u+1 -- and arrive again -- before that wait
    // has observed pair u; with one barrier its phase would then be missed.  Pair u+2 cannot start before.)
    for (int s = 0; s < 2; ++s) { mbar_init(&sm.ds_full[s], 256); mbar_init(&sm.s_read[s], 256); }
    for (int s = 0; s < 4; ++s) mbar_init(&sm.dp_full[s], 1);
    mbar_init(&sm.phase_a_done, 1);
    for (int s = 0; s < kBwdKStages / 2; ++s) mbar_init(&sm.kp_full[s], 1);
    for (int s = 0; s < kBwdKStages; ++s) mbar_init(&sm.kp_empty[s], 1);
    mbar_init(&sm.vp_full[0], 2); mbar_init(&sm.vp_full[1], 2);
    mbar_init(&sm.dq_done, 1); mbar_init(&sm.dq_staged, 256);
    sm.abort = 0;
    fence_barrier_init();
  }
  if (warp < 8) {
    // Q and dO do not depend on the routing: their copies start first, one box per warp (issuing a box
    // costs its warp a few hundred cycles; eight warps issue in parallel).  Barrier 2 makes the mbarrier
    // initialisation above visible to the eight issuing warps.
    asm volatile("bar.sync 2, 256;" ::: "memory");
    if (lane == 0) {
      if (warp == 0) mbar_arrive_expect_tx(&sm.q_full, 2 * 128 * kBwdD * 2);
      // four boxes of 64 rows x one 64-element panel per tensor, laid out [panel][128 rows][128 B]
      const int half = warp & 1, panel = (warp >> 1) & 1;
      const int r = mt * 128 + 64 * half;
      const int a = r / dm.Bq, t = r % dm.Bq;
      const uint32_t off = (uint32_t)panel * 16384 + (uint32_t)half * 8192;
      if (warp < 4) tma_load_5d(sm.q + off, &map_q, &sm.q_full, 0, qb * dm.Bq + t, panel, h * dm.G + a, b);
      else tma_load_5d(sm.dO + off, &map_do, &sm.q_full, 0, qb * dm.Bq + t, panel, h * dm.G + a, b);
    }
    __syncwarp();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
    // with bf16 outputs the conversion kernel follows this grid: let its launch overlap this grid's tail
    if (lane == 0 && (dm.flags & HGA_FLAG_BWD_BF16_GRADS)) pdl_launch_dependents();
  }
  if (warp == 0) {
    if (lane == 0) { prefetch_tensormap(&map_k); prefetch_tensormap(&map_v); }
    bool bad;   // invalid entries are skipped exactly as in the forward kernel (which reports them)
    const int n_oct = build_octet_table(dm, w, group_idx + (int64_t)item * dm.width, n_groups + item, sm.oct_row, &bad);
    // Keys that receive dK/dV from this kernel: positions in [H, hi), where hi is the start of the
    // local band (the key-major band kernel has written that part).
    // Rows ascend, so these octets are a contiguous range [oa, ob) of the list.
    const int hi = w.ls;
    int below_h = 0, below_hi = 0;
    for (int o = lane; o < n_oct; o += 32) {
      const int row = sm.oct_row[o];
      below_h += row + 8 <= dm.H;
      below_hi += row < hi;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      below_h += __shfl_xor_sync(0xffffffffu, below_h, off);
      below_hi += __shfl_xor_sync(0xffffffffu, below_hi, off);
    }
    if (lane == 0) {
      sm.n_oct = n_oct;
      const int oa = below_h, ob = below_hi;
      sm.dkv_lo = oa / 8;
      sm.n_dkv = ob > oa ? (ob + 7) / 8 - oa / 8 : 0;
    }
  }
  // Row threads: LSE of the thread's own row, and the half of its O row (64 elements: warpgroup 0 the
  // first half, warpgroup 1 the second) that its share of delta = rowsum(dO o O) needs.  Requested here
  // so the latency hides behind the set-up.
  float row_lse = 0.f;
  uint4 o_half[8];
  if (warp >= 2 && warp < 10) {
    const int r = mt * 128 + (warp & 3) * 32 + lane;
    const int hq = h * dm.G + r / dm.Bq, srow = qb * dm.Bq + r % dm.Bq;
    row_lse = LSE[((int64_t)b * dm.Hq + hq) * dm.S + srow];
    const uint4* op = reinterpret_cast<const uint4*>(O + b * dm.os[0] + hq * dm.os[1] + (int64_t)srow * dm.os[2]) +
                      8 * ((warp - 2) >> 2);
#pragma unroll
    for (int i = 0; i < 8; ++i) o_half[i] = __ldg(op + i);
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tmem = sm.tmem_base;
  const int n_oct = sm.n_oct;
  const int n_keys = n_oct * 8;
  const int n_tiles = (n_oct + 7) / 8;
  const int n_act = sm.n_dkv;                       // steps 0 .. n_act-1 are dK/dV steps
  const int dkv_hi = sm.dkv_lo + n_act;
  const int n_pairs = (n_tiles - n_act + 1) / 2;    // paired steps; the last may hold one tile only
  // Ring slots: dK/dV step s takes TWO slots of the K ring, 2s for its K tile and 2s+1 for its V tile, so that
  // the V ring proper stays free and the first V pair of the paired steps is copied while the dK/dV steps
  // still run; the paired steps continue the slot numbering (a pair of stages is one contiguous operand).
  const int n_act_even = 2 * n_act;
  const int red_hi = w.ls;
  // Step order: the dK/dV tiles first (descending), so their atomics drain while the rest is
  // computed; then every other tile, descending.
  auto tile_of_step = [&](int s) {
    if (s < n_act) return dkv_hi - 1 - s;
    const int j = n_tiles - 1 - (s - n_act);
    return j >= dkv_hi ? j : j - n_act;
  };
  volatile int* abort = &sm.abort;
  HGA_TRACE_POINT(1);

  if (warp == 0 || warp >= 14) {
    // ------------------------------------------------------------------ producers
    // K and V advance independently (a V tile is released long before the K tile of the same step):
    // warp 0 copies the K tiles (eight octet boxes, one per lane) and runs several steps ahead; warps 14
    // and 15 copy the V tiles (four boxes each); in the paired steps their short ring is refilled only
    // after the dP GEMM of the pair before the previous one, so their issue time is on the critical path.  Issuing a box costs the issuing warp on the order of a hundred cycles;
    // different warps issue in parallel.
    const bool is_v = warp != 0;
    const CUtensorMap* map = is_v ? &map_v : &map_k;
    bool ok = true;
    // ---- slots of the dK/dV steps: one tile per slot, one full/empty barrier pair per stage
    {
      const int oct_in_tile = is_v ? (warp == 14 ? lane : 4 + lane) : lane;
      const bool copy_lane = is_v ? lane < 4 : lane < 8;
      const uint32_t my_bytes = (uint32_t)(is_v ? 4 : 8) * kOct;
      for (int step = 0; step < n_act && ok; ++step) {
        const int slot = 2 * step + (is_v ? 1 : 0);
        const int st = slot % kBwdKStages;
        int row = dm.L;                                      // past the list: zeros
        const int o = 8 * tile_of_step(step) + oct_in_tile;
        if (o < n_oct) row = sm.oct_row[o];
        if (lane == 0 && slot >= kBwdKStages) ok = bwd_wait(&sm.k_empty[st], (uint32_t)(slot / kBwdKStages - 1) & 1, abort);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(&sm.k_full[st], my_bytes);
        __syncwarp();
        if (copy_lane) tma_load_5d(sm.k[st] + oct_in_tile * kOct, map, &sm.k_full[st], 0, row, 0, h, b);
        HGA_TRACE_POINT(2);
      }
    }
    // ---- paired steps: pair p fills stages 2*ps, 2*ps+1 (ps continues the slot numbering) and
    // completes ONE barrier per operand, so the MMA thread observes one barrier per operand and
    // pair.  Lanes 0-7 (K) / 0-3 (V): first tile, lanes 8-15 / 4-7: second tile.
    {
      const int n_ps = kBwdKStages / 2;
      const int which = is_v ? lane >> 2 : lane >> 3;                     // tile of the pair
      const int oct_in_tile = is_v ? (warp == 14 ? 0 : 4) + (lane & 3) : lane & 7;
      const bool copy_lane = is_v ? lane < 8 : lane < 16;
      for (int p = 0; p < n_pairs && ok; ++p) {
        // K: three pairs of stages, continuing the slot numbering.  V: two pairs, pair p in slot p & 1; slot 0
        // is the V ring, slot 1 the P and dS tiles (adjacent, one K/V tile each), which only the dK/dV steps
        // use otherwise.  A V pair is free once its dP GEMM is done, a K pair only after its dQ GEMM.
        const int ps = is_v ? (p & 1) : (n_act_even / 2 + p) % n_ps;
        uint64_t* full = is_v ? &sm.vp_full[ps] : &sm.kp_full[ps];
        const int s = n_act + 2 * p + which;                              // step (tile order)
        int row = dm.L;
        if (s < n_tiles) {
          const int o = 8 * tile_of_step(s) + oct_in_tile;
          if (o < n_oct) row = sm.oct_row[o];
        }
        if (lane == 0) {
          if (is_v) {
            // first pair: the V ring is free from the start; second: the dK/dV steps (which use the P and dS
            // tiles) must be over; later: dP of pair p-2 is done
            if (p < 2) { if (p == 1 && n_act > 0) ok = bwd_wait(&sm.phase_a_done, 0, abort); }
            else ok = bwd_wait(&sm.dp_full[(p - 2) & 3], (uint32_t)((p - 2) >> 2) & 1, abort);
          } else if (p < n_ps) {
            // first paired use of these stages: if a dK/dV step used them, those steps must be over
            if (2 * ps < n_act_even) ok = bwd_wait(&sm.phase_a_done, 0, abort);
          } else {
            ok = bwd_wait(&sm.kp_empty[(n_act_even / 2 + p - 3) % kBwdKStages], (uint32_t)((p - 3) / kBwdKStages) & 1, abort);   // dQ of pair p-3 is done
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(full, (uint32_t)(is_v ? 8 : 16) * kOct);
        __syncwarp();
        if (copy_lane)
          tma_load_5d((is_v ? (ps == 0 ? sm.v[0] : sm.p) + which * kKvTile : sm.k[2 * ps + which]) + oct_in_tile * kOct, map, full,
                      0, row, 0, h, b);
        HGA_TRACE_POINT(2);
      }
    }
    if (*abort && lane == 0) {
      // giving up: give the copies still in flight time to land before shared memory is released
      // (the full barriers may never complete once another role has stopped, hence a bounded sleep)
      if (warp == 0) mbar_wait(&sm.q_full, 0);
      for (int it = 0; it < 64; ++it) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs this branch converged (waits included) and one elected lane issues: see mma_ss_w.
    {
      auto mma_wait = [&](uint64_t* bar, uint32_t parity, volatile int* ab) {
        return __all_sync(0xffffffffu, bwd_wait(bar, parity, ab));
      };
      constexpr uint32_t idesc_sdp = idesc_bf16_f32(128, kKT, 0, 0);       // rows x 64 keys, both K-major
      constexpr uint32_t idesc_sdp2 = idesc_bf16_f32(128, 2 * kKT, 0, 0);  // rows x 128 keys
      constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, 0, 1);          // dS K-major, K tile MN-major
      constexpr uint32_t idesc_dkv = idesc_bf16_f32(D, kKT, 1, 1);         // both MN-major
      // Descriptors are built once; inside the loops an MMA costs two integer adds.
      // Q, dO: [panel][128 rows][128 B] (8-row groups 1024 B apart, panels 16 KB apart)
      const uint64_t q_k = smem_desc_sw128(smem_u32(sm.q), 16, 1024);        // Q  as K-major A   (S)
      const uint64_t do_k = smem_desc_sw128(smem_u32(sm.dO), 16, 1024);      // dO as K-major A   (dP)
      const uint64_t q_mn = smem_desc_sw128(smem_u32(sm.q), 16384, 1024);    // Q^T  as MN-major A (dK^T)
      const uint64_t do_mn = smem_desc_sw128(smem_u32(sm.dO), 16384, 1024);  // dO^T as MN-major A (dV^T)
      const uint64_t k_k0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, kOct);    // K tile(s), K-major B  (S)
      const uint64_t v_k0 = smem_desc_sw128(smem_u32(sm.v[0]), 16, kOct);    // V tile(s), K-major B  (dP)
      const uint64_t v_k1 = smem_desc_sw128(smem_u32(sm.p), 16, kOct);       // second V pair of the paired steps (P, dS tiles)
      const uint64_t k_mn0 = smem_desc_sw128(smem_u32(sm.k[0]), 1024, kOct); // K tile(s), MN-major B (dQ)
      const uint64_t dsd = smem_desc_sw128(smem_u32(sm.ds), 16, 1024);       // dS: K-major A (dQ) and MN-major B (dK^T)
      const uint64_t pd = smem_desc_sw128(smem_u32(sm.p), 16, 1024);         // P : MN-major B (dV^T)
      // (arguments are ring slots)
      auto wait_k = [&](int s) { return mma_wait(&sm.k_full[s % kBwdKStages], (s / kBwdKStages) & 1, abort); };
      // acc (128 rows x N keys) = a (Q or dO, K-major) x b^T (key tiles at ring stage st, K-major)
      auto issue_qk = [&](uint32_t acc, uint64_t a, uint64_t b0, int st, uint32_t idesc) {   // st: ring stage
        const uint64_t bd = desc_advance(b0, (uint32_t)st * kKvTile);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t a_off = (kk >> 2) * 16384 + (kk & 3) * 32, b_off = (kk >> 2) * 1024 + (kk & 3) * 32;
          mma_ss_w(acc, desc_advance(a, a_off), desc_advance(bd, b_off), idesc, kk > 0);
        }
      };
      bool ok = mma_wait(&sm.q_full, 0, abort);
      HGA_TRACE_POINT(40);
      bool dq_started = false;
      // ---- dK/dV steps: one at a time, every operand from shared memory.  The tensor pipe runs in
      // issue order and a commit covers everything issued before it, so sdp_full of step s+1 also
      // tells the row threads that the GEMMs reading P/dS of step s are done.
      for (int s = 0; s < n_act && ok; ++s) {
        const int st = (2 * s) % kBwdKStages, vst = (2 * s + 1) % kBwdKStages;      // K tile, V tile
        ok = wait_k(2 * s);
        HGA_TRACE_POINT(41);
        ok = ok && wait_k(2 * s + 1);
        HGA_TRACE_POINT(42);
        if (!ok) break;
        tc_fence_after_sync();
        issue_qk(tmem + region(0), q_k, k_k0, st, idesc_sdp);
        issue_qk(tmem + region(0) + 64, do_k, k_k0, vst, idesc_sdp);
        mma_commit_w(&sm.sdp_full);
        mma_commit_w(&sm.k_empty[vst]);
        HGA_TRACE_POINT(44);
        ok = mma_wait(&sm.pds_full, s & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        HGA_TRACE_POINT(45);
        const uint64_t kmn = desc_advance(k_mn0, (uint32_t)st * kKvTile);
#pragma unroll
        for (int kk = 0; kk < kKT / 16; ++kk)   // dQ += dS K : 16 keys per MMA
          mma_ss_w(tmem + kColDQ, desc_advance(dsd, kk * 32), desc_advance(kmn, kk * 2 * kOct), idesc_dq,
                 (dq_started || kk > 0));
        dq_started = true;
        if (s > 0) {
          ok = mma_wait(&sm.dkv_free, (s - 1) & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
        }
#pragma unroll
        for (int kk = 0; kk < 128 / 16; ++kk)    // 16 query rows per MMA (2 row octets)
          mma_ss_w(tmem + kColDV, desc_advance(do_mn, kk * 2048), desc_advance(pd, kk * 2048), idesc_dkv, kk > 0);
#pragma unroll
        for (int kk = 0; kk < 128 / 16; ++kk)
          mma_ss_w(tmem + kColDK, desc_advance(q_mn, kk * 2048), desc_advance(dsd, kk * 2048), idesc_dkv, kk > 0);
        mma_commit_w(&sm.dkv_full);
        mma_commit_w(&sm.k_empty[st]);
        HGA_TRACE_POINT(4);
      }
      // ---- paired steps.  Step u covers ring stages st, st+1 (contiguous); S(u) lives in region
      // (2u)%3, dP(u) and later dS(u) in region (2u+1)%3.
      if (ok && n_pairs > 0) {
        if (ok && n_act_even > 0) mma_commit_w(&sm.phase_a_done);
        const int ps0 = (n_act_even / 2) % (kBwdKStages / 2);
        if (ok) ok = mma_wait(&sm.kp_full[ps0], 0, abort);
        HGA_TRACE_POINT(43);
        if (ok) {
          tc_fence_after_sync();
          issue_qk(tmem + region(0), q_k, k_k0, 2 * ps0, idesc_sdp2);
          mma_commit_w(&sm.s_full[0]);
        }
        if (ok) ok = mma_wait(&sm.vp_full[0], 0, abort);
        if (ok) {
          tc_fence_after_sync();
          issue_qk(tmem + region(1), do_k, v_k0, 0, idesc_sdp2);
          mma_commit_w(&sm.dp_full[0]);    // also tells the V producers that the V pair is free
        }
        HGA_TRACE_POINT(3);
      }
      int rs = 0;                                     // region of S(u)
      for (int u = 0; u < n_pairs && ok; ++u) {
        constexpr int kPs = kBwdKStages / 2;
        const int ps = (n_act_even / 2 + u) % kPs, ps_n = (ps + 1) % kPs;     // pair stages of steps u, u+1
        const int rp = rs == 2 ? 0 : rs + 1;          // region of dP(u), dS(u)
        const int rs_n = rp == 2 ? 0 : rp + 1;        // region of S(u+1): two steps ago it held dP(u-1)
        if (u + 1 < n_pairs) {
          ok = mma_wait(&sm.kp_full[ps_n], (uint32_t)((u + 1) / kPs) & 1, abort);
          // S(1) is the first to use the region that aliases the dK^T/dV^T accumulators: the
          // reduction warps must have read the last ones
          if (ok && u == 0 && n_act > 0) ok = mma_wait(&sm.dkv_free, (n_act - 1) & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
          issue_qk(tmem + region(rs_n), q_k, k_k0, 2 * ps_n, idesc_sdp2);
          mma_commit_w(&sm.s_full[(u + 1) & 1]);
          HGA_TRACE_POINT(6);
          // dP(u+1) goes into the region of S(u) as soon as the row threads have read S(u) (they keep P in
          // registers): it is then complete long before they finish dS(u) and P(u+1) and ask for it
          ok = mma_wait(&sm.s_read[u & 1], (uint32_t)(u >> 1) & 1, abort) &&
               mma_wait(&sm.vp_full[(u + 1) & 1], (uint32_t)((u + 1) >> 1) & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
          issue_qk(tmem + region(rs), do_k, ((u + 1) & 1) ? v_k1 : v_k0, 0, idesc_sdp2);
          mma_commit_w(&sm.dp_full[(u + 1) & 3]);
          HGA_TRACE_POINT(8);
        }
        ok = mma_wait(&sm.ds_full[u & 1], (uint32_t)(u >> 1) & 1, abort);     // the row threads are done with dP(u): dS(u) is in its place
        if (!ok) break;
        tc_fence_after_sync();
        HGA_TRACE_POINT(5);
        // dQ += dS K over 128 keys: bf16 dS from TMEM (first tile at columns 0-31 of its region,
        // second tile at 64-95), the two K stages as one MN-major B operand
        const uint64_t kmn = desc_advance(k_mn0, (uint32_t)(2 * ps) * kKvTile);
        const uint32_t ds_base = tmem + region(rp);
#pragma unroll
        for (int kk = 0; kk < 2 * kKT / 16; ++kk)
          mma_ts_w(tmem + kColDQ, ds_base + (kk < 4 ? 8 * kk : 64 + 8 * (kk - 4)), desc_advance(kmn, kk * 2 * kOct),
                 idesc_dq, (dq_started || kk > 0));
        dq_started = true;
        mma_commit_w(&sm.kp_empty[(n_act_even / 2 + u) % kBwdKStages]);
        HGA_TRACE_POINT(7);
        rs = rs_n;
      }
      if (ok) mma_commit_w(&sm.dq_done);
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------------ one thread per query row
    const int wg = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const int t = (mt * 128 + row_in_tile) % dm.Bq;         // position of the row inside its query block
    const int limit = n_keys - dm.Bq + t + 1;
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    const float sl2 = dm.scale * 1.4426950408889634f;
    const float neg_lse2 = -row_lse * 1.4426950408889634f;
    // delta: this warpgroup's 64-element half of the row's dot product (dO from the tile in shared memory:
    // panel wg, 128-byte line of the row, 16-byte chunks XOR-swizzled), then the sum of the two halves
    bool ok = __all_sync(0xffffffffu, bwd_wait(&sm.q_full, 0, abort));
    {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      if (ok) {
        const uint32_t line = smem_u32(sm.dO) + (uint32_t)wg * 16384 + (uint32_t)row_in_tile * 128;
        const uint32_t key7 = (uint32_t)(row_in_tile & 7);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          uint32_t y0, y1, y2, y3;
          ld_shared_v4(line + (((uint32_t)i ^ key7) * 16), y0, y1, y2, y3);
          const uint32_t xs[4] = {o_half[i].x, o_half[i].y, o_half[i].z, o_half[i].w}, ys[4] = {y0, y1, y2, y3};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            acc[e] = fmaf(__uint_as_float(xs[e] << 16), __uint_as_float(ys[e] << 16), acc[e]);
            acc[e] = fmaf(__uint_as_float(xs[e] & 0xffff0000u), __uint_as_float(ys[e] & 0xffff0000u), acc[e]);
          }
        }
      }
      // the two halves meet in tensor memory: columns 0 and 1 of the dQ accumulator, which no GEMM writes
      // before the first dS exists (every shared-memory buffer may already be receiving copies)
      tmem_st1(lane_base + kColDQ + wg, __float_as_uint((acc[0] + acc[1]) + (acc[2] + acc[3])));
      tmem_wait_st();
    }
    tc_fence_before_sync();
    asm volatile("bar.sync 3, 256;" ::: "memory");           // the 256 row threads (reached on every path)
    tc_fence_after_sync();
    uint32_t d_lo, d_hi;
    tmem_ld2(lane_base + kColDQ, d_lo, d_hi);
    tmem_wait_ld();
    // (the first dQ GEMM must not overwrite these two columns before every row thread has read them)
    tc_fence_before_sync();
    asm volatile("bar.sync 3, 256;" ::: "memory");
    const float neg_delta_s = -(__uint_as_float(d_lo) + __uint_as_float(d_hi)) * dm.scale;
    HGA_TRACE_POINT(10);
    {
      // ---- dK/dV steps: P and dS go to shared memory as operands of dV^T / dK^T / dQ; warpgroup wg takes
      // keys 32*wg .. 32*wg+31 of the tile.
      // this row's 128-byte line inside the P / dS buffers, and its swizzle key
      const uint32_t line = (uint32_t)(row_in_tile >> 3) * 1024 + (uint32_t)(row_in_tile & 7) * 128;
      const uint32_t key = (uint32_t)(row_in_tile & 7);
      const uint32_t p_line = smem_u32(sm.p) + line, ds_line = smem_u32(sm.ds) + line;
      const uint32_t sdp_addr = lane_base + region(0);
      for (int s = 0; s < n_act && ok; ++s) {
        ok = __all_sync(0xffffffffu, bwd_wait(&sm.sdp_full, s & 1, abort));
        if (!ok) break;
        tc_fence_after_sync();
        HGA_TRACE_POINT(12);
        const int vis = limit - kKT * tile_of_step(s);
#pragma unroll
        for (int q4 = 2 * wg; q4 < 2 * wg + 2; ++q4) {   // 16 columns (keys) at a time
          uint32_t sv[16], dp[16];
          tmem_ld16(sdp_addr + q4 * 16, sv);
          tmem_ld16(sdp_addr + 64 + q4 * 16, dp);
          tmem_wait_ld();
          uint32_t pk[8], dk[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float p0 = fast_exp2(fmaf(__uint_as_float(sv[2 * i]), sl2, neg_lse2));
            float p1 = fast_exp2(fmaf(__uint_as_float(sv[2 * i + 1]), sl2, neg_lse2));
            if (vis < kKT) {                  // diagonal / ragged tile only
              if (q4 * 16 + 2 * i >= vis) p0 = 0.f;
              if (q4 * 16 + 2 * i + 1 >= vis) p1 = 0.f;
            }
            const float d0 = p0 * fmaf(__uint_as_float(dp[2 * i]), dm.scale, neg_delta_s);
            const float d1 = p1 * fmaf(__uint_as_float(dp[2 * i + 1]), dm.scale, neg_delta_s);
            pk[i] = pack_bf16(p0, p1);
            dk[i] = pack_bf16(d0, d1);
          }
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {    // two 16-byte chunks (8 keys each), XOR-swizzled
            const uint32_t off = ((uint32_t)(2 * q4 + cc) ^ key) * 16;
            st_shared_v4(p_line + off, pk[4 * cc], pk[4 * cc + 1], pk[4 * cc + 2], pk[4 * cc + 3]);
            st_shared_v4(ds_line + off, dk[4 * cc], dk[4 * cc + 1], dk[4 * cc + 2], dk[4 * cc + 3]);
          }
        }
        tc_fence_before_sync();
        fence_proxy_async_smem();
        mbar_arrive(&sm.pds_full);
        HGA_TRACE_POINT(17);
      }
    }
    // ---- paired steps: warpgroup wg owns the wg-th tile of each pair (64 of the 128 columns)
    const uint64_t sl2_2 = pack_f32x2(sl2, sl2), neg_lse2_2 = pack_f32x2(neg_lse2, neg_lse2);
    const uint64_t scale_2 = pack_f32x2(dm.scale, dm.scale), neg_delta_s_2 = pack_f32x2(neg_delta_s, neg_delta_s);
    int rs = 0;
    for (int u = 0; u < n_pairs && ok; ++u) {
      const int rp = rs == 2 ? 0 : rs + 1;
      const int s = n_act + 2 * u + wg;
      const int vis = s < n_tiles ? limit - kKT * tile_of_step(s) : 0;     // a missing tile is fully masked
      const uint32_t s_addr = lane_base + region(rs) + wg * 64;
      const uint32_t dp_addr = lane_base + region(rp) + wg * 64;
      uint32_t pk[32];                                // P of this row, 64 keys, packed bf16
      ok = __all_sync(0xffffffffu, bwd_wait(&sm.s_full[u & 1], (u >> 1) & 1, abort));
      if (!ok) break;
      tc_fence_after_sync();
      HGA_TRACE_POINT(11);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t sv[16];
        tmem_ld16(s_addr + q4 * 16, sv);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float a0, a1;            // packed fp32 pairs: one FMA for the two exponent arguments
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1])), sl2_2, neg_lse2_2), a0, a1);
          float p0 = fast_exp2(a0), p1 = fast_exp2(a1);
          if (vis < kKT) {
            if (q4 * 16 + 2 * i >= vis) p0 = 0.f;
            if (q4 * 16 + 2 * i + 1 >= vis) p1 = 0.f;
          }
          pk[8 * q4 + i] = pack_bf16(p0, p1);
        }
      }
      tc_fence_before_sync();
      mbar_arrive(&sm.s_read[u & 1]);                 // S(u) has been read: its region may take dP(u+1)
      ok = __all_sync(0xffffffffu, bwd_wait(&sm.dp_full[u & 3], (u >> 2) & 1, abort));
      if (!ok) break;
      tc_fence_after_sync();
      HGA_TRACE_POINT(13);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t dp[16], dk[8];
        tmem_ld16(dp_addr + q4 * 16, dp);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint64_t p2 = pack_f32x2(__uint_as_float(pk[8 * q4 + i] << 16), __uint_as_float(pk[8 * q4 + i] & 0xffff0000u));
          const uint64_t g2 = fma_f32x2(pack_f32x2(__uint_as_float(dp[2 * i]), __uint_as_float(dp[2 * i + 1])), scale_2, neg_delta_s_2);
          float d0, d1;
          unpack_f32x2(mul_f32x2(p2, g2), d0, d1);
          dk[i] = pack_bf16(d0, d1);
        }
        // bf16 dS over the dP columns already read (8 columns per 16 keys): the A operand of dQ
        tmem_st8(dp_addr + q4 * 8, dk);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(&sm.ds_full[u & 1]);
      HGA_TRACE_POINT(14);
      rs = rp == 2 ? 0 : rp + 1;
    }
    if (ok) ok = __all_sync(0xffffffffu, bwd_wait(&sm.dq_done, 0, abort));
    HGA_TRACE_POINT(20);
    if (ok) {
      // dQ epilogue through shared memory and TMA: a thread's own row is 256 bytes away from its
      // neighbour's, so direct 16-byte stores would touch 32 different sectors per instruction.
      // Warpgroup wg holds columns 64*wg .. 64*wg+63 of its rows = panel wg of the Q-shaped tile,
      // which goes into Q's shared memory (all GEMMs that read it are complete) in the swizzled
      // [panel][128 rows][128 B] layout and leaves as four boxes.
      tc_fence_after_sync();
      uint32_t x[2][32];
      tmem_ld32(lane_base + kColDQ + wg * 64, x[0]);
      tmem_ld32(lane_base + kColDQ + wg * 64 + 32, x[1]);
      tmem_wait_ld();
      const uint32_t key = (uint32_t)(row_in_tile & 7);
      const uint32_t line = smem_u32(sm.q) + (uint32_t)wg * 16384 + (uint32_t)row_in_tile * 128;
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int i = 0; i < 4; ++i)
          st_shared_v4(line + (((uint32_t)(4 * c + i) ^ key) * 16),
                       pack_bf16(__uint_as_float(x[c][8 * i]), __uint_as_float(x[c][8 * i + 1])),
                       pack_bf16(__uint_as_float(x[c][8 * i + 2]), __uint_as_float(x[c][8 * i + 3])),
                       pack_bf16(__uint_as_float(x[c][8 * i + 4]), __uint_as_float(x[c][8 * i + 5])),
                       pack_bf16(__uint_as_float(x[c][8 * i + 6]), __uint_as_float(x[c][8 * i + 7])));
      fence_proxy_async_smem();
      mbar_arrive(&sm.dq_staged);
      if (warp == 2 && lane < 4 && bwd_wait(&sm.dq_staged, 0, abort)) {      // all 256 rows are in shared memory
        const int half = lane & 1, panel = lane >> 1;
        const int r0 = mt * 128 + 64 * half;
        tma_store_5d(&map_dq, sm.q + panel * 16384 + half * 8192, 0, qb * dm.Bq + r0 % dm.Bq, panel,
                     h * dm.G + r0 / dm.Bq, b);
        tma_store_commit();
        tma_store_wait_read();      // (the source tile has been read; the writes complete before the grid does)
      }
    }
  } else {
    // ------------------------------------------------------------------ dK / dV reduction
    const int quarter = warp & 3;
    const int e = quarter * 32 + lane;                       // head_dim element = TMEM lane
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    float* dKb = dK + ((int64_t)(b * dm.Hkv + h) * dm.S) * D + e;
    float* dVb = dV + ((int64_t)(b * dm.Hkv + h) * dm.S) * D + e;
    bool ok = true;
    // The band kernel, which precedes this one in the stream, stores its dK/dV rows plainly: the adds
    // below must come after it.  Nothing else in this kernel depends on it, so this is the only wait
    // (a no-op unless the launch carried the programmatic-serialization attribute).
    if (n_act > 0) pdl_wait();
    for (int s = 0; s < n_act; ++s) {
      const int j = tile_of_step(s);
      ok = __all_sync(0xffffffffu, bwd_wait(&sm.dkv_full, s & 1, abort));
      if (!ok) break;
      tc_fence_after_sync();
      HGA_TRACE_POINT(16);
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t gv[32], gk[32];
        tmem_ld32(lane_base + kColDV + half * 32, gv);
        tmem_ld32(lane_base + kColDK + half * 32, gk);
        tmem_wait_ld();
        if (half == 1) {
          tc_fence_before_sync();
          mbar_arrive(&sm.dkv_free);
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int o = 8 * j + half * 4 + (i >> 3);
          if (o < n_oct) {
            const int pos = sm.oct_row[o] + (i & 7);
            if (pos >= dm.H && pos < red_hi) {   // warp-uniform: a key this kernel owes dK/dV
              atomicAdd(dVb + (int64_t)(pos - dm.H) * D, __uint_as_float(gv[i]));
              atomicAdd(dKb + (int64_t)(pos - dm.H) * D, __uint_as_float(gk[i]));
            }
          }
        }
      }
      HGA_TRACE_POINT(18);
    }
  }
  HGA_TRACE_POINT(30);

  // Common exit.  The single-thread roles leave their warps diverged, so every warp reconverges
  // first: a block barrier reached by part of a warp would count that warp as arrived.
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  HGA_TRACE_POINT(31);
  HGA_TRACE_DUMP;
  if (tid == 0 && sm.abort && status_word) atomicOr(status_word, HGA_ABORT_CODE(3, sm.abort));
  if (warp == 1) tmem_dealloc(tmem, 512);
}

bool attn_bwd_sm100_supported(const Dims& dm) {
  if (dm.flags & HGA_FLAG_GENERIC_KERNELS) return false;
  return dm.d == 128 && dm.rows % 128 == 0 && dm.g % 8 == 0 && dm.Bq % 64 == 0;
}

int launch_attn_bwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const void* O,
                          const float* LSE, const void* dO, const int32_t* group_idx,
                          const int32_t* n_groups, void* dQ, float* dK, float* dV, int32_t* status_word,
                          cudaStream_t st) {
  if (!attn_bwd_band_sm100_supported(dm)) return HGA_ERR_UNSUPPORTED;
  CUtensorMap mq, mdo, mk, mv, mdq;
  const uint32_t box[5] = {64, 8, 2, 1, 1};
  const uint32_t box_q[5] = {64, 64, 1, 1, 1};
  const uint64_t dq[5] = {64, (uint64_t)dm.S, 2, (uint64_t)dm.Hq, (uint64_t)dm.B};
  const uint64_t dk[5] = {64, (uint64_t)dm.L, 2, (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t sq[4] = {(uint64_t)dm.qs[2] * 2, 128, (uint64_t)dm.qs[1] * 2, (uint64_t)dm.qs[0] * 2};
  const uint64_t so[4] = {(uint64_t)dm.os[2] * 2, 128, (uint64_t)dm.os[1] * 2, (uint64_t)dm.os[0] * 2};
  const uint64_t sk[4] = {(uint64_t)dm.ks[2] * 2, 128, (uint64_t)dm.ks[1] * 2, (uint64_t)dm.ks[0] * 2};
  const uint64_t sv[4] = {(uint64_t)dm.vs[2] * 2, 128, (uint64_t)dm.vs[1] * 2, (uint64_t)dm.vs[0] * 2};
  if (encode_tensor_map_bf16(&mq, Q, 5, dq, sq, box_q, true) ||
      encode_tensor_map_bf16(&mdo, dO, 5, dq, so, box_q, true) ||
      encode_tensor_map_bf16(&mdq, dQ, 5, dq, sq, box_q, true) ||
      encode_tensor_map_bf16(&mk, K, 5, dk, sk, box, true) ||
      encode_tensor_map_bf16(&mv, V, 5, dk, sv, box, true))
    return HGA_ERR_UNSUPPORTED;
  // the octet table starts inside the struct's tail padding; 1024 bytes of slack for the manual alignment
  const size_t smem = offsetof(BwdSmem, oct_row) + sizeof(int) * (max_routed_tokens(dm) / 8 + 8) + 1024;
  if (smem > 227 * 1024) return HGA_ERR_UNSUPPORTED;
  int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(&k_attn_bwd_sm100), smem);
  if (rc) return rc;
  cudaError_t e;
  // dK/dV of the local band: written once per key tile by the key-major kernel, with plain stores that
  // cover every row of the active segment (so nothing has to be zero-filled); this kernel then adds the
  // contributions of the keys before the band atomically.
  rc = launch_attn_bwd_band_sm100(dm, Q, K, V, O, LSE, dO, dK, dV, status_word, st);
  if (rc != HGA_OK) return rc;
  const int units = dm.B * dm.Hkv * dm.NQB * (dm.rows / 128);
  // The sweep is launched with programmatic serialization behind the band kernel: its CTAs may start on
  // SMs the band kernel leaves idle (they wait for it only before adding to dK/dV).
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)units);
  cfg.blockDim = dim3(kBwdThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = (dm.flags & kFlagNoPdl) ? 0 : 1;
  e = cudaLaunchKernelEx(&cfg, k_attn_bwd_sm100, mq, mdo, mk, mv, mdq, (const uint16_t*)O, LSE, group_idx, n_groups,
                         dm, dK, dV, status_word);
  count_launch(HGA_KERNELS_BWD_TENSOR);
  return record_cuda(e);
}

}  // namespace hga

#ifdef HGA_DEBUG_WAIT
extern "C" __attribute__((visibility("default"))) int hga_debug_dump(int* out64) {
  cudaMemcpyFromSymbol(out64, hga::g_dbg_fail, sizeof(int) * 64);
  int zero[64] = {0};
  cudaMemcpyToSymbol(hga::g_dbg_fail, zero, sizeof(zero));
  return 0;
}
#endif
