// hga_attn_bwd for sm_100a (head_dim 128): backward of routed exact-token attention with the
// routing frozen (Section 2.1, last paragraph) and history K/V detached (Section 2.2).
//
// Work unit (one CTA): one 128-row M-tile of one item, swept over the item's routed keys in
// 64-key tiles (8 octets, gathered by TMA exactly as in the forward kernel).  Per tile:
//   S  = Q K^T, dP = dO V^T   (smem x smem)  -> one of three S/dP buffers in TMEM
//   P  = 2^(S*c - LSE*log2e),  dS = scale * P o (dP - delta)            (one thread per row)
//   dQ += dS K                (dS as bf16 in TMEM over the S columns, K tile MN-major from smem)
// and, only for tiles holding keys whose dK/dV this kernel must add (keys of the active segment
// selected through routing; the local band is written by k_attn_bwd_band_sm100; without that
// kernel, every active key), P and dS also pass through shared memory for
//   dV^T = dO^T P,  dK^T = Q^T dS   (M = head_dim, N = 64 keys, K = 128 rows) -> TMEM.
// dK^T/dV^T are produced transposed so that a reduction warp's 32 lanes hold 32 consecutive
// elements of one key row: its red.global.add.f32 is one coalesced 128-byte request.
//
// The dK/dV tiles are processed first (their atomics drain while the rest is computed), then all
// other tiles in descending key order.
//
// Warp roles (512 threads): warps 0 and 14 producers (TMA), warp 1 issues S/dP, warp 15 issues
// dQ and dK^T/dV^T (two issuing threads, so neither hand-off stalls the other's GEMMs), warps 2-5
// and 6-9 two warpgroups of one thread per query row taking alternate tiles (P, dS, dQ epilogue),
// warps 10-13 dK/dV reduction (thread = head_dim lane).
// TMEM (512 columns): S/dP buffer 0 | buffer 1 (aliased by dV^T, dK^T while dK/dV tiles run) |
// dQ | buffer 2.  Shared memory: Q, dO (32 KB each), K ring (5 x 16 KB; a K tile is held until
// its dQ GEMM), V ring (3 x 16 KB; a V tile is free once dP is done), P and dS (16 KB each).
#include "hga_bwd_sm100.cuh"
#include "hga_common.cuh"
#include "hga_octets.cuh"
#include "hga_sm100.cuh"

#include <cstddef>

namespace hga {

using namespace sm100;

constexpr int kBwdThreads = 512;                // 16 warps: 128 registers per thread
constexpr int kBwdProducers = 2;                // warps 0 and 14 issue the K/V copies
constexpr int kBwdKStages = 5;                  // a K tile is held until its dQ GEMM is done
constexpr int kBwdVStages = 3;                  // a V tile is free once dP is done
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
  uint64_t q_full, k_full[kBwdKStages], k_empty[kBwdKStages], v_full[kBwdVStages], v_empty[kBwdVStages];
  uint64_t sdp_full[3], pds_full[3], buf_free[3], dkv_full, dkv_free, dq_done;
  uint32_t tmem_base;
  int n_oct, dkv_lo, n_dkv;    // tiles [dkv_lo, dkv_lo + n_dkv) hold keys whose dK/dV this kernel adds
  volatile int abort;
  int oct_row[1];
};

__device__ __forceinline__ float dot4_bf16(uint2 x, uint2 y) {
  float s = __uint_as_float(x.x << 16) * __uint_as_float(y.x << 16);
  s = fmaf(__uint_as_float(x.x & 0xffff0000u), __uint_as_float(y.x & 0xffff0000u), s);
  s = fmaf(__uint_as_float(x.y << 16), __uint_as_float(y.y << 16), s);
  s = fmaf(__uint_as_float(x.y & 0xffff0000u), __uint_as_float(y.y & 0xffff0000u), s);
  return s;
}

__global__ void __launch_bounds__(kBwdThreads, 1)
k_attn_bwd_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                 const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                 const float* __restrict__ delta_ws, const float* __restrict__ LSE, const int32_t* __restrict__ group_idx,
                 const int32_t* __restrict__ n_groups, Dims dm, uint16_t* __restrict__ dQ,
                 float* __restrict__ dK, float* __restrict__ dV, int band_done, int32_t* status_word) {
  constexpr int D = kBwdD;
  // three S/dP buffers of 128 columns (S at +0, dP at +64; bf16 dS later overwrites S): 0, 128, 384
  auto buf_col = [](uint32_t bf) -> uint32_t { return bf == 2 ? 384u : bf * 128u; };
  constexpr uint32_t kColDV = 128, kColDK = 192;   // alias buffer 1, which the dK/dV steps leave idle
  constexpr uint32_t kColDQ = 256;
  extern __shared__ uint8_t smem_raw[];
  BwdSmem& sm = *reinterpret_cast<BwdSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  HGA_TRACE_DECL;
  const int n_mt_item = dm.rows / 128;
  const int item = blockIdx.x / n_mt_item;
  const int mt = blockIdx.x % n_mt_item;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);

  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kBwdKStages; ++s) { mbar_init(&sm.k_full[s], kBwdProducers); mbar_init(&sm.k_empty[s], 1); }
    for (int s = 0; s < kBwdVStages; ++s) { mbar_init(&sm.v_full[s], kBwdProducers); mbar_init(&sm.v_empty[s], 1); }
    for (int s = 0; s < 3; ++s) {
      mbar_init(&sm.sdp_full[s], 1); mbar_init(&sm.buf_free[s], 1);
      mbar_init(&sm.pds_full[s], 128);
    }
    mbar_init(&sm.dkv_full, 1); mbar_init(&sm.dkv_free, 128);
    mbar_init(&sm.dq_done, 1);
    sm.abort = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  if (warp == 0) {
    // Q and dO do not depend on the routing: start their copies first
    if (lane == 0) {
      prefetch_tensormap(&map_q); prefetch_tensormap(&map_do);
      prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
      mbar_arrive_expect_tx(&sm.q_full, 2 * 128 * kBwdD * 2);
    }
    __syncwarp();
    {
      const int o = lane & 15;
      const int r = mt * 128 + 8 * o;
      const int a = r / dm.Bq, t = r % dm.Bq;
      if (lane < 16) tma_load_5d(sm.q + o * kOct, &map_q, &sm.q_full, 0, qb * dm.Bq + t, 0, h * dm.G + a, b);
      else tma_load_5d(sm.dO + o * kOct, &map_do, &sm.q_full, 0, qb * dm.Bq + t, 0, h * dm.G + a, b);
    }
    bool bad;   // invalid entries are skipped exactly as in the forward kernel (which reports them)
    const int n_oct = build_octet_table(dm, w, group_idx + (int64_t)item * dm.width, n_groups + item, sm.oct_row, &bad);
    // Keys that receive dK/dV from this kernel: positions in [H, hi), where hi is the start of the
    // local band when the key-major band kernel has already written that part, else no limit.
    // Rows ascend, so these octets are a contiguous range [oa, ob) of the list.
    const int hi = band_done ? w.ls : 0x7fffffff;
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
  // Row threads: LSE and delta = rowsum(dO o O) of the thread's own row (delta comes from a
  // coalesced pre-pass, k_bwd_delta_sm100).  Loaded here so the latency hides behind the set-up.
  float delta = 0.f, row_lse = 0.f;
  if (warp >= 2 && warp < 10) {
    const int r = mt * 128 + (warp & 3) * 32 + lane;
    const int64_t row = ((int64_t)b * dm.Hq + h * dm.G + r / dm.Bq) * dm.S + qb * dm.Bq + r % dm.Bq;
    delta = delta_ws[row];
    row_lse = LSE[row];
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tmem = sm.tmem_base;
  const int n_oct = sm.n_oct;
  const int n_keys = n_oct * 8;
  const int n_tiles = (n_oct + 7) / 8;
  const int n_active = sm.n_dkv;                    // steps 0 .. n_active-1 produce dK/dV
  const int dkv_hi = sm.dkv_lo + n_active;
  const int red_hi = band_done ? w.ls : 0x7fffffff;
  // Step order: the dK/dV tiles first (descending), so their atomics drain while the rest is
  // computed; then every other tile, descending.
  auto tile_of_step = [&](int s) {
    if (s < n_active) return dkv_hi - 1 - s;
    const int j = n_tiles - 1 - (s - n_active);
    return j >= dkv_hi ? j : j - n_active;
  };
  volatile int* abort = &sm.abort;
  HGA_TRACE_POINT(1);

  if (warp == 0 || warp == 14) {
    // ------------------------------------------------------------------ producers
    // Issuing one TMA box costs the issuing warp on the order of a hundred cycles, so the sixteen
    // octet boxes of a step are spread over two warps: producer p takes octets p, p+2, p+4, p+6 of
    // the K tile (lanes 0-3) and of the V tile (lanes 8-11).  Every producer arrives on the full
    // barriers with the byte count of its own boxes.
    const int pi = warp == 0 ? 0 : 1;
    const int sub = lane & 7;
    const int oct_in_tile = pi + kBwdProducers * sub;          // < 8 for the lanes that copy
    const bool k_lane = lane < 8 && oct_in_tile < 8, v_lane = lane >= 8 && lane < 16 && oct_in_tile < 8;
    const uint32_t my_bytes = (uint32_t)((8 - pi + kBwdProducers - 1) / kBwdProducers) * kOct;
    bool ok = true;
    int issued = 0;
    for (int s = 0; s < n_tiles; ++s) {
      const int j = tile_of_step(s);
      const int ks = s % kBwdKStages, vs = s % kBwdVStages;
      const int o = 8 * j + oct_in_tile;
      const int row = o < n_oct ? sm.oct_row[o] : dm.L;    // past the list: zeros
      if (lane == 0 && s >= kBwdKStages) ok = bwd_wait(&sm.k_empty[ks], (s / kBwdKStages - 1) & 1, abort);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      HGA_TRACE_POINT(21);
      if (lane == 0) mbar_arrive_expect_tx(&sm.k_full[ks], my_bytes);
      __syncwarp();
      if (k_lane) tma_load_5d(sm.k[ks] + oct_in_tile * kOct, &map_k, &sm.k_full[ks], 0, row, 0, h, b);
      HGA_TRACE_POINT(22);
      if (lane == 0 && s >= kBwdVStages) ok = bwd_wait(&sm.v_empty[vs], (s / kBwdVStages - 1) & 1, abort);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      HGA_TRACE_POINT(23);
      if (lane == 0) mbar_arrive_expect_tx(&sm.v_full[vs], my_bytes);
      __syncwarp();
      if (v_lane) tma_load_5d(sm.v[vs] + oct_in_tile * kOct, &map_v, &sm.v_full[vs], 0, row, 0, h, b);
      issued = s + 1;
      HGA_TRACE_POINT(2);
    }
    if (*abort && lane == 0) {
      // giving up: let the copies still in flight land before shared memory is released (bounded:
      // a full barrier also needs the other producers, which may have stopped earlier)
      if (pi == 0) mbar_wait(&sm.q_full, 0);
      for (int s = issued > kBwdKStages ? issued - kBwdKStages : 0; s < issued; ++s)
        mbar_wait(&sm.k_full[s % kBwdKStages], (s / kBwdKStages) & 1);
      for (int s = issued > kBwdVStages ? issued - kBwdVStages : 0; s < issued; ++s)
        mbar_wait(&sm.v_full[s % kBwdVStages], (s / kBwdVStages) & 1);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_sdp = idesc_bf16_f32(128, kKT, 0, 0);   // rows x keys, both K-major
      // Descriptors are built once; inside the loops an MMA costs two integer adds.
      const uint64_t q_k = smem_desc_sw128(smem_u32(sm.q), 16, kOct);        // Q  as K-major A   (S, dK/dV steps)
      const uint64_t do_k = smem_desc_sw128(smem_u32(sm.dO), 16, kOct);      // dO as K-major A   (dP, dK/dV steps)
      const uint64_t k_k0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, kOct);    // K tile, K-major B  (S)
      const uint64_t v_k0 = smem_desc_sw128(smem_u32(sm.v[0]), 16, kOct);    // V tile, K-major B  (dP)
      // Two threads feed the tensor pipe.  This one (warp 1) issues S and dP of every step and
      // runs ahead as far as the three TMEM buffers allow; the other (warp 15) issues the GEMMs
      // that consume the row threads' output (dQ, and dV^T/dK^T on dK/dV steps).  Neither waits
      // for barriers that only concern the other.
      // Step s uses buffer 0 while it is a dK/dV step, then buffers 0,1,2,0,... .
      auto buf_of = [&](int s) -> uint32_t { return s < n_active ? 0u : (uint32_t)((s - n_active) % 3); };
      auto use_of = [&](int s) {              // earlier uses of the buffer of step s
        const int i = s - n_active;
        return s < n_active ? s : (i % 3 == 0 ? n_active : 0) + i / 3;
      };
      auto wait_k = [&](int s) { return bwd_wait(&sm.k_full[s % kBwdKStages], (s / kBwdKStages) & 1, abort); };
      auto wait_v = [&](int s) { return bwd_wait(&sm.v_full[s % kBwdVStages], (s / kBwdVStages) & 1, abort); };
      auto wait_buf = [&](int s) {
        bool good = true;
        // the GEMMs that read the previous contents of this buffer (dS, or P/dS in shared memory) are done
        const int use = use_of(s);
        if (use > 0) good = bwd_wait(&sm.buf_free[buf_of(s)], (use - 1) & 1, abort);
        // buffer 1 aliases the dK^T/dV^T accumulators: the reduction warps must have read the last ones
        if (good && n_active > 0 && s == n_active + 1) good = bwd_wait(&sm.dkv_free, (n_active - 1) & 1, abort);
        return good;
      };
      bool ok = bwd_wait(&sm.q_full, 0, abort);
      for (int s = 0; s < n_tiles && ok; ++s) {
        const uint32_t buf = buf_of(s);
        ok = wait_k(s) && wait_v(s) && wait_buf(s);
        if (!ok) break;
        tc_fence_after_sync();
        HGA_TRACE_POINT(6);
        const uint64_t kd = desc_advance(k_k0, (uint32_t)(s % kBwdKStages) * kKvTile);
        const uint64_t vd = desc_advance(v_k0, (uint32_t)(s % kBwdVStages) * kKvTile);
        const uint32_t s_acc = tmem + buf_col(buf);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * 1024 + (kk & 3) * 32;
          mma_ss(s_acc, desc_advance(q_k, off), desc_advance(kd, off), idesc_sdp, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * 1024 + (kk & 3) * 32;
          mma_ss(s_acc + 64, desc_advance(do_k, off), desc_advance(vd, off), idesc_sdp, kk > 0);
        }
        mma_commit(&sm.sdp_full[buf]);
        mma_commit(&sm.v_empty[s % kBwdVStages]);      // the V tile is only needed for dP
        HGA_TRACE_POINT(8);
      }
    }
  } else if (warp == 15) {
    // ------------------------------------------------------------------ second MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, 0, 1);      // dS K-major, K tile MN-major
      constexpr uint32_t idesc_dkv = idesc_bf16_f32(D, kKT, 1, 1);     // both MN-major
      const uint64_t q_mn = smem_desc_sw128(smem_u32(sm.q), 1024, kOct);     // Q^T  as MN-major A (dK^T)
      const uint64_t do_mn = smem_desc_sw128(smem_u32(sm.dO), 1024, kOct);   // dO^T as MN-major A (dV^T)
      const uint64_t k_mn0 = smem_desc_sw128(smem_u32(sm.k[0]), 1024, kOct); // K tile, MN-major B (dQ)
      const uint64_t dsd = smem_desc_sw128(smem_u32(sm.ds), 16, 1024);       // dS: K-major A (dQ) and MN-major B (dK^T)
      const uint64_t pd = smem_desc_sw128(smem_u32(sm.p), 16, 1024);         // P : MN-major B (dV^T)
      bool ok = true;
      for (int s = 0; s < n_tiles && ok; ++s) {
        const bool dkv_step = s < n_active;
        const int i = s - n_active;
        const uint32_t buf = dkv_step ? 0u : (uint32_t)(i % 3);
        const int use = dkv_step ? s : (buf == 0 ? n_active : 0) + i / 3;
        ok = bwd_wait(&sm.pds_full[buf], use & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        HGA_TRACE_POINT(5);
        const uint64_t kmn = desc_advance(k_mn0, (uint32_t)(s % kBwdKStages) * kKvTile);
        if (dkv_step) {
#pragma unroll
          for (int kk = 0; kk < kKT / 16; ++kk)   // dQ += dS K : 16 keys per MMA, dS from shared memory
            mma_ss(tmem + kColDQ, desc_advance(dsd, kk * 32), desc_advance(kmn, kk * 2 * kOct), idesc_dq,
                   (s > 0 || kk > 0));
          if (s > 0) {
            ok = bwd_wait(&sm.dkv_free, (s - 1) & 1, abort);
            if (!ok) break;
            tc_fence_after_sync();
          }
#pragma unroll
          for (int kk = 0; kk < 128 / 16; ++kk)    // 16 query rows per MMA (2 row octets)
            mma_ss(tmem + kColDV, desc_advance(do_mn, kk * 2 * kOct), desc_advance(pd, kk * 2048), idesc_dkv, kk > 0);
#pragma unroll
          for (int kk = 0; kk < 128 / 16; ++kk)
            mma_ss(tmem + kColDK, desc_advance(q_mn, kk * 2 * kOct), desc_advance(dsd, kk * 2048), idesc_dkv, kk > 0);
          mma_commit(&sm.dkv_full);
        } else {
#pragma unroll
          for (int kk = 0; kk < kKT / 16; ++kk)   // dS (bf16) from TMEM, 8 columns per 16 keys
            mma_ts(tmem + kColDQ, tmem + buf_col(buf) + 8 * kk, desc_advance(kmn, kk * 2 * kOct), idesc_dq,
                   (s > 0 || kk > 0));
        }
        mma_commit(&sm.k_empty[s % kBwdKStages]);
        mma_commit(&sm.buf_free[buf]);
        HGA_TRACE_POINT(7);
      }
      if (ok) mma_commit(&sm.dq_done);
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------------ one thread per query row
    // Warpgroup 0 (warps 2-5) takes the dK/dV steps and then the even ones of the remaining steps,
    // warpgroup 1 (warps 6-9) the odd ones, each with its own S/dP buffer in TMEM, so the exp2 / dS
    // work of one step overlaps the GEMMs of the next.
    const int wg = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const int r = mt * 128 + row_in_tile;
    const int a = r / dm.Bq, t = r % dm.Bq;
    const int hq = h * dm.G + a, srow = qb * dm.Bq + t;
    const int limit = n_keys - dm.Bq + t + 1;
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    const float sl2 = dm.scale * 1.4426950408889634f;
    const float neg_lse2 = -row_lse * 1.4426950408889634f;
    const float neg_delta_s = -delta * dm.scale;
    HGA_TRACE_POINT(10);
    // this row's 128-byte line inside the P / dS buffers, and its swizzle key
    const uint32_t line = (uint32_t)(row_in_tile >> 3) * 1024 + (uint32_t)(row_in_tile & 7) * 128;
    const uint32_t key = (uint32_t)(row_in_tile & 7);
    const uint32_t p_line = smem_u32(sm.p) + line, ds_line = smem_u32(sm.ds) + line;
    bool ok = true;
    const int n_rest = n_tiles - n_active;
    const int n_mine = wg == 0 ? n_active + (n_rest + 1) / 2 : n_rest / 2;
    for (int u = 0; u < n_mine && ok; ++u) {
      const bool dkv_step = wg == 0 && u < n_active;
      const int s = dkv_step ? u : n_active + 2 * (u - (wg == 0 ? n_active : 0)) + wg;
      const int i = s - n_active;
      const uint32_t buf = dkv_step ? 0u : (uint32_t)(i % 3);
      const int use = dkv_step ? s : (buf == 0 ? n_active : 0) + i / 3;     // earlier uses of buf
      const uint32_t sdp_addr = lane_base + buf_col(buf);
      const int j = tile_of_step(s);
      ok = __all_sync(0xffffffffu, bwd_wait(&sm.sdp_full[buf], use & 1, abort));
      if (!ok) break;
      tc_fence_after_sync();
      HGA_TRACE_POINT(11);
      const int vis = limit - kKT * j;
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {               // 16 columns (keys) at a time: 128-register budget
        uint32_t sv[16], dp[16];
        tmem_ld16(sdp_addr + q4 * 16, sv);
        tmem_ld16(sdp_addr + 64 + q4 * 16, dp);
        tmem_wait_ld();
        uint32_t pk[8], dk[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float p0 = fast_exp2(fmaf(__uint_as_float(sv[2 * i]), sl2, neg_lse2));
          float p1 = fast_exp2(fmaf(__uint_as_float(sv[2 * i + 1]), sl2, neg_lse2));
          if (vis < kKT) {                    // diagonal / ragged tile only
            if (q4 * 16 + 2 * i >= vis) p0 = 0.f;
            if (q4 * 16 + 2 * i + 1 >= vis) p1 = 0.f;
          }
          const float d0 = p0 * fmaf(__uint_as_float(dp[2 * i]), dm.scale, neg_delta_s);
          const float d1 = p1 * fmaf(__uint_as_float(dp[2 * i + 1]), dm.scale, neg_delta_s);
          pk[i] = pack_bf16(p0, p1);
          dk[i] = pack_bf16(d0, d1);
        }
        if (dkv_step) {
          // P and dS feed the dV^T / dK^T GEMMs as shared-memory operands
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {    // two 16-byte chunks (8 keys each), XOR-swizzled
            const uint32_t off = ((uint32_t)(2 * q4 + cc) ^ key) * 16;
            st_shared_v4(p_line + off, pk[4 * cc], pk[4 * cc + 1], pk[4 * cc + 2], pk[4 * cc + 3]);
            st_shared_v4(ds_line + off, dk[4 * cc], dk[4 * cc + 1], dk[4 * cc + 2], dk[4 * cc + 3]);
          }
        } else {
          // bf16 dS over the S columns already read (8 columns per 16 keys): the A operand of dQ
          tmem_st8(sdp_addr + q4 * 8, dk);
        }
      }
      if (dkv_step) {
        fence_proxy_async_smem();
      } else {
        tmem_wait_st();
        tc_fence_before_sync();
      }
      mbar_arrive(&sm.pds_full[buf]);
      HGA_TRACE_POINT(14);
    }
    if (ok) ok = __all_sync(0xffffffffu, bwd_wait(&sm.dq_done, 0, abort));
    HGA_TRACE_POINT(20);
    if (ok) {
      // dQ epilogue: each warpgroup writes half of the row (64 columns)
      tc_fence_after_sync();
      uint16_t* qrow = dQ + b * dm.qs[0] + hq * dm.qs[1] + (int64_t)srow * dm.qs[2] + wg * 64;
      uint32_t x[2][32];
      tmem_ld32(lane_base + kColDQ + wg * 64, x[0]);
      tmem_ld32(lane_base + kColDQ + wg * 64 + 32, x[1]);
      tmem_wait_ld();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint4* dst = reinterpret_cast<uint4*>(qrow + c * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          dst[i] = make_uint4(pack_bf16(__uint_as_float(x[c][8 * i]), __uint_as_float(x[c][8 * i + 1])),
                              pack_bf16(__uint_as_float(x[c][8 * i + 2]), __uint_as_float(x[c][8 * i + 3])),
                              pack_bf16(__uint_as_float(x[c][8 * i + 4]), __uint_as_float(x[c][8 * i + 5])),
                              pack_bf16(__uint_as_float(x[c][8 * i + 6]), __uint_as_float(x[c][8 * i + 7])));
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
    for (int s = 0; s < n_active; ++s) {
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
  if (tid == 0 && sm.abort && status_word) atomicOr(status_word, HGA_STATUS_WAIT_TIMEOUT);
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// delta[row] = sum_e dO[row][e] * O[row][e]: one warp per row, 8-byte loads (a 256-byte row per
// request), an HBM stream of O and dO at full-GPU bandwidth.
__global__ void __launch_bounds__(256)
k_bwd_delta_sm100(const uint16_t* __restrict__ O, const uint16_t* __restrict__ dO, Dims dm,
                  float* __restrict__ delta) {
  // half a warp per row (16 lanes x 16 bytes = one 256-byte row), 8 rows per warp in flight
  const int lane = threadIdx.x & 31, sub = lane >> 4, chunk = lane & 15;
  const int64_t n_rows = (int64_t)dm.B * dm.Hq * dm.S;
  const int64_t warp_id = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t base = warp_id * 8; base < n_rows; base += n_warps * 8) {
    uint4 x[4], y[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t row = base + 2 * u + sub;
      x[u] = y[u] = make_uint4(0, 0, 0, 0);
      if (row < n_rows) {
        const int s = row % dm.S, hq = (row / dm.S) % dm.Hq, b = row / ((int64_t)dm.S * dm.Hq);
        const int64_t off = b * dm.os[0] + hq * dm.os[1] + (int64_t)s * dm.os[2] + chunk * 8;
        x[u] = *reinterpret_cast<const uint4*>(O + off);
        y[u] = *reinterpret_cast<const uint4*>(dO + off);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float part = dot4_bf16(make_uint2(x[u].x, x[u].y), make_uint2(y[u].x, y[u].y)) +
                   dot4_bf16(make_uint2(x[u].z, x[u].w), make_uint2(y[u].z, y[u].w));
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      const int64_t row = base + 2 * u + sub;
      if (chunk == 0 && row < n_rows) delta[row] = part;
    }
  }
}

bool attn_bwd_sm100_supported(const Dims& dm) {
  if (dm.flags & HGA_FLAG_GENERIC_KERNELS) return false;
  return dm.d == 128 && dm.rows % 128 == 0 && dm.g % 8 == 0;
}

int launch_attn_bwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const void* O,
                          const float* LSE, const void* dO, const int32_t* group_idx,
                          const int32_t* n_groups, void* dQ, float* dK, float* dV, float* delta_ws,
                          bool zero_grads, int32_t* status_word, cudaStream_t st) {
  CUtensorMap mq, mdo, mk, mv;
  const uint32_t box[5] = {64, 8, 2, 1, 1};
  const uint64_t dq[5] = {64, (uint64_t)dm.S, 2, (uint64_t)dm.Hq, (uint64_t)dm.B};
  const uint64_t dk[5] = {64, (uint64_t)dm.L, 2, (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t sq[4] = {(uint64_t)dm.qs[2] * 2, 128, (uint64_t)dm.qs[1] * 2, (uint64_t)dm.qs[0] * 2};
  const uint64_t so[4] = {(uint64_t)dm.os[2] * 2, 128, (uint64_t)dm.os[1] * 2, (uint64_t)dm.os[0] * 2};
  const uint64_t sk[4] = {(uint64_t)dm.ks[2] * 2, 128, (uint64_t)dm.ks[1] * 2, (uint64_t)dm.ks[0] * 2};
  const uint64_t sv[4] = {(uint64_t)dm.vs[2] * 2, 128, (uint64_t)dm.vs[1] * 2, (uint64_t)dm.vs[0] * 2};
  if (encode_tensor_map_bf16(&mq, Q, 5, dq, sq, box, true) ||
      encode_tensor_map_bf16(&mdo, dO, 5, dq, so, box, true) ||
      encode_tensor_map_bf16(&mk, K, 5, dk, sk, box, true) ||
      encode_tensor_map_bf16(&mv, V, 5, dk, sv, box, true))
    return HGA_ERR_UNSUPPORTED;
  // the octet table starts inside the struct's tail padding; 1024 bytes of slack for the manual alignment
  const size_t smem = offsetof(BwdSmem, oct_row) + sizeof(int) * (max_routed_tokens(dm) / 8 + 8) + 1024;
  if (smem > 227 * 1024) return HGA_ERR_UNSUPPORTED;
  cudaError_t e = cudaFuncSetAttribute(k_attn_bwd_sm100, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return record_cuda(e);
  const int64_t n_rows = (int64_t)dm.B * dm.Hq * dm.S;
  // one block = 8 warps x 8 rows; a multiple of the SM count when there is enough work
  const int64_t want_blocks = (n_rows + 63) / 64;
  const int delta_blocks = (int)(want_blocks < 148 * 8 ? want_blocks : 148 * 8);
  k_bwd_delta_sm100<<<delta_blocks, 256, 0, st>>>((const uint16_t*)O, (const uint16_t*)dO, dm, delta_ws);
  e = cudaGetLastError();
  if (e != cudaSuccess) return record_cuda(e);
  // dK/dV of the local band: written once per key tile by the key-major kernel (plain stores that
  // cover every row of the active segment), which also makes zero-filling unnecessary.  Where that
  // kernel does not apply, this kernel adds every contribution atomically onto zeroed buffers.
  int band_done = 0;
  if (attn_bwd_band_sm100_supported(dm)) {
    const int rc = launch_attn_bwd_band_sm100(dm, Q, K, V, LSE, dO, dK, dV, delta_ws, status_word, st);
    if (rc == HGA_OK) band_done = 1;
    else if (rc != HGA_ERR_UNSUPPORTED) return rc;
  }
  if (!band_done && zero_grads) {
    const size_t bytes = (size_t)dm.B * dm.Hkv * dm.S * dm.d * sizeof(float);
    if ((e = cudaMemsetAsync(dK, 0, bytes, st)) != cudaSuccess) return record_cuda(e);
    if ((e = cudaMemsetAsync(dV, 0, bytes, st)) != cudaSuccess) return record_cuda(e);
  }
  const int units = dm.B * dm.Hkv * dm.NQB * (dm.rows / 128);
  k_attn_bwd_sm100<<<units, kBwdThreads, smem, st>>>(mq, mdo, mk, mv, delta_ws, LSE, group_idx, n_groups, dm,
                                                    (uint16_t*)dQ, dK, dV, band_done, status_word);
  count_launch(2);
  return record_cuda(cudaGetLastError());
}

}  // namespace hga
