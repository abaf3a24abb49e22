// Key-major backward of the local band for sm_100a (head_dim 128): dK and dV of the keys that query
// blocks see through their local window or their own causal block (Section 2.1: the dense part of
// the routed set; Section 2.2: only keys of the active segment receive gradients).
//
// Every key of the active segment lies in the band of a few consecutive query blocks (its own
// block and the ones whose local window still reaches it).  Summing those contributions with
// atomics from the query-major sweep costs one red.add per element per contributing M-tile; here
// one CTA owns a 64-key tile instead, loops over every 128-row M-tile of every query block whose
// band holds the tile, accumulates dK^T and dV^T in TMEM and writes the tile once with plain stores.
// The query-major sweep (k_attn_bwd_sm100) then adds only the contributions of keys selected
// through routing, and computes dQ for all keys.
//
// Work unit (one CTA): (batch, kv head, 64-key tile of the active segment).  Per M-tile m:
//   S = Q K^T, dP = dO V^T                       (smem x smem) -> TMEM, double buffered
//   P = 2^(S*c - LSE*log2e), dS = scale * P o (dP - delta)     (one thread per query row) -> smem
//   dV^T += dO^T P,  dK^T += Q^T dS              (M = head_dim, N = 64 keys, K = 128 rows) -> TMEM
// Q and dO tiles stream through a two-stage ring as boxes of 64 rows x one 64-element panel, laid
// out [panel][128 rows][128 B]: the 128-byte-swizzled layout the GEMMs read both K-major (S, dP)
// and MN-major (dK^T, dV^T).  The MMA thread issues whichever GEMM group (S,dP of the next M-tile or
// dK,dV of the previous one) has its inputs ready, so the two ring stages advance independently.
//
// Warp roles (320 threads): warp 0 producer, warp 1 MMA issuer, warps 2-5 and 6-9 two warpgroups
// of row threads on alternate M-tiles; at the end warps 2-5 store dV, warps 6-9 store dK.
// TMEM (512 columns allocated): S[2] dP[2] (64 each) | dV^T 64 | dK^T 64.
#include "hga_bwd_sm100.cuh"
#include "hga_common.cuh"
#include "hga_sm100.cuh"

namespace hga {

using namespace sm100;

namespace {

constexpr int kBandThreads = 320;
constexpr int kD = 128;
constexpr int kKT = 64;                          // keys per tile
constexpr int kQTile = 128 * kD * 2;             // bytes of one Q or dO tile
constexpr int kKvTile = kKT * kD * 2;
constexpr int kPdsTile = 128 * kKT * 2;

struct BandSmem {
  alignas(1024) uint8_t q[2][kQTile];            // [panel][128 rows][128 B]
  alignas(1024) uint8_t dO[2][kQTile];
  alignas(1024) uint8_t k[kKvTile];              // [panel][64 keys][128 B]
  alignas(1024) uint8_t v[kKvTile];
  alignas(1024) uint8_t p[2][kPdsTile];          // [16 row octets][8 rows][128 B]
  alignas(1024) uint8_t ds[2][kPdsTile];
  uint64_t kv_full, qdo_full[2], qdo_empty[2], sdp_full[2], sdp_free[2], pds_full[2], pds_free[2], acc_done;
  uint32_t tmem_base;
  volatile int abort;
};

__global__ void __launch_bounds__(kBandThreads, 1)
k_attn_bwd_band_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                      const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const float* __restrict__ delta_ws, const float* __restrict__ LSE, Dims dm,
                      float* __restrict__ dK, float* __restrict__ dV, int32_t* status_word) {
  constexpr uint32_t kColSdP = 0;       // S[b] at 128*b, dP[b] at 128*b + 64
  constexpr uint32_t kColDV = 256, kColDK = 320;
  extern __shared__ uint8_t smem_raw[];
  BandSmem& sm = *reinterpret_cast<BandSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  HGA_TRACE_DECL;
  const int tiles_per_seq = dm.S / kKT;
  const int kt = blockIdx.x % tiles_per_seq;
  const int bh = blockIdx.x / tiles_per_seq;
  const int h = bh % dm.Hkv, b = bh / dm.Hkv;
  const int k0 = dm.H + kt * kKT;                 // first key position of the tile
  // query blocks whose band [ls, p0 + Bq) holds the tile: the tile's own block and the following
  // ones while their local window still starts at or before the tile
  const int qb_own = (kt * kKT) / dm.Bq;
  int n_qb = 1;
  while (qb_own + n_qb < dm.NQB && window_of(dm, qb_own + n_qb).ls <= k0) ++n_qb;
  const int n_mt = dm.rows / 128;
  const int n_steps = n_qb * n_mt;

  if (tid == 0) {
    mbar_init(&sm.kv_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.qdo_full[s], 1); mbar_init(&sm.qdo_empty[s], 1);
      mbar_init(&sm.sdp_full[s], 1); mbar_init(&sm.sdp_free[s], 128);
      mbar_init(&sm.pds_full[s], 128); mbar_init(&sm.pds_free[s], 1);
    }
    mbar_init(&sm.acc_done, 1);
    sm.abort = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tmem = sm.tmem_base;
  volatile int* abort = &sm.abort;
  HGA_TRACE_POINT(1);

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    // A copy is latency-bound per box, so a Q or dO tile travels as four boxes of 64 rows x one
    // 64-element panel (8 KB each), issued by eight lanes at once: lanes 0-3 Q, lanes 4-7 dO.
    if (lane == 0) {
      prefetch_tensormap(&map_q); prefetch_tensormap(&map_do);
      prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
      mbar_arrive_expect_tx(&sm.kv_full, 2 * kKvTile);
      tma_load_5d(sm.k, &map_k, &sm.kv_full, 0, k0, 0, h, b);
      tma_load_5d(sm.v, &map_v, &sm.kv_full, 0, k0, 0, h, b);
    }
    const int half = lane & 1, panel = (lane >> 1) & 1;       // 64-row half of the M-tile, d panel
    bool ok = true;
    int issued = 0;
    for (int m = 0; m < n_steps; ++m) {
      const int st = m & 1;
      const int qb = qb_own + m / n_mt, r0 = (m % n_mt) * 128 + half * 64;
      if (lane == 0 && m >= 2) ok = bwd_wait(&sm.qdo_empty[st], ((m >> 1) - 1) & 1, abort);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) mbar_arrive_expect_tx(&sm.qdo_full[st], 2 * kQTile);
      __syncwarp();
      const int row = qb * dm.Bq + r0 % dm.Bq, head = h * dm.G + r0 / dm.Bq;
      const uint32_t off = (uint32_t)panel * 16384 + (uint32_t)half * 8192;
      if (lane < 4) tma_load_5d(sm.q[st] + off, &map_q, &sm.qdo_full[st], 0, row, panel, head, b);
      else if (lane < 8) tma_load_5d(sm.dO[st] + off, &map_do, &sm.qdo_full[st], 0, row, panel, head, b);
      issued = m + 1;
      HGA_TRACE_POINT(2);
    }
    if (*abort && lane == 0) {
      // giving up: let the copies still in flight land before shared memory is released
      mbar_wait(&sm.kv_full, 0);
      for (int m = issued > 2 ? issued - 2 : 0; m < issued; ++m) mbar_wait(&sm.qdo_full[m & 1], (m >> 1) & 1);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_sdp = idesc_bf16_f32(128, kKT, 0, 0);   // rows x keys, both K-major
      constexpr uint32_t idesc_dkv = idesc_bf16_f32(kD, kKT, 1, 1);    // both MN-major
      const uint64_t q_k0 = smem_desc_sw128(smem_u32(sm.q[0]), 16, 1024);       // Q  K-major A (S)
      const uint64_t do_k0 = smem_desc_sw128(smem_u32(sm.dO[0]), 16, 1024);     // dO K-major A (dP)
      const uint64_t q_mn0 = smem_desc_sw128(smem_u32(sm.q[0]), 16384, 1024);   // Q^T  MN-major A (dK^T)
      const uint64_t do_mn0 = smem_desc_sw128(smem_u32(sm.dO[0]), 16384, 1024); // dO^T MN-major A (dV^T)
      const uint64_t k_k = smem_desc_sw128(smem_u32(sm.k), 16, 1024);           // K tile K-major B (S)
      const uint64_t v_k = smem_desc_sw128(smem_u32(sm.v), 16, 1024);           // V tile K-major B (dP)
      const uint64_t ds0 = smem_desc_sw128(smem_u32(sm.ds[0]), 16, 1024);       // dS MN-major B (dK^T)
      const uint64_t p0 = smem_desc_sw128(smem_u32(sm.p[0]), 16, 1024);         // P  MN-major B (dV^T)
      auto issue_sdp = [&](int m) {
        const uint32_t st = (uint32_t)(m & 1);
        const uint64_t qd = desc_advance(q_k0, st * kQTile), dod = desc_advance(do_k0, st * kQTile);
        const uint32_t s_acc = tmem + kColSdP + st * 128;
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk)
          mma_ss(s_acc, desc_advance(qd, (kk >> 2) * 16384 + (kk & 3) * 32),
                 desc_advance(k_k, (kk >> 2) * 8192 + (kk & 3) * 32), idesc_sdp, kk > 0);
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk)
          mma_ss(s_acc + 64, desc_advance(dod, (kk >> 2) * 16384 + (kk & 3) * 32),
                 desc_advance(v_k, (kk >> 2) * 8192 + (kk & 3) * 32), idesc_sdp, kk > 0);
        mma_commit(&sm.sdp_full[st]);
      };
      auto issue_dkv = [&](int m) {
        const uint32_t st = (uint32_t)(m & 1);
        const uint64_t pd = desc_advance(p0, st * kPdsTile), dsd = desc_advance(ds0, st * kPdsTile);
        const uint64_t dom = desc_advance(do_mn0, st * kQTile), qm = desc_advance(q_mn0, st * kQTile);
#pragma unroll
        for (int kk = 0; kk < 128 / 16; ++kk)    // 16 query rows per step
          mma_ss(tmem + kColDV, desc_advance(dom, kk * 2048), desc_advance(pd, kk * 2048), idesc_dkv,
                 (m > 0 || kk > 0));
#pragma unroll
        for (int kk = 0; kk < 128 / 16; ++kk)
          mma_ss(tmem + kColDK, desc_advance(qm, kk * 2048), desc_advance(dsd, kk * 2048), idesc_dkv,
                 (m > 0 || kk > 0));
        mma_commit(&sm.pds_free[st]);
        mma_commit(&sm.qdo_empty[st]);
      };
      // The two ring stages form two independent chains (copy -> S,dP -> row threads -> dK,dV ->
      // next copy); whichever GEMM group has its inputs ready is issued next, the dK/dV group
      // first because it releases a stage.
      bool ok = bwd_wait(&sm.kv_full, 0, abort);
      int next_sdp = 0, next_dkv = 0;
      uint32_t idle = 0;
      while (ok && next_dkv < n_steps) {
        bool did = false;
        if (next_dkv < next_sdp && mbar_test_wait(&sm.pds_full[next_dkv & 1], (next_dkv >> 1) & 1)) {
          tc_fence_after_sync();
          issue_dkv(next_dkv);
          ++next_dkv;
          did = true;
          HGA_TRACE_POINT(7);
        }
        if (next_sdp < n_steps && mbar_test_wait(&sm.qdo_full[next_sdp & 1], (next_sdp >> 1) & 1) &&
            (next_sdp < 2 || mbar_test_wait(&sm.sdp_free[next_sdp & 1], ((next_sdp >> 1) - 1) & 1))) {
          // (a full stage implies that dK/dV of M-tile next_sdp-2 were issued, hence that its row
          // threads are done with TMEM buffer next_sdp&1; the sdp_free test makes that visible here)
          tc_fence_after_sync();
          issue_sdp(next_sdp);
          ++next_sdp;
          did = true;
          HGA_TRACE_POINT(6);
        }
        if (did) idle = 0;
        else if (++idle >= (1u << 22) || ((idle & 255u) == 255u && *abort)) { *abort = 1; ok = false; }
      }
      if (ok) mma_commit(&sm.acc_done);
    }
  } else {
    // ------------------------------------------------------------------ one thread per query row
    const int wg = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    const float sl2 = dm.scale * 1.4426950408889634f;
    const uint32_t line = (uint32_t)(row_in_tile >> 3) * 1024 + (uint32_t)(row_in_tile & 7) * 128;
    const uint32_t key = (uint32_t)(row_in_tile & 7);
    const uint32_t p_line = smem_u32(sm.p[wg]) + line, ds_line = smem_u32(sm.ds[wg]) + line;
    const uint32_t sdp_addr = lane_base + kColSdP + wg * 128;
    // LSE, delta and the causal limit of this thread's row in M-tile m
    auto row_of = [&](int m, float& lse, float& dl, int& vis) {
      const int qb = qb_own + m / n_mt, r = (m % n_mt) * 128 + row_in_tile;
      const int a = r / dm.Bq, t = r % dm.Bq;
      const int64_t row = ((int64_t)b * dm.Hq + h * dm.G + a) * dm.S + qb * dm.Bq + t;
      lse = LSE[row];
      dl = delta_ws[row];
      vis = qb * dm.Bq + t - kt * kKT + 1;       // keys of the tile at or before the query position
    };
    float lse = 0.f, dl = 0.f;
    int vis = 0;
    // This kernel is launched with programmatic serialization behind the delta pre-pass: everything up to
    // here (set-up, the K/V tile and the first Q/dO tiles, which are inputs of the call) may have run
    // while that kernel was still busy; delta is read from here on.  Only then is the sweep, which follows
    // in the stream and reads delta too, allowed to start on the SMs this grid leaves idle (it waits for
    // this grid itself only before it adds to dK/dV).
    pdl_wait();
    if (warp == 2 && lane == 0) pdl_launch_dependents();
    if (wg < n_steps) row_of(wg, lse, dl, vis);
    bool ok = true;
    for (int m = wg; m < n_steps; m += 2) {
      const float neg_lse2 = -lse * 1.4426950408889634f;
      const float neg_delta_s = -dl * dm.scale;
      const uint64_t sl2_2 = pack_f32x2(sl2, sl2), neg_lse2_2 = pack_f32x2(neg_lse2, neg_lse2);
      const uint64_t scale_2 = pack_f32x2(dm.scale, dm.scale), neg_delta_s_2 = pack_f32x2(neg_delta_s, neg_delta_s);
      const int vis_m = vis;
      if (m + 2 < n_steps) row_of(m + 2, lse, dl, vis);      // prefetch the next M-tile's row data
      ok = __all_sync(0xffffffffu, bwd_wait(&sm.sdp_full[wg], (m >> 1) & 1, abort));
      if (!ok) break;
      tc_fence_after_sync();
      HGA_TRACE_POINT(11);
      if (m >= 2) {     // the GEMMs that read this P/dS buffer two steps ago must have finished
        ok = __all_sync(0xffffffffu, bwd_wait(&sm.pds_free[wg], ((m >> 1) - 1) & 1, abort));
        if (!ok) break;
      }
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {               // 16 keys at a time
        uint32_t sv[16], dp[16];
        tmem_ld16(sdp_addr + q4 * 16, sv);
        tmem_ld16(sdp_addr + 64 + q4 * 16, dp);
        tmem_wait_ld();
        if (q4 == 3) {
          tc_fence_before_sync();
          mbar_arrive(&sm.sdp_free[wg]);
        }
        uint32_t pk[8], dk[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          // packed fp32 pairs: one FMA-pipe instruction for two columns
          float a0, a1, d0, d1;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1])), sl2_2, neg_lse2_2), a0, a1);
          float p0 = fast_exp2(a0), p1 = fast_exp2(a1);
          if (vis_m < kKT) {                  // the tile's own query block: causal mask
            if (q4 * 16 + 2 * i >= vis_m) p0 = 0.f;
            if (q4 * 16 + 2 * i + 1 >= vis_m) p1 = 0.f;
          }
          const uint64_t g2 = fma_f32x2(pack_f32x2(__uint_as_float(dp[2 * i]), __uint_as_float(dp[2 * i + 1])), scale_2, neg_delta_s_2);
          unpack_f32x2(mul_f32x2(pack_f32x2(p0, p1), g2), d0, d1);
          pk[i] = pack_bf16(p0, p1);
          dk[i] = pack_bf16(d0, d1);
        }
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {      // two 16-byte chunks (8 keys each), XOR-swizzled
          const uint32_t off = ((uint32_t)(2 * q4 + cc) ^ key) * 16;
          st_shared_v4(p_line + off, pk[4 * cc], pk[4 * cc + 1], pk[4 * cc + 2], pk[4 * cc + 3]);
          st_shared_v4(ds_line + off, dk[4 * cc], dk[4 * cc + 1], dk[4 * cc + 2], dk[4 * cc + 3]);
        }
      }
      fence_proxy_async_smem();
      mbar_arrive(&sm.pds_full[wg]);
      HGA_TRACE_POINT(14);
    }
    if (ok) ok = __all_sync(0xffffffffu, bwd_wait(&sm.acc_done, 0, abort));
    HGA_TRACE_POINT(20);
    if (ok) {
      // epilogue: thread = head_dim element (TMEM lane); a warp's store covers 128 contiguous bytes
      tc_fence_after_sync();
      const int e = quarter * 32 + lane;
      float* dst = (wg == 0 ? dV : dK) + ((int64_t)(b * dm.Hkv + h) * dm.S + kt * kKT) * kD + e;
      const uint32_t col = wg == 0 ? kColDV : kColDK;
      const bool accumulate = dm.flags & HGA_FLAG_BWD_ACCUMULATE;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t x[32];
        tmem_ld32(lane_base + col + half * 32, x);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float* d = dst + (int64_t)(half * 32 + i) * kD;
          *d = accumulate ? *d + __uint_as_float(x[i]) : __uint_as_float(x[i]);
        }
      }
    }
  }
  HGA_TRACE_POINT(30);

  // every warp reconverges before the block barrier (a barrier reached by part of a warp would
  // count that warp as arrived)
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  HGA_TRACE_DUMP;
  if (tid == 0 && sm.abort && status_word) atomicOr(status_word, HGA_STATUS_WAIT_TIMEOUT);
  if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace

bool attn_bwd_band_sm100_supported(const Dims& dm) {
  if (dm.flags & HGA_FLAG_GENERIC_KERNELS) return false;
  return dm.d == 128 && dm.rows % 128 == 0 && dm.Bq % 64 == 0 && dm.c % kKT == 0 && dm.H % kKT == 0 && dm.S % kKT == 0;
}

int launch_attn_bwd_band_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const float* LSE,
                               const void* dO, float* dK, float* dV, const float* delta_ws, int32_t* status_word,
                               cudaStream_t st) {
  CUtensorMap mq, mdo, mk, mv;
  const uint32_t box_q[5] = {64, 64, 1, 1, 1};
  const uint32_t box_k[5] = {64, kKT, 2, 1, 1};
  const uint64_t dq[5] = {64, (uint64_t)dm.S, 2, (uint64_t)dm.Hq, (uint64_t)dm.B};
  const uint64_t dk[5] = {64, (uint64_t)dm.L, 2, (uint64_t)dm.Hkv, (uint64_t)dm.B};
  const uint64_t sq[4] = {(uint64_t)dm.qs[2] * 2, 128, (uint64_t)dm.qs[1] * 2, (uint64_t)dm.qs[0] * 2};
  const uint64_t so[4] = {(uint64_t)dm.os[2] * 2, 128, (uint64_t)dm.os[1] * 2, (uint64_t)dm.os[0] * 2};
  const uint64_t sk[4] = {(uint64_t)dm.ks[2] * 2, 128, (uint64_t)dm.ks[1] * 2, (uint64_t)dm.ks[0] * 2};
  const uint64_t sv[4] = {(uint64_t)dm.vs[2] * 2, 128, (uint64_t)dm.vs[1] * 2, (uint64_t)dm.vs[0] * 2};
  if (encode_tensor_map_bf16(&mq, Q, 5, dq, sq, box_q, true) ||
      encode_tensor_map_bf16(&mdo, dO, 5, dq, so, box_q, true) ||
      encode_tensor_map_bf16(&mk, K, 5, dk, sk, box_k, true) ||
      encode_tensor_map_bf16(&mv, V, 5, dk, sv, box_k, true))
    return HGA_ERR_UNSUPPORTED;
  const size_t smem = sizeof(BandSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(k_attn_bwd_band_sm100, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return record_cuda(e);
  const int units = dm.B * dm.Hkv * (dm.S / kKT);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)units);
  cfg.blockDim = dim3(kBandThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;   // behind the delta pre-pass of the same call
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = (dm.flags & kFlagNoPdl) ? 0 : 1;
  e = cudaLaunchKernelEx(&cfg, k_attn_bwd_band_sm100, mq, mdo, mk, mv, delta_ws, LSE, dm, dK, dV, status_word);
  count_launch(1);
  return record_cuda(e);
}

}  // namespace hga
