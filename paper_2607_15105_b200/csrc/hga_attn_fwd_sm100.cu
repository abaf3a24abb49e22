// hga_attn_fwd for sm_100a: routed exact-token attention as a TMA-gather-fed tcgen05 / TMEM
// flash-style kernel (Section 2.1 item 3).
//
// Work unit (one CTA): up to two 128-row M-tiles of one item (b, kv head, query block); the
// G*Bq query rows of the item share one routed key set, so K/V are gathered once per unit.
// Keys are addressed in "octets" (8 consecutive tokens = one 8-row 128-byte-swizzle atom per
// 64-element panel): sink, each selected group and the local window are runs of octets, and a
// 128-key tile is 16 octets fetched by 16 TMA boxes (one lane each), K and V on separate
// barriers.  Octets past the end of the list load an out-of-range row and arrive as zeros.
//
// Warp roles (320 threads):
//   warp 0      producer: octet table, Q load, K/V tile ring (2 stages each)
//   warp 1      MMA issuer (one thread): S = Q K^T (smem x smem), O += P V (P from TMEM)
//   warps 2-5   softmax of M-tile 0, one thread per row (thread owns TMEM lane = row)
//   warps 6-9   softmax of M-tile 1
// The two M-tiles ping-pong on the tensor core: while one tile's rows do exp2, the other
// tile's GEMM runs.  TMEM (512 columns): S0 | S1 | O0 | O1; P (bf16) overwrites S in place.
// The running maximum is only raised when it grows by more than 2^8 (rescaling O is then done
// by the row's own thread between the S and the PV of that tile), so rescales are rare.
#include "hga_common.cuh"
#include "hga_sm100.cuh"

namespace hga {

using namespace sm100;

constexpr int kFwdThreads = 320;
constexpr int kStages = 2;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

template <int D>
struct FwdSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  alignas(1024) uint8_t q[2][kTileBytes];
  alignas(1024) uint8_t k[kStages][kTileBytes];
  alignas(1024) uint8_t v[kStages][kTileBytes];
  uint64_t q_full;
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[2], p_full[2], o_done[2];
  uint32_t tmem_base;
  int n_oct;
  volatile int abort;
  int oct_row[1];   // really max_routed_tokens/8 entries (dynamic shared memory follows)
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort) {
  for (uint32_t i = 0; i < (1u << 20); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort) return false;
  }
  *abort = 1;
  return false;
}

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
k_attn_fwd_sm100(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ group_idx,
                 const int32_t* __restrict__ n_groups, Dims dm, uint16_t* __restrict__ O,
                 float* __restrict__ LSE, int32_t* status_word) {
  constexpr int kPanels = D / 64;
  constexpr int kOctBytes = 8 * D * 2;            // one octet of rows, all panels
  constexpr int kTileBytes = 128 * D * 2;
  constexpr uint32_t kSbo = kOctBytes;            // byte distance between 8-row groups
  constexpr uint32_t kColS = 0, kColO = 256;      // TMEM columns: S0 S1 at 0,128; O0 O1 at 256, 256+D
  extern __shared__ uint8_t smem_raw[];
  FwdSmem<D>& sm = *reinterpret_cast<FwdSmem<D>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_mt_item = dm.rows / 128;
  const int units_per_item = (n_mt_item + 1) / 2;
  const int item = blockIdx.x / units_per_item;
  const int mt0 = (blockIdx.x % units_per_item) * 2;
  const int mt_count = n_mt_item - mt0 < 2 ? n_mt_item - mt0 : 2;
  int b, h, qb;
  item_coords(dm, item, b, h, qb);
  const Window w = window_of(dm, qb);

  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], 1); mbar_init(&sm.k_empty[s], 1);
      mbar_init(&sm.v_full[s], 1); mbar_init(&sm.v_empty[s], 1);
    }
    for (int m = 0; m < 2; ++m) {
      mbar_init(&sm.s_full[m], 1); mbar_init(&sm.p_full[m], 128); mbar_init(&sm.o_done[m], 1);
    }
    sm.abort = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  if (warp == 0) {
    // octet table: lane 0 validates the group list (ascending, between sink and local window)
    if (lane == 0) {
      prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
      const int32_t* gi = group_idx + (int64_t)item * dm.width;
      int ng = n_groups[item], bad = 0, n = w.se / 8, prev = -1;
      if (ng > dm.width) { ng = dm.width; bad = 1; }
      if (ng < 0) { ng = 0; bad = 1; }
      const int opg = dm.g / 8;
      for (int i = 0; i < ng; ++i) {
        const int m = gi[i];
        if (m > prev && (int64_t)m * dm.g >= w.se && ((int64_t)m + 1) * dm.g <= w.ls) {
          for (int u = 0; u < opg; ++u) sm.oct_row[n++] = m * dm.g + 8 * u;
          prev = m;
        } else {
          bad = 1;
        }
      }
      sm.n_oct = n;   // octets before the local window (sink entries are filled below)
      if (bad && status_word) atomicOr(status_word, HGA_STATUS_BAD_INDEX);
    }
    __syncwarp();
    const int n_far = sm.n_oct;
    for (int o = lane; o < w.se / 8; o += 32) sm.oct_row[o] = 8 * o;
    const int n_local = (w.p0 + dm.Bq - w.ls) / 8;
    for (int o = lane; o < n_local; o += 32) sm.oct_row[n_far + o] = w.ls + 8 * o;
    __syncwarp();
    if (lane == 0) sm.n_oct = n_far + n_local;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tmem = sm.tmem_base;
  const int n_oct = sm.n_oct;
  const int n_keys = n_oct * 8;
  const int n_tiles = (n_oct + 15) / 16;
  volatile int* abort = &sm.abort;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) mbar_arrive_expect_tx(&sm.q_full, (uint32_t)(mt_count * kTileBytes));
    __syncwarp();
    for (int o = lane; o < mt_count * 16; o += 32) {
      const int r = mt0 * 128 + 8 * o;                 // first row of the octet inside the item
      const int a = r / dm.Bq, t = r % dm.Bq;
      tma_load_5d(sm.q[o >> 4] + (o & 15) * kOctBytes, &map_q, &sm.q_full, 0, qb * dm.Bq + t, 0,
                  h * dm.G + a, b);
    }
    bool ok = true;
    int issued = 0;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const int s = j % kStages, use = j / kStages;
      if (lane == 0 && use > 0) {
        ok = wait_or_abort(&sm.k_empty[s], (use - 1) & 1, abort) &&
             wait_or_abort(&sm.v_empty[s], (use - 1) & 1, abort);
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) {
        mbar_arrive_expect_tx(&sm.k_full[s], kTileBytes);
        mbar_arrive_expect_tx(&sm.v_full[s], kTileBytes);
      }
      __syncwarp();
      const int o = 16 * j + (lane & 15);
      const int row = o < n_oct ? sm.oct_row[o] : dm.L;     // past the list: out of range -> zeros
      if (lane < 16) tma_load_5d(sm.k[s] + lane * kOctBytes, &map_k, &sm.k_full[s], 0, row, 0, h, b);
      else tma_load_5d(sm.v[s] + (lane - 16) * kOctBytes, &map_v, &sm.v_full[s], 0, row, 0, h, b);
      issued = j + 1;
    }
    if (*abort && lane == 0) {
      // giving up: let the copies still in flight land before shared memory is released
      mbar_wait(&sm.q_full, 0);
      for (int j = issued > kStages ? issued - kStages : 0; j < issued; ++j) {
        mbar_wait(&sm.k_full[j % kStages], (j / kStages) & 1);
        mbar_wait(&sm.v_full[j % kStages], (j / kStages) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
      constexpr uint32_t idesc_o = idesc_bf16_f32(128, D, 0, 1);
      auto issue_s = [&](int mt, int stage) {
        const uint32_t qa = smem_u32(sm.q[mt]), ka = smem_u32(sm.k[stage]);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * 1024 + (kk & 3) * 32;   // panel, then 32-byte K step
          mma_ss(tmem + kColS + mt * 128, smem_desc_sw128(qa + off, 16, kSbo),
                 smem_desc_sw128(ka + off, 16, kSbo), idesc_s, kk > 0);
        }
        mma_commit(&sm.s_full[mt]);
      };
      bool ok = wait_or_abort(&sm.q_full, 0, abort) && wait_or_abort(&sm.k_full[0], 0, abort);
      if (ok) {
        tc_fence_after_sync();
        for (int mt = 0; mt < mt_count; ++mt) issue_s(mt, 0);
        mma_commit(&sm.k_empty[0]);          // K stage 0 is free once S of tile 0 has been computed
      }
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int sv = j % kStages, sk = (j + 1) % kStages;
        const bool more = j + 1 < n_tiles;
        ok = wait_or_abort(&sm.v_full[sv], (j / kStages) & 1, abort);
        if (ok && more) ok = wait_or_abort(&sm.k_full[sk], ((j + 1) / kStages) & 1, abort);
        for (int mt = 0; mt < mt_count && ok; ++mt) {
          ok = wait_or_abort(&sm.p_full[mt], j & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t va = smem_u32(sm.v[sv]);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {   // 16 keys per step: 2 octets in smem, 8 TMEM columns of P
            mma_ts(tmem + kColO + mt * D, tmem + kColS + mt * 128 + kk * 8,
                   smem_desc_sw128(va + kk * 2 * kOctBytes, 1024, kSbo), idesc_o, (j > 0 || kk > 0));
          }
          if (more) issue_s(mt, sk);
          else mma_commit(&sm.o_done[mt]);
        }
        if (ok) {
          mma_commit(&sm.v_empty[sv]);
          if (more) mma_commit(&sm.k_empty[sk]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    const int mt = (warp - 2) >> 2;
    if (mt < mt_count) {
      const int quarter = warp & 3;                       // TMEM lanes this warp may touch
      const int row_in_tile = quarter * 32 + lane;
      const int r = (mt0 + mt) * 128 + row_in_tile;       // row inside the item
      const int a = r / dm.Bq, t = r % dm.Bq;
      const int limit = n_keys - dm.Bq + t + 1;           // visible key slots (causal inside the block)
      const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
      const uint32_t s_addr = lane_base + kColS + mt * 128;
      const uint32_t o_addr = lane_base + kColO + mt * D;
      const float sl2 = dm.scale * 1.4426950408889634f;   // softmax scale in log2 units
      float m_used = -INFINITY, l = 0.f, l_mma = 0.f;
      bool ok = true;
      for (int j = 0; j < n_tiles; ++j) {
        ok = __all_sync(0xffffffffu, wait_or_abort(&sm.s_full[mt], j & 1, abort));
        if (!ok) break;                                   // warp-uniform
        tc_fence_after_sync();
        const int vis = limit - 128 * j;                  // visible columns of this tile (may be <= 0)
        // pass 1: row maximum over the visible columns
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t x[32];
          tmem_ld32(s_addr + c * 32, x);
          tmem_wait_ld();
          if (vis >= 32 * c + 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(x[i]));
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (32 * c + i < vis) mx = fmaxf(mx, __uint_as_float(x[i]));
          }
        }
        mx *= sl2;
        float corr = 1.f;
        bool raise = mx > m_used + kRescaleThreshold;     // also true for the first visible tile
        if (raise) {
          corr = fast_exp2(m_used - mx);                  // 0 when m_used is -inf
          m_used = mx;
          l *= corr;
          l_mma *= corr;
        }
        // O holds the sum up to tile j-1 (its MMA finished before S of tile j was signalled)
        if (j > 0 && __any_sync(0xffffffffu, raise)) {
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t x[32];
            tmem_ld32(o_addr + c * 32, x);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) x[i] = __float_as_uint(__uint_as_float(x[i]) * corr);
            tmem_st32(o_addr + c * 32, x);
          }
        }
        // pass 2: p = 2^(x - m), row sum, P (bf16) written over S
        const float neg_m = -m_used;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t x[32];
          tmem_ld32(s_addr + c * 32, x);
          tmem_wait_ld();
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float p0 = fast_exp2(fmaf(__uint_as_float(x[2 * i]), sl2, neg_m));
            float p1 = fast_exp2(fmaf(__uint_as_float(x[2 * i + 1]), sl2, neg_m));
            if (32 * c + 2 * i >= vis) p0 = 0.f;
            if (32 * c + 2 * i + 1 >= vis) p1 = 0.f;
            l += p0 + p1;
            const __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
            pk[i] = *reinterpret_cast<const uint32_t*>(&hh);
            // the weights the MMA really applies are the rounded ones: normalising O by THEIR sum
            // makes the rounding of a dominant weight cancel; LSE keeps the unrounded sum
            l_mma += __uint_as_float(pk[i] << 16) + __uint_as_float(pk[i] & 0xffff0000u);
          }
          tmem_st16(s_addr + c * 16, pk);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&sm.p_full[mt]);
      }
      if (ok) ok = __all_sync(0xffffffffu, wait_or_abort(&sm.o_done[mt], 0, abort));
      if (ok) {
        tc_fence_after_sync();
        const float inv = 1.f / l_mma;
        const int hq = h * dm.G + a, srow = qb * dm.Bq + t;
        uint16_t* orow = O + b * dm.os[0] + hq * dm.os[1] + (int64_t)srow * dm.os[2];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t x[32];
          tmem_ld32(o_addr + c * 32, x);
          tmem_wait_ld();
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(x[2 * i]) * inv,
                                                             __uint_as_float(x[2 * i + 1]) * inv);
            pk[i] = *reinterpret_cast<const uint32_t*>(&hh);
          }
          uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
        }
        LSE[((int64_t)b * dm.Hq + hq) * dm.S + srow] = (m_used + log2f(l)) * 0.6931471805599453f;
      }
    }
  }

  // common exit: every role has either finished or given up; tensor memory is released
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && sm.abort && status_word) atomicOr(status_word, HGA_STATUS_WAIT_TIMEOUT);
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, 512);
  }
}

bool attn_fwd_sm100_supported(const Dims& dm) {
  if (dm.flags & HGA_FLAG_GENERIC_KERNELS) return false;
  if (dm.rows % 128 != 0) return false;
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
  if (smem > 227 * 1024) return HGA_ERR_UNSUPPORTED;
  cudaError_t e = cudaFuncSetAttribute(k_attn_fwd_sm100<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return record_cuda(e);
  const int n_mt_item = dm.rows / 128;
  const int units = dm.B * dm.Hkv * dm.NQB * ((n_mt_item + 1) / 2);
  k_attn_fwd_sm100<D><<<units, kFwdThreads, smem, st>>>(mq, mk, mv, group_idx, n_groups, dm, (uint16_t*)O, LSE,
                                                       status_word);
  count_launch();
  return record_cuda(cudaGetLastError());
}

int launch_attn_fwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V,
                          const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                          int32_t* status_word, cudaStream_t st) {
  if (dm.d == 128) return launch_fwd<128>(dm, Q, K, V, group_idx, n_groups, O, LSE, status_word, st);
  return launch_fwd<64>(dm, Q, K, V, group_idx, n_groups, O, LSE, status_word, st);
}

}  // namespace hga
