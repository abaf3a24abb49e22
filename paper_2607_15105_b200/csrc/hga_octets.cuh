// Octet table of an item's routed key set, built by one warp.
//
// The routed set of an item (sink, selected groups, local window) is addressed in octets of 8
// consecutive tokens; oct_row[o] is the first token of octet o, in ascending token order.  The
// group list is validated on the way: an entry must be greater than the last accepted entry
// and lie wholly between the sink and the local window; other entries are skipped and
// reported.  The common case (a valid ascending list) is checked with one coalesced load and a
// warp vote per 32 entries; only a list that fails the vote is walked sequentially.
#pragma once

#include "hga_common.cuh"

namespace hga {

// Must be called by all 32 lanes of one warp.  Returns the number of octets (same value in
// every lane).  *bad_out (lane-uniform) tells whether an entry was skipped.
__device__ inline int build_octet_table(const Dims& dm, const Window& w, const int32_t* __restrict__ gi,
                                        const int32_t* __restrict__ ng_ptr, int* oct_row, bool* bad_out) {
  const unsigned full = 0xffffffffu;
  const int lane = threadIdx.x & 31;
  // the first 64 entries are fetched before the count is known, so the two loads overlap
  const int pre0 = lane < dm.width ? gi[lane] : 0x7fffffff;
  const int pre1 = lane + 32 < dm.width ? gi[lane + 32] : 0x7fffffff;
  int ng = *ng_ptr;
  bool bad = false;
  if (ng > dm.width) { ng = dm.width; bad = true; }
  if (ng < 0) { ng = 0; bad = true; }
  const int opg = dm.g / 8;           // octets per group
  const int n_sink = w.se / 8;
  bool all_ok = true;
  int prev = -1;
  for (int base = 0; base < ng; base += 32) {
    const int i = base + lane;
    const int m = i >= ng ? 0x7fffffff : base == 0 ? pre0 : base == 32 ? pre1 : gi[i];
    int left = __shfl_up_sync(full, m, 1);
    if (lane == 0) left = prev;
    const bool ok = i >= ng || (m > left && (int64_t)m * dm.g >= w.se && ((int64_t)m + 1) * dm.g <= w.ls);
    all_ok = all_ok && __all_sync(full, ok);
    if (all_ok && i < ng)
      for (int u = 0; u < opg; ++u) oct_row[n_sink + i * opg + u] = m * dm.g + 8 * u;
    prev = __shfl_sync(full, m, 31);
  }
  int n_far = n_sink + ng * opg;
  if (!all_ok) {
    bad = true;
    int n = n_sink;
    if (lane == 0) {
      int last = -1;
      for (int i = 0; i < ng; ++i) {
        const int m = gi[i];
        if (m > last && (int64_t)m * dm.g >= w.se && ((int64_t)m + 1) * dm.g <= w.ls) {
          for (int u = 0; u < opg; ++u) oct_row[n++] = m * dm.g + 8 * u;
          last = m;
        }
      }
    }
    n_far = __shfl_sync(full, n, 0);
  }
  for (int o = lane; o < n_sink; o += 32) oct_row[o] = 8 * o;
  const int n_local = (w.p0 + dm.Bq - w.ls + 7) / 8;      // the last octet may be partial (decode shapes)
  for (int o = lane; o < n_local; o += 32) oct_row[n_far + o] = w.ls + 8 * o;
  __syncwarp();
  *bad_out = bad;
  return n_far + n_local;
}

}  // namespace hga
