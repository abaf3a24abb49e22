// Timeline harness for the tensor-core attention kernels (see csrc/hga_trace.cuh): a configuration-3-shaped
// problem (32 query / 8 kv heads, head_dim 128, 2048 active tokens behind 14336 resident ones, 64 routed
// groups per item drawn at random among the candidates), random data, L2 flushed before every repetition.
// Prints the call's time, every traced CTA's place on its SM, and for one CTA the (tag:cycle) records of
// each warp, cycles counted from the CTA's earliest record.
//
//   python -m paper_2607_15105_b200.build --trace          builds paper_2607_15105_b200/hga_trace
//   ./paper_2607_15105_b200/hga_trace <block size of the kernel: 256 forward, 448 band, 512 sweep> [block index]
//
// Tags (see the kernels): 1 set-up done; 2 a producer issued a tile; 3 first GEMMs issued; 5/6/7/8 the
// issuing warp (barrier observed / S issued / dQ or PV issued / dP issued); 11/13/14/15 a row or key
// thread (S observed / second operand observed / results handed over); 20/21 epilogue; 30 role finished, 31
// past the final block barrier.  Sweep only: 4 a dK/dV step issued; 10 delta known; 12/17 a row thread in a
// dK/dV step (S, dP observed / P, dS written); 16/18 a reduction warp (accumulators observed / atomics issued);
// 40-45 the issuing warp before the pairs (Q and dO / K tile / V tile / first K pair arrived, S and dP of a dK/dV
// step issued, its P and dS observed).  Band only: 11/13/15/14 in the statistics warps = dO rows arrived / O tile
// arrived / delta computed / statistics published.
// Built with -DHGA_TRACE; includes the kernels' translation units directly, so it needs no library.
#include <algorithm>
#include <array>
#include <cstdio>
#include <cstdlib>
#include <vector>

#include <cuda_bf16.h>

#include "../csrc/hga_attn_fwd_sm100.cu"
#include "../csrc/hga_attn_bwd_sm100.cu"
#include "../csrc/hga_attn_bwd_band_sm100.cu"
#include "../csrc/hga_tma.cu"

namespace hga {
void count_launch(int, int) {}
int record_cuda(cudaError_t e) { if (e != cudaSuccess) printf("cuda error %s\n", cudaGetErrorString(e)); return e == cudaSuccess ? 0 : -6; }
}
using namespace hga;

int main(int argc, char** argv) {
  const int trace_threads = argc > 1 ? atoi(argv[1]) : 512;
  const int trace_blk = argc > 2 ? atoi(argv[2]) : 300;
  Dims dm{};
  dm.B = 1; dm.Hq = 32; dm.Hkv = 8; dm.G = 4; dm.d = 128; dm.L = 16384; dm.S = 2048; dm.H = dm.L - dm.S;
  dm.c = 64; dm.g = 8; dm.Bq = 64; dm.kc = 16; dm.kg = 4; dm.kge = 4; dm.per = 8; dm.sink = 64; dm.local = 128;
  dm.NQB = dm.S / dm.Bq; dm.Nc = dm.L / dm.c; dm.Ng = dm.L / dm.g; dm.NcS = dm.Nc; dm.NgS = dm.Ng; dm.width = 64; dm.rows = 256; dm.flags = 0;
  dm.scale = 1.f / sqrtf(128.f);
  auto dense = [&](int64_t* s, int heads, int toks) { s[2] = dm.d; s[1] = (int64_t)toks * dm.d; s[0] = (int64_t)heads * toks * dm.d; };
  dense(dm.qs, dm.Hq, dm.S); dense(dm.ks, dm.Hkv, dm.L); dense(dm.vs, dm.Hkv, dm.L); dense(dm.os, dm.Hq, dm.S);
  size_t nq = (size_t)dm.Hq * dm.S * dm.d, nk = (size_t)dm.Hkv * dm.L * dm.d;
  std::vector<__nv_bfloat16> q(nq), k(nk), v(nk);
  srand(3);
  auto rnd = [] { return (rand() % 2001 - 1000) / 500.f; };
  for (auto& x : q) x = __float2bfloat16(rnd());
  for (auto& x : k) x = __float2bfloat16(rnd());
  for (auto& x : v) x = __float2bfloat16(rnd());
  int items = dm.Hkv * dm.NQB;
  std::vector<int> gi(items * 64), ng(items, 64);
  for (int it = 0; it < items; ++it) {
    int qb = it % dm.NQB;
    Window w = window_of(dm, qb);
    int lo = w.se / 8, hi = w.ls / 8;
    std::vector<int> pool;
    // 16 chunks x 4 groups, as the router would select (history mostly)
    while ((int)pool.size() < 64) { int m = lo + rand() % (hi - lo); if (std::find(pool.begin(), pool.end(), m) == pool.end()) pool.push_back(m); }
    std::sort(pool.begin(), pool.end());
    for (int i = 0; i < 64; ++i) gi[it * 64 + i] = pool[i];
  }
  __nv_bfloat16 *dq, *dk, *dv, *dO, *ddO, *ddQ; int *dgi, *dng, *dst; float* dlse; float *ddK, *ddV;
  cudaMalloc(&dq, nq * 2); cudaMalloc(&dk, nk * 2); cudaMalloc(&dv, nk * 2); cudaMalloc(&dO, nq * 2);
  cudaMalloc(&ddO, nq * 2); cudaMalloc(&ddQ, nq * 2); cudaMalloc(&ddK, (size_t)dm.Hkv * dm.S * dm.d * 4); cudaMalloc(&ddV, (size_t)dm.Hkv * dm.S * dm.d * 4);
  cudaMemcpy(ddO, q.data(), nq * 2, cudaMemcpyHostToDevice);
  cudaMalloc(&dgi, gi.size() * 4); cudaMalloc(&dng, ng.size() * 4); cudaMalloc(&dst, 4); cudaMalloc(&dlse, nq / dm.d * 4);
  cudaMemcpy(dq, q.data(), nq * 2, cudaMemcpyHostToDevice); cudaMemcpy(dk, k.data(), nk * 2, cudaMemcpyHostToDevice);
  cudaMemcpy(dv, v.data(), nk * 2, cudaMemcpyHostToDevice); cudaMemcpy(dgi, gi.data(), gi.size() * 4, cudaMemcpyHostToDevice);
  cudaMemcpy(dng, ng.data(), ng.size() * 4, cudaMemcpyHostToDevice); cudaMemset(dst, 0, 4);
  cudaMemcpyToSymbol(g_trace_threads, &trace_threads, 4); cudaMemcpyToSymbol(g_trace_blk, &trace_blk, 4);
  char* flush; cudaMalloc(&flush, 512u << 20);
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  launch_attn_fwd_sm100(dm, dq, dk, dv, dgi, dng, dO, dlse, dst, 0); cudaDeviceSynchronize();
  const bool fwd_mode = trace_threads == 256 || trace_threads == 384;
  for (int rep = 0; rep < 4; ++rep) {
    cudaMemsetAsync(flush, rep, 512u << 20);
    { void* p_; cudaGetSymbolAddress(&p_, g_trace_log); cudaMemsetAsync(p_, 0, sizeof(unsigned) * HGA_TRACE_WARPS * HGA_TRACE_SLOTS); }
    cudaEventRecord(e0);
    int rc = fwd_mode ? launch_attn_fwd_sm100(dm, dq, dk, dv, dgi, dng, dO, dlse, dst, 0)
                      : launch_attn_bwd_sm100(dm, dq, dk, dv, dO, dlse, ddO, dgi, dng, ddQ, ddK, ddV, dst, 0);
    cudaEventRecord(e1);
    cudaError_t ce = cudaDeviceSynchronize();
    float ms; cudaEventElapsedTime(&ms, e0, e1);
    printf("rep %d rc=%d %s  %.1f us\n", rep, rc, cudaGetErrorString(ce), ms * 1e3);
  }
  int st; cudaMemcpy(&st, dst, 4, cudaMemcpyDeviceToHost); printf("status %d\n", st);
  static unsigned long long hc[2048][3]; cudaMemcpyFromSymbol(hc, g_trace_cta, sizeof(hc));
  const int ncta = trace_threads == 448 ? 128 : trace_threads == 384 ? 256 : 512;
  unsigned long long t0 = ~0ull, t1 = 0;
  for (int i = 0; i < ncta; ++i) { t0 = std::min(t0, hc[i][1]); t1 = std::max(t1, hc[i][2]); }
  printf("kernel span by globaltimer: %.1f us\n", (t1 - t0) / 1e3);
  double sum = 0; for (int i = 0; i < ncta; ++i) sum += (hc[i][2] - hc[i][1]) / 1e3; printf("mean CTA duration %.1f us\n", sum / ncta);
  { unsigned sm_sel = (unsigned)hc[trace_blk][0];
    std::vector<std::array<unsigned long long, 2>> vv;
    for (int i = 0; i < ncta; ++i) if (hc[i][0] == sm_sel) vv.push_back({hc[i][1], hc[i][2]});
    std::sort(vv.begin(), vv.end());
    printf("SM %u:", sm_sel);
    for (auto& x : vv) printf(" [%.1f .. %.1f]", (x[0] - t0) / 1e3, (x[1] - t0) / 1e3);
    printf("\n"); }
  static unsigned tl[HGA_TRACE_WARPS][HGA_TRACE_SLOTS];
  cudaMemcpyFromSymbol(tl, g_trace_log, sizeof(tl));
  unsigned base = 0; bool have = false;
  for (int w = 0; w < HGA_TRACE_WARPS && !have; ++w) if (tl[w][0]) { base = tl[w][0] >> 6; have = true; }
  for (int w = 0; w < HGA_TRACE_WARPS; ++w) if (tl[w][0]) base = std::min(base, tl[w][0] >> 6);
  printf("blk %d CTA duration %.2f us\n", trace_blk, (hc[trace_blk][2] - hc[trace_blk][1]) / 1e3);
  for (int w = 0; w < HGA_TRACE_WARPS; ++w) {
    if (!tl[w][0]) continue;
    printf("warp%2d:", w);
    for (int i = 0; i < HGA_TRACE_SLOTS && tl[w][i]; ++i) printf(" %u:%d", tl[w][i] & 63, (int)(((tl[w][i] >> 6) - base) & 0x3ffffff));
    printf("\n");
  }
  return 0;
}
