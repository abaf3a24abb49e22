// C-ABI entry points of libhga: argument validation, stride resolution, dispatch.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <vector>

#include "hga_common.cuh"

namespace hga {

static std::atomic<int64_t> g_launches[HGA_KERNELS_FAMILIES];
static std::atomic<int> g_last_cuda{0};

void count_launch(int family, int n) { g_launches[family].fetch_add(n, std::memory_order_relaxed); }

// Set while hga_step_host calls the exported steps with the library's internal flag bits.
static thread_local bool t_internal_flags = false;
struct InternalFlagsScope {
  InternalFlagsScope() { t_internal_flags = true; }
  ~InternalFlagsScope() { t_internal_flags = false; }
};

int record_cuda(cudaError_t e) {
  if (e == cudaSuccess) return HGA_OK;
  g_last_cuda.store((int)e, std::memory_order_relaxed);
  return HGA_ERR_CUDA;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

static void dense_strides(int64_t* s, int heads, int tokens, int d) {
  s[2] = d;
  s[1] = (int64_t)tokens * d;
  s[0] = (int64_t)heads * tokens * d;
}

// Validates p and fills dm.  Returns an HGA status.
static int resolve(const hga_params* p, Dims& dm) {
  if (!p) return HGA_ERR_NULL;
  if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1) return HGA_ERR_SHAPE;
  if (p->n_q_heads % p->n_kv_heads) return HGA_ERR_SHAPE;
  if (p->head_dim != 64 && p->head_dim != 128) return HGA_ERR_UNSUPPORTED;
  if (p->seg_len < 1 || p->total_len < p->seg_len) return HGA_ERR_SHAPE;
  if (p->group < 1 || p->chunk < p->group || p->chunk % p->group) return HGA_ERR_SHAPE;
  if (p->q_block < 1 || p->seg_len % p->q_block) return HGA_ERR_SHAPE;
  if (!(p->flags & HGA_FLAG_DECODE)) {
    if (p->q_block < p->chunk || p->q_block % p->chunk) return HGA_ERR_SHAPE;
    if ((p->total_len - p->seg_len) % p->q_block) return HGA_ERR_SHAPE;
    if (p->total_len % p->chunk) return HGA_ERR_SHAPE;
  }
  if (p->topk_chunks < 0 || p->topk_groups < 1) return HGA_ERR_SHAPE;
  if (p->sink < 0 || p->local < 0 || p->sink % p->chunk || p->local % p->chunk) return HGA_ERR_SHAPE;
  if (p->chunk / p->group > 64) return HGA_ERR_UNSUPPORTED;
  if (p->topk_chunks > 1024) return HGA_ERR_UNSUPPORTED;
  if ((p->flags & HGA_FLAG_SCORE_MEAN) && (p->flags & HGA_FLAG_SCORE_LSE)) return HGA_ERR_UNSUPPORTED;
  if (p->flags & ~0x7f & ~(t_internal_flags ? kFlagNoPdl : 0)) return HGA_ERR_UNSUPPORTED;   // unknown flag bits
  if ((p->flags & HGA_FLAG_GLOBAL_GROUP_BUDGET) && (int64_t)p->topk_chunks * (p->chunk / p->group) > 4096)
    return HGA_ERR_UNSUPPORTED;
  dm.B = p->batch; dm.Hq = p->n_q_heads; dm.Hkv = p->n_kv_heads; dm.G = dm.Hq / dm.Hkv;
  dm.d = p->head_dim; dm.L = p->total_len; dm.S = p->seg_len; dm.H = dm.L - dm.S;
  dm.c = p->chunk; dm.g = p->group; dm.Bq = p->q_block;
  dm.kc = p->topk_chunks; dm.kg = p->topk_groups; dm.per = dm.c / dm.g;
  dm.kge = dm.kg < dm.per ? dm.kg : dm.per;
  dm.sink = p->sink; dm.local = p->local;
  dm.NQB = dm.S / dm.Bq; dm.Nc = dm.L / dm.c; dm.Ng = dm.L / dm.g;
  if (p->summary_len != 0 && (p->summary_len < p->total_len || p->summary_len % p->chunk)) return HGA_ERR_SHAPE;
  dm.NcS = (p->summary_len ? p->summary_len : dm.L) / dm.c;
  dm.NgS = (p->summary_len ? p->summary_len : dm.L) / dm.g;
  dm.width = dm.kc * dm.kge; dm.rows = dm.G * dm.Bq;
  dm.flags = p->flags;
  dm.scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)dm.d);
  if ((int64_t)dm.B * dm.Hkv * dm.NQB > 0x7fffffff) return HGA_ERR_SHAPE;
  struct { const int64_t* in; int64_t* out; int heads, tokens; } t[4] = {
      {p->q_stride, dm.qs, dm.Hq, dm.S}, {p->k_stride, dm.ks, dm.Hkv, dm.L},
      {p->v_stride, dm.vs, dm.Hkv, dm.L}, {p->o_stride, dm.os, dm.Hq, dm.S}};
  for (auto& e : t) {
    if (e.in[0] == 0 && e.in[1] == 0 && e.in[2] == 0) {
      dense_strides(e.out, e.heads, e.tokens, dm.d);
    } else {
      for (int i = 0; i < 3; ++i) {
        if (e.in[i] < 0 || (e.in[i] % 8)) return HGA_ERR_ALIGN;
        e.out[i] = e.in[i];
      }
      if (e.out[2] < dm.d) return HGA_ERR_SHAPE;
    }
  }
  return HGA_OK;
}

int resolve_params(const hga_params* p, Dims& dm) { return resolve(p, dm); }

size_t route_workspace_bytes(const Dims& dm) {
  // chunk scores fp32 [items, Nc]; with a global group budget also the group scores of the opened
  // chunks, fp32 [items, k_c * (c/g)] (the generic router keeps them there until it selects)
  const size_t per_item = (size_t)dm.Nc + ((dm.flags & HGA_FLAG_GLOBAL_GROUP_BUDGET) ? (size_t)dm.kc * dm.per : 0);
  return (size_t)dm.B * dm.Hkv * dm.NQB * per_item * sizeof(float) + 16;
}

static size_t bwd_delta_bytes(const Dims& dm) {
  return (((size_t)dm.B * dm.Hq * dm.S * sizeof(float)) + 255) & ~(size_t)255;
}

size_t bwd_workspace_bytes(const Dims& dm) {
  // delta = rowsum(dO * O), fp32 [B, Hq, S]; with bf16 gradient outputs also the fp32 dK and dV sums
  size_t bytes = bwd_delta_bytes(dm) + 16;
  if (dm.flags & HGA_FLAG_BWD_BF16_GRADS) bytes += 2 * (size_t)dm.B * dm.Hkv * dm.S * dm.d * sizeof(float);
  return bytes;
}

// Copy streams and events of hga_step_host, created once per device and kept until exit.
struct StepPipe {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
  std::vector<cudaEvent_t> in_done, comp_done;
};

static StepPipe* step_pipe(int n_pairs) {
  static std::mutex mu;
  static std::map<int, StepPipe> pipes;
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  StepPipe& sp = pipes[dev];
  if (!sp.in) {
    if (cudaStreamCreateWithFlags(&sp.in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&sp.out, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&sp.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&sp.join, cudaEventDisableTiming) != cudaSuccess) {
      record_cuda(cudaGetLastError());
      return nullptr;
    }
  }
  while ((int)sp.in_done.size() < n_pairs) {
    cudaEvent_t a = nullptr, b = nullptr;
    if (cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) {
      record_cuda(cudaGetLastError());
      return nullptr;
    }
    sp.in_done.push_back(a);
    sp.comp_done.push_back(b);
  }
  return &sp;
}

}  // namespace hga

using namespace hga;

extern "C" {

int hga_version(void) { return HGA_VERSION; }

int hga_last_cuda_error(void) { return g_last_cuda.load(); }

int64_t hga_kernel_launch_count(void) {
  int64_t n = 0;
  for (auto& c : g_launches) n += c.load();
  return n;
}

int64_t hga_kernel_launch_count_by_family(int family) {
  if (family < 0 || family >= HGA_KERNELS_FAMILIES) return -1;
  return g_launches[family].load();
}

const char* hga_status_string(int s) {
  switch (s) {
    case HGA_OK: return "ok";
    case HGA_ERR_NULL: return "a required pointer is NULL";
    case HGA_ERR_SHAPE: return "sizes violate the shape rules of hga_params";
    case HGA_ERR_ALIGN: return "pointer not 16-byte aligned or stride not a multiple of 8 elements";
    case HGA_ERR_UNSUPPORTED: return "unsupported head_dim, size or device";
    case HGA_ERR_WORKSPACE: return "workspace missing or too small";
    case HGA_ERR_CUDA: return "a CUDA call failed (see hga_last_cuda_error)";
    default: return "unknown status";
  }
}

int hga_workspace_bytes(const hga_params* p, size_t* route_bytes, size_t* bwd_bytes) {
  Dims dm;
  int rc = resolve(p, dm);
  if (rc) return rc;
  if (route_bytes) *route_bytes = route_workspace_bytes(dm);
  if (bwd_bytes) *bwd_bytes = bwd_workspace_bytes(dm);
  return HGA_OK;
}

int hga_build_summaries(const hga_params* p, const void* K, int32_t tok_begin, int32_t tok_end,
                        void* chunk_sum, void* group_sum, void* stream) {
  Dims dm;
  int rc = resolve(p, dm);
  if (rc) return rc;
  if (!K || !chunk_sum || !group_sum) return HGA_ERR_NULL;
  if (!aligned16(K) || !aligned16(chunk_sum) || !aligned16(group_sum)) return HGA_ERR_ALIGN;
  if (tok_begin < 0 || tok_end > dm.L || tok_begin > tok_end || tok_begin % dm.c || tok_end % dm.c)
    return HGA_ERR_SHAPE;
  if (tok_begin == tok_end) return HGA_OK;
  return launch_build_summaries(dm, K, tok_begin, tok_end, chunk_sum, group_sum, (cudaStream_t)stream);
}

int hga_route(const hga_params* p, const void* Q, const void* chunk_sum, const void* group_sum,
              int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, float* chunk_scores,
              float* group_scores, void* workspace, size_t workspace_bytes, void* stream) {
  Dims dm;
  int rc = resolve(p, dm);
  if (rc) return rc;
  if (!Q || !chunk_sum || !group_sum || !n_groups) return HGA_ERR_NULL;
  if (dm.kc > 0 && (!chunk_idx || !group_idx)) return HGA_ERR_NULL;   // zero-width lists may be NULL
  if (!aligned16(Q) || !aligned16(chunk_sum) || !aligned16(group_sum)) return HGA_ERR_ALIGN;
  if (!workspace || workspace_bytes < route_workspace_bytes(dm)) return HGA_ERR_WORKSPACE;
  if (!aligned16(workspace)) return HGA_ERR_ALIGN;
  if (route_sm100_supported(dm)) {
    rc = launch_route_sm100(dm, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, chunk_scores,
                            group_scores, (cudaStream_t)stream);
    if (rc != HGA_ERR_UNSUPPORTED) return rc;
  }
  return launch_route_generic(dm, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups,
                              chunk_scores, group_scores, workspace, (cudaStream_t)stream);
}

int hga_attn_fwd(const hga_params* p, const void* Q, const void* K, const void* V,
                 const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                 int32_t* status_word, void* stream) {
  Dims dm;
  int rc = resolve(p, dm);
  if (rc) return rc;
  if (!Q || !K || !V || (!group_idx && dm.width > 0) || !n_groups || !O || !LSE) return HGA_ERR_NULL;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return HGA_ERR_ALIGN;
  if (attn_fwd_sm100_supported(dm)) {
    rc = launch_attn_fwd_sm100(dm, Q, K, V, group_idx, n_groups, O, LSE, status_word, (cudaStream_t)stream);
    if (rc != HGA_ERR_UNSUPPORTED) return rc;
  }
  return launch_attn_fwd_generic(dm, Q, K, V, group_idx, n_groups, O, LSE, status_word,
                                 (cudaStream_t)stream);
}

int hga_attn_bwd(const hga_params* p, const void* Q, const void* K, const void* V, const void* O,
                 const float* LSE, const void* dO, const int32_t* group_idx,
                 const int32_t* n_groups, void* dQ, void* dK_out, void* dV_out, void* workspace,
                 size_t workspace_bytes, int32_t* status_word, void* stream) {
  Dims dm;
  int rc = resolve(p, dm);
  if (rc) return rc;
  if (dm.flags & HGA_FLAG_DECODE) return HGA_ERR_UNSUPPORTED;     // forward only
  const bool bf16_grads = (dm.flags & HGA_FLAG_BWD_BF16_GRADS) != 0;
  if (bf16_grads && (dm.flags & HGA_FLAG_BWD_ACCUMULATE)) return HGA_ERR_UNSUPPORTED;
  float* dK = (float*)dK_out;
  float* dV = (float*)dV_out;
  if (!Q || !K || !V || !O || !LSE || !dO || (!group_idx && dm.width > 0) || !n_groups || !dQ || !dK || !dV)
    return HGA_ERR_NULL;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) ||
      !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
    return HGA_ERR_ALIGN;
  if (!workspace || workspace_bytes < bwd_workspace_bytes(dm)) return HGA_ERR_WORKSPACE;
  if (!aligned16(workspace)) return HGA_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  const bool zero_grads = !(dm.flags & HGA_FLAG_BWD_ACCUMULATE);
  const size_t n_kv = (size_t)dm.B * dm.Hkv * dm.S * dm.d;
  if (bf16_grads) {
    // the sums over query blocks run in fp32 in the workspace and are rounded once at the end, by one
    // conversion launch for both tensors
    dK = (float*)((char*)workspace + bwd_delta_bytes(dm));
    dV = dK + n_kv;
  }
  rc = HGA_ERR_UNSUPPORTED;
  bool tensor_path = false;
  if (attn_bwd_sm100_supported(dm)) {
    // its band kernel stores every row of dK/dV (or adds to it); UNSUPPORTED is returned before any launch
    rc = launch_attn_bwd_sm100(dm, Q, K, V, O, LSE, dO, group_idx, n_groups, dQ, dK, dV, status_word, st);
    tensor_path = rc == HGA_OK;
  }
  if (rc == HGA_ERR_UNSUPPORTED) {
    if (zero_grads) {
      rc = record_cuda(cudaMemsetAsync(dK, 0, n_kv * sizeof(float), st));
      if (rc) return rc;
      rc = record_cuda(cudaMemsetAsync(dV, 0, n_kv * sizeof(float), st));
      if (rc) return rc;
    }
    rc = launch_attn_bwd_generic(dm, Q, K, V, O, LSE, dO, group_idx, n_groups, dQ, dK, dV,
                                 (float*)workspace, status_word, st);
  }
  if (rc || !bf16_grads) return rc;
  return launch_grads_to_bf16(dK, dK_out, dV_out, n_kv, tensor_path && !(dm.flags & kFlagNoPdl), st);
}

int hga_step_arena_bytes(const hga_params* p, size_t* bytes) {
  Dims dm;
  int rc = resolve(p, dm);
  if (rc) return rc;
  if (!bytes) return HGA_ERR_NULL;
  size_t q = (size_t)dm.B * dm.Hq * dm.S * dm.d * 2;           // Q, dO, O, dQ (bf16)
  size_t kv32 = (size_t)dm.B * dm.Hkv * dm.S * dm.d * 4;       // dK, dV (fp32)
  size_t items = (size_t)dm.B * dm.Hkv * dm.NQB;
  size_t idx = items * (dm.kc + dm.width + 1) * 4 + 64;
  size_t lse = (size_t)dm.B * dm.Hq * dm.S * 4;
  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  *bytes = 4 * up(q) + 2 * up(kv32) + up(idx) + up(lse) +
           up(route_workspace_bytes(dm)) + up(bwd_workspace_bytes(dm)) + 256;
  return HGA_OK;
}

int hga_step_host(const hga_params* p, const void* Q_host, const void* Kseg_host,
                  const void* Vseg_host, const void* dO_host, void* K_dev, void* V_dev,
                  void* chunk_sum, void* group_sum, void* O_host, void* dQ_host, float* dK_host,
                  float* dV_host, void* arena, size_t arena_bytes, int32_t* status_word,
                  void* stream) {
  Dims dm;
  int rc = resolve(p, dm);
  if (rc) return rc;
  if (dm.flags & (HGA_FLAG_DECODE | HGA_FLAG_BWD_BF16_GRADS)) return HGA_ERR_UNSUPPORTED;
  if (!Q_host || !Kseg_host || !Vseg_host || !K_dev || !V_dev || !chunk_sum || !group_sum ||
      !O_host || !arena)
    return HGA_ERR_NULL;
  const bool bwd = dO_host != nullptr;
  if (bwd && (!dQ_host || !dK_host || !dV_host)) return HGA_ERR_NULL;
  // this convenience call works on dense tensors only
  const int64_t zero[3] = {0, 0, 0};
  if (memcmp(p->q_stride, zero, sizeof zero) || memcmp(p->k_stride, zero, sizeof zero) ||
      memcmp(p->v_stride, zero, sizeof zero) || memcmp(p->o_stride, zero, sizeof zero))
    return HGA_ERR_UNSUPPORTED;
  size_t need = 0;
  hga_step_arena_bytes(p, &need);
  if (arena_bytes < need) return HGA_ERR_WORKSPACE;
  if (!aligned16(arena) || !aligned16(K_dev) || !aligned16(V_dev)) return HGA_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;

  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  char* a = (char*)(((uintptr_t)arena + 255) & ~(uintptr_t)255);
  auto take = [&](size_t n) { char* r = a; a += up(n); return (void*)r; };
  size_t qb = (size_t)dm.B * dm.Hq * dm.S * dm.d * 2;
  size_t kv32 = (size_t)dm.B * dm.Hkv * dm.S * dm.d * 4;
  size_t items = (size_t)dm.B * dm.Hkv * dm.NQB;
  char* dQin = (char*)take(qb); char* ddO = (char*)take(qb); char* dOut = (char*)take(qb); char* ddQ = (char*)take(qb);
  char* ddK = (char*)take(kv32); char* ddV = (char*)take(kv32);
  int32_t* cidx = (int32_t*)take(items * (dm.kc + dm.width + 1) * 4 + 64);
  int32_t* gidx = cidx + items * dm.kc;
  int32_t* ng = gidx + items * dm.width;
  float* lse = (float*)take((size_t)dm.B * dm.Hq * dm.S * 4);
  void* rws = take(route_workspace_bytes(dm));
  void* bws = take(bwd_workspace_bytes(dm));

  // The (batch, kv head) pairs are independent problems (routing, attention and dK/dV never cross kv
  // heads), so the step runs as a pipeline over them: while one pair's kernels run, the next pair's
  // inputs arrive on a copy stream and the previous pair's results leave on another (the two copy
  // directions overlap as well).  Everything is ordered after the work already queued on `stream`,
  // and `stream` ends up waiting for the last copy, so the caller sees one stream as before.
  StepPipe* pipe = step_pipe(dm.B * dm.Hkv);
  if (!pipe) return HGA_ERR_CUDA;
  hga_params pc = *p;                                // one (batch, kv head): B = 1, Hkv = 1, Hq = G, dense
  pc.batch = 1;
  pc.n_q_heads = dm.G;
  pc.n_kv_heads = 1;
  pc.flags |= kFlagNoPdl;                            // this pipeline is bound by the host link (see hga_common.cuh)
  InternalFlagsScope internal;                       // lets the exported steps below accept that bit
  const size_t q_c = (size_t)dm.G * dm.S * dm.d * 2;           // bytes of one pair's Q / dO / O / dQ rows
  const size_t kvseg_c = (size_t)dm.S * dm.d * 2, kv32_c = (size_t)dm.S * dm.d * 4;
  const size_t kv_c = (size_t)dm.L * dm.d * 2;                 // one (batch, kv head) of the resident K / V
  const size_t hist = (size_t)dm.H * dm.d * 2;
  const size_t cs_c = (size_t)dm.NcS * dm.d * 2, gs_c = (size_t)dm.NgS * dm.d * 2;
#define HGA_TRY(x) do { rc = (x); if (rc) return rc; } while (0)
  HGA_TRY(record_cuda(cudaEventRecord(pipe->fork, st)));
  HGA_TRY(record_cuda(cudaStreamWaitEvent(pipe->in, pipe->fork, 0)));
  HGA_TRY(record_cuda(cudaStreamWaitEvent(pipe->out, pipe->fork, 0)));
  const int n_pairs = dm.B * dm.Hkv;
  for (int c = 0; c < n_pairs; ++c) {
    // host -> device: this pair's Q, (dO), and its active-segment K/V rows straight behind the history
    HGA_TRY(record_cuda(cudaMemcpyAsync(dQin + c * q_c, (const char*)Q_host + c * q_c, q_c, cudaMemcpyHostToDevice, pipe->in)));
    if (bwd)
      HGA_TRY(record_cuda(cudaMemcpyAsync(ddO + c * q_c, (const char*)dO_host + c * q_c, q_c, cudaMemcpyHostToDevice, pipe->in)));
    HGA_TRY(record_cuda(cudaMemcpyAsync((char*)K_dev + c * kv_c + hist, (const char*)Kseg_host + c * kvseg_c, kvseg_c,
                                        cudaMemcpyHostToDevice, pipe->in)));
    HGA_TRY(record_cuda(cudaMemcpyAsync((char*)V_dev + c * kv_c + hist, (const char*)Vseg_host + c * kvseg_c, kvseg_c,
                                        cudaMemcpyHostToDevice, pipe->in)));
    HGA_TRY(record_cuda(cudaEventRecord(pipe->in_done[c], pipe->in)));
    HGA_TRY(record_cuda(cudaStreamWaitEvent(st, pipe->in_done[c], 0)));

    const char* Kc = (const char*)K_dev + c * kv_c;
    const char* Vc = (const char*)V_dev + c * kv_c;
    char* csc = (char*)chunk_sum + c * cs_c;
    char* gsc = (char*)group_sum + c * gs_c;
    int32_t* gic = gidx + (size_t)c * dm.NQB * dm.width;
    int32_t* ngc = ng + (size_t)c * dm.NQB;
    float* lsec = lse + (size_t)c * dm.G * dm.S;
    HGA_TRY(hga_build_summaries(&pc, Kc, dm.H, dm.L, csc, gsc, stream));
    HGA_TRY(hga_route(&pc, dQin + c * q_c, csc, gsc, cidx + (size_t)c * dm.NQB * dm.kc, gic, ngc, nullptr, nullptr, rws,
                      route_workspace_bytes(dm), stream));
    HGA_TRY(hga_attn_fwd(&pc, dQin + c * q_c, Kc, Vc, gic, ngc, dOut + c * q_c, lsec, status_word, stream));
    if (bwd)
      HGA_TRY(hga_attn_bwd(&pc, dQin + c * q_c, Kc, Vc, dOut + c * q_c, lsec, ddO + c * q_c, gic, ngc, ddQ + c * q_c,
                           (float*)(ddK + c * kv32_c), (float*)(ddV + c * kv32_c), bws, bwd_workspace_bytes(dm),
                           status_word, stream));
    HGA_TRY(record_cuda(cudaEventRecord(pipe->comp_done[c], st)));
    HGA_TRY(record_cuda(cudaStreamWaitEvent(pipe->out, pipe->comp_done[c], 0)));
    // device -> host: this pair's results
    HGA_TRY(record_cuda(cudaMemcpyAsync((char*)O_host + c * q_c, dOut + c * q_c, q_c, cudaMemcpyDeviceToHost, pipe->out)));
    if (bwd) {
      HGA_TRY(record_cuda(cudaMemcpyAsync((char*)dQ_host + c * q_c, ddQ + c * q_c, q_c, cudaMemcpyDeviceToHost, pipe->out)));
      HGA_TRY(record_cuda(cudaMemcpyAsync((char*)dK_host + c * kv32_c, ddK + c * kv32_c, kv32_c, cudaMemcpyDeviceToHost, pipe->out)));
      HGA_TRY(record_cuda(cudaMemcpyAsync((char*)dV_host + c * kv32_c, ddV + c * kv32_c, kv32_c, cudaMemcpyDeviceToHost, pipe->out)));
    }
  }
  HGA_TRY(record_cuda(cudaEventRecord(pipe->join, pipe->out)));
  HGA_TRY(record_cuda(cudaStreamWaitEvent(st, pipe->join, 0)));
#undef HGA_TRY
  return HGA_OK;
}

int hga_tbptt_walk(const hga_params* p, const void* Q, const void* K, const void* V, const void* dO,
                   void* chunk_sum, void* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                   int32_t* n_groups, void* O, float* LSE, void* dQ, void* dK, void* dV,
                   void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream) {
  if (!p) return HGA_ERR_NULL;
  if (p->flags & HGA_FLAG_DECODE) return HGA_ERR_UNSUPPORTED;
  if (p->seg_len < 1 || p->total_len < p->seg_len || p->total_len % p->seg_len) return HGA_ERR_SHAPE;
  hga_params full = *p;                 // the last segment's problem: validates shapes, resolves the full-length strides
  full.summary_len = 0;
  Dims dmf;
  int rc = resolve(&full, dmf);
  if (rc) return rc;
  if (!Q || !K || !V || !chunk_sum || !group_sum || !group_idx || !n_groups || !O || !LSE || !workspace)
    return HGA_ERR_NULL;
  if (dmf.kc > 0 && !chunk_idx) return HGA_ERR_NULL;
  const bool bwd = dO != nullptr;
  if (bwd && (!dQ || !dK || !dV)) return HGA_ERR_NULL;
  const size_t route_ws = route_workspace_bytes(dmf), bwd_ws = bwd_workspace_bytes(dmf);
  const size_t route_ws_up = (route_ws + 255) & ~(size_t)255;
  if (workspace_bytes < route_ws_up + bwd_ws) return HGA_ERR_WORKSPACE;
  const int S = p->seg_len, n_seg = p->total_len / S;
  // full-length strides (elements): dmf's token counts are those of the last segment (S active rows,
  // L keys), so the Q/O strides are rebuilt for L rows when the caller gave none
  hga_params ps = *p;
  ps.summary_len = p->total_len;
  const int64_t zero[3] = {0, 0, 0};
  const int64_t d = p->head_dim, L = p->total_len;
  auto fill = [&](int64_t* s, const int64_t* given, int heads) {
    if (memcmp(given, zero, sizeof zero) == 0) { s[2] = d; s[1] = L * d; s[0] = (int64_t)heads * L * d; }
  };
  fill(ps.q_stride, p->q_stride, p->n_q_heads);
  fill(ps.o_stride, p->o_stride, p->n_q_heads);
  fill(ps.k_stride, p->k_stride, p->n_kv_heads);
  fill(ps.v_stride, p->v_stride, p->n_kv_heads);
  const size_t items = (size_t)dmf.B * dmf.Hkv * dmf.NQB;
  const size_t lse_seg = (size_t)dmf.B * dmf.Hq * S, kv_seg = (size_t)dmf.B * dmf.Hkv * S * dmf.d;
  const size_t grad_bytes = (p->flags & HGA_FLAG_BWD_BF16_GRADS) ? 2 : 4;    // element size of dK/dV
  // The backward of segment s depends on that segment's forward only, and the forward chain of segment
  // s+1 (summaries -> route -> forward) on nothing the backward writes: the backward calls go to a
  // second, library-owned stream (the one hga_step_host copies in on), so the two chains fill each
  // other's idle SMs (kernel tails, the one-wave router).  The caller's stream is joined at the end.
  cudaStream_t st = (cudaStream_t)stream;
  StepPipe* pipe = bwd ? step_pipe(n_seg) : nullptr;
  if (bwd && !pipe) return HGA_ERR_CUDA;
  if (bwd) {
    rc = record_cuda(cudaEventRecord(pipe->fork, st));
    if (rc) return rc;
    rc = record_cuda(cudaStreamWaitEvent(pipe->in, pipe->fork, 0));
    if (rc) return rc;
  }
  for (int s = 0; s < n_seg; ++s) {
    ps.total_len = (s + 1) * S;
    const int64_t q_off = (int64_t)s * S * ps.q_stride[2] * 2, o_off = (int64_t)s * S * ps.o_stride[2] * 2;   // bytes
    const char* Qs = (const char*)Q + q_off;
    char* Os = (char*)O + o_off;
    int32_t* ci = chunk_idx ? chunk_idx + s * items * dmf.kc : nullptr;
    int32_t* gi = group_idx + s * items * dmf.width;
    int32_t* ng = n_groups + s * items;
    float* lse = LSE + s * lse_seg;
    rc = hga_build_summaries(&ps, K, s * S, (s + 1) * S, chunk_sum, group_sum, stream);
    if (rc) return rc;
    rc = hga_route(&ps, Qs, chunk_sum, group_sum, ci, gi, ng, nullptr, nullptr, workspace, route_ws, stream);
    if (rc) return rc;
    rc = hga_attn_fwd(&ps, Qs, K, V, gi, ng, Os, lse, status_word, stream);
    if (rc) return rc;
    if (bwd) {
      rc = record_cuda(cudaEventRecord(pipe->in_done[s], st));          // forward of segment s queued
      if (rc) return rc;
      rc = record_cuda(cudaStreamWaitEvent(pipe->in, pipe->in_done[s], 0));
      if (rc) return rc;
      rc = hga_attn_bwd(&ps, Qs, K, V, Os, lse, (const char*)dO + o_off, gi, ng, (char*)dQ + q_off,
                        (char*)dK + s * kv_seg * grad_bytes, (char*)dV + s * kv_seg * grad_bytes,
                        (char*)workspace + route_ws_up, bwd_ws, status_word, pipe->in);
      if (rc) return rc;
    }
  }
  if (bwd) {
    rc = record_cuda(cudaEventRecord(pipe->join, pipe->in));
    if (rc) return rc;
    rc = record_cuda(cudaStreamWaitEvent(st, pipe->join, 0));
    if (rc) return rc;
  }
  return HGA_OK;
}

// Batch-1 parameters of sequence i of a packed variable-length batch (token-major tensors).
static int varlen_params(const hga_params* p, int32_t n_seq, const int32_t* cu_q, const int32_t* cu_k, int i,
                         hga_params& ps) {
  const int64_t S = (int64_t)cu_q[i + 1] - cu_q[i], L = (int64_t)cu_k[i + 1] - cu_k[i];
  const int64_t L_all = cu_k[n_seq];
  if (S < 1 || L < S || cu_q[i] < 0 || cu_k[i] < 0) return HGA_ERR_SHAPE;
  if (p->chunk < 1 || p->q_block < 1 || cu_k[i] % p->chunk || cu_q[i] % p->q_block) return HGA_ERR_SHAPE;
  ps = *p;
  ps.batch = 1;
  ps.total_len = (int32_t)L;
  ps.seg_len = (int32_t)S;
  ps.summary_len = (int32_t)L_all;
  const int64_t d = p->head_dim;
  const int64_t qs[3] = {S * p->n_q_heads * d, d, (int64_t)p->n_q_heads * d};
  const int64_t ks[3] = {L * p->n_kv_heads * d, d, (int64_t)p->n_kv_heads * d};
  for (int a = 0; a < 3; ++a) { ps.q_stride[a] = ps.o_stride[a] = qs[a]; ps.k_stride[a] = ps.v_stride[a] = ks[a]; }
  return HGA_OK;
}

int hga_varlen_workspace_bytes(const hga_params* p, int32_t n_seq, const int32_t* cu_q, const int32_t* cu_k,
                               size_t* bytes) {
  if (!p || !cu_q || !cu_k || !bytes) return HGA_ERR_NULL;
  if (n_seq < 1 || cu_q[0] != 0 || cu_k[0] != 0) return HGA_ERR_SHAPE;
  if (p->flags & HGA_FLAG_DECODE) return HGA_ERR_UNSUPPORTED;
  size_t route_max = 0, bwd_max = 0;
  for (int i = 0; i < n_seq; ++i) {
    hga_params ps;
    int rc = varlen_params(p, n_seq, cu_q, cu_k, i, ps);
    if (rc) return rc;
    Dims dm;
    rc = resolve(&ps, dm);
    if (rc) return rc;
    route_max = std::max(route_max, route_workspace_bytes(dm));
    bwd_max = std::max(bwd_max, bwd_workspace_bytes(dm));
  }
  // two lanes (see hga_varlen_step): each has its own routing and backward scratch
  *bytes = 2 * (((route_max + 255) & ~(size_t)255) + ((bwd_max + 255) & ~(size_t)255));
  return HGA_OK;
}

int hga_varlen_step(const hga_params* p, int32_t n_seq, const int32_t* cu_q, const int32_t* cu_k,
                    const void* Q, const void* K, const void* V, const void* dO, void* chunk_sum,
                    void* group_sum, int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, void* O,
                    float* LSE, void* dQ, void* dK, void* dV, void* workspace, size_t workspace_bytes,
                    int32_t* status_word, void* stream) {
  size_t need = 0;
  int rc = hga_varlen_workspace_bytes(p, n_seq, cu_q, cu_k, &need);     // validates every sequence
  if (rc) return rc;
  if (!Q || !K || !V || !chunk_sum || !group_sum || !group_idx || !n_groups || !O || !LSE || !workspace)
    return HGA_ERR_NULL;
  if (p->topk_chunks > 0 && !chunk_idx) return HGA_ERR_NULL;
  const bool bwd = dO != nullptr;
  if (bwd && (!dQ || !dK || !dV)) return HGA_ERR_NULL;
  if (workspace_bytes < need) return HGA_ERR_WORKSPACE;
  const int64_t d = p->head_dim, Hq = p->n_q_heads, Hkv = p->n_kv_heads;
  const int per = p->chunk / p->group;
  const int kge = p->topk_groups < per ? p->topk_groups : per;
  const size_t grad_bytes = (p->flags & HGA_FLAG_BWD_BF16_GRADS) ? 2 : 4;
  // The sequences are independent problems.  A short sequence fills only part of the GPU (its kernels are
  // one or two CTAs per SM wide and a few waves deep at most), so the sequences go alternately to two
  // library-owned streams ("lanes"), each with its own half of the workspace: the kernels of two sequences
  // run side by side.  Both lanes start behind the work already queued on `stream` and are joined back into
  // it before the call returns.
  cudaStream_t st = (cudaStream_t)stream;
  StepPipe* pipe = n_seq > 1 ? step_pipe(1) : nullptr;
  if (n_seq > 1 && !pipe) return HGA_ERR_CUDA;
  cudaStream_t lanes[2] = {pipe ? pipe->in : st, pipe ? pipe->out : st};
  if (pipe) {
    rc = record_cuda(cudaEventRecord(pipe->fork, st));
    if (rc) return rc;
    for (int l = 0; l < 2; ++l) {
      rc = record_cuda(cudaStreamWaitEvent(lanes[l], pipe->fork, 0));
      if (rc) return rc;
    }
  }
  const size_t lane_bytes = need / 2;
  for (int i = 0; i < n_seq; ++i) {
    hga_params ps;
    varlen_params(p, n_seq, cu_q, cu_k, i, ps);
    Dims dm;
    rc = resolve(&ps, dm);
    if (rc) return rc;
    void* lane_stream = (void*)lanes[i & 1];
    char* ws = (char*)workspace + (size_t)(i & 1) * lane_bytes;
    const int64_t q0 = cu_q[i], k0 = cu_k[i];
    const char* Qi = (const char*)Q + q0 * Hq * d * 2;
    const char* Ki = (const char*)K + k0 * Hkv * d * 2;
    const char* Vi = (const char*)V + k0 * Hkv * d * 2;
    char* Oi = (char*)O + q0 * Hq * d * 2;
    char* csi = (char*)chunk_sum + (k0 / p->chunk) * d * 2;
    char* gsi = (char*)group_sum + (k0 / p->group) * d * 2;
    const int64_t item0 = Hkv * (q0 / p->q_block);
    int32_t* ci = chunk_idx ? chunk_idx + item0 * p->topk_chunks : nullptr;
    int32_t* gi = group_idx + item0 * p->topk_chunks * kge;
    int32_t* ng = n_groups + item0;
    float* lse = LSE + Hq * q0;
    const size_t route_ws = route_workspace_bytes(dm), bwd_ws = bwd_workspace_bytes(dm);
    rc = hga_build_summaries(&ps, Ki, dm.H, dm.L, csi, gsi, lane_stream);
    if (rc) return rc;
    rc = hga_route(&ps, Qi, csi, gsi, ci, gi, ng, nullptr, nullptr, ws, route_ws, lane_stream);
    if (rc) return rc;
    rc = hga_attn_fwd(&ps, Qi, Ki, Vi, gi, ng, Oi, lse, status_word, lane_stream);
    if (rc) return rc;
    if (bwd) {
      rc = hga_attn_bwd(&ps, Qi, Ki, Vi, Oi, lse, (const char*)dO + q0 * Hq * d * 2, gi, ng,
                        (char*)dQ + q0 * Hq * d * 2, (char*)dK + Hkv * d * q0 * grad_bytes,
                        (char*)dV + Hkv * d * q0 * grad_bytes,
                        ws + ((route_ws + 255) & ~(size_t)255), bwd_ws, status_word, lane_stream);
      if (rc) return rc;
    }
  }
  if (pipe) {
    // `stream` waits for both lanes (one event each; recorded and waited on in turn)
    for (int l = 0; l < 2; ++l) {
      rc = record_cuda(cudaEventRecord(pipe->join, lanes[l]));
      if (rc) return rc;
      rc = record_cuda(cudaStreamWaitEvent(st, pipe->join, 0));
      if (rc) return rc;
    }
  }
  return HGA_OK;
}

}  // extern "C"
