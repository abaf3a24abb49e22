/*
 * libhga -- Hierarchical Global Attention (HGA) hot path for NVIDIA B200 (sm_100a).
 *
 * C ABI of the four steps of one HGA attention-layer step as stated in "Long-Context
 * Fine-Tuning with Limited VRAM", Section 2.1 (exact-token hierarchical routing) and
 * Section 2.2 (segment-wise backward):
 *
 *   hga_build_summaries  two levels of key summaries from the projected keys   (Sec. 2.1)
 *   hga_route            chunk selection, then group selection                 (Sec. 2.1, items 1-2)
 *   hga_attn_fwd         exact-token softmax attention over the routed set     (Sec. 2.1, item 3)
 *   hga_attn_bwd         its backward; history K/V are detached constants      (Sec. 2.1 last par., Sec. 2.2)
 *
 * General rules
 *   - Unless a parameter says "host", every data pointer is a DEVICE pointer owned by the
 *     caller.  The library allocates and frees no device memory, never synchronises the
 *     device, and launches on the `stream` it is given (a cudaStream_t passed as void*).
 *   - Every call returns an int status: HGA_OK (0) or a negative HGA_ERR_* code.  On an
 *     error nothing has been launched.  hga_status_string() names a code.
 *   - bf16 data are raw 16-bit patterns.  The innermost (head_dim) axis is contiguous.
 *
 * Shapes (B batch, Hq/Hkv query/kv heads, G = Hq/Hkv, d head_dim, L total tokens,
 * S active-segment tokens, H = L - S detached history, c chunk, g group, Bq query block,
 * NQB = S/Bq):
 *   Q, O, dO, dQ  bf16 [B, Hq,  S, d]   row t is absolute position H + t
 *   K, V          bf16 [B, Hkv, L, d]   history rows first, the active segment last
 *   chunk_sum     bf16 [B, Hkv, L/c, d] group_sum bf16 [B, Hkv, L/g, d]        (dense)
 *   chunk_idx     int32 [B, Hkv, NQB, k_c]            ascending chunk ids, -1 padded
 *   group_idx     int32 [B, Hkv, NQB, k_c * kg_eff]   ascending global group ids (group m
 *                 covers tokens [m*g, (m+1)*g)), -1 padded; kg_eff = min(k_g, c/g)
 *   n_groups      int32 [B, Hkv, NQB]                 number of real entries in group_idx
 *   LSE           fp32 [B, Hq, S]  natural-log sum of exp of the scaled logits
 *   dK, dV        fp32 [B, Hkv, S, d]  rows of the ACTIVE segment only (row t = position H + t)
 *
 * One routing decision is taken per "item" (b, kv head, query block) and shared by the
 * G*Bq query rows of that item.  Window geometry of query block qb, p0 = H + qb*Bq:
 *   local start ls = max(0, floor((p0 - local)/c)*c);  sink end se = min(sink, ls);
 *   candidate chunks j: se <= j*c and (j+1)*c <= ls;
 *   routed set = [0, se)  U  selected groups  U  [ls, p0 + Bq), causal inside the block.
 */
#ifndef HGA_H
#define HGA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HGA_VERSION 100

#if defined(__GNUC__)
#define HGA_API __attribute__((visibility("default")))
#else
#define HGA_API
#endif

/* status codes */
#define HGA_OK 0
#define HGA_ERR_NULL (-1)        /* a required pointer is NULL */
#define HGA_ERR_SHAPE (-2)       /* sizes violate the divisibility / range rules below */
#define HGA_ERR_ALIGN (-3)       /* pointer not 16-byte aligned or stride not a multiple of 8 */
#define HGA_ERR_UNSUPPORTED (-4) /* head_dim / device not supported */
#define HGA_ERR_WORKSPACE (-5)   /* workspace missing or too small */
#define HGA_ERR_CUDA (-6)        /* a CUDA call failed; see hga_last_cuda_error() */

/* hga_params.flags */
#define HGA_FLAG_BWD_ACCUMULATE 1  /* hga_attn_bwd adds into dK/dV instead of overwriting */
#define HGA_FLAG_GENERIC_KERNELS 2 /* use the shape-generic CUDA-core kernels even where a
                                      tensor-core kernel exists (debugging / cross-checks) */
#define HGA_FLAG_GLOBAL_GROUP_BUDGET 4 /* hga_route: Section 2.1 item 2 read as ONE budget over all
                                          selected chunks: the (selected chunks * kg_eff) best groups of
                                          all opened chunks together, instead of the kg_eff best inside
                                          each chunk.  Needs k_c * (c/g) <= 4096. */
#define HGA_FLAG_SCORE_MEAN 8  /* hga_route: a query block's score of a summary is the MEAN over its
                                  G*Bq rows of the dot product (= the mean query row's dot product)
                                  instead of the maximum (Section 2.1 item 1 leaves the reduction open) */
#define HGA_FLAG_SCORE_LSE 16  /* hga_route: the score is ln sum_rows exp(dot product).  At most one of
                                  SCORE_MEAN / SCORE_LSE may be set (else HGA_ERR_UNSUPPORTED). */
#define HGA_FLAG_DECODE 32     /* generation-shaped use (Sections 1 and 5 name generation as a use of the
                                  same routed attention): the query block is the few newest tokens
                                  behind a history of any length.  Lifts the rules Bq % c == 0,
                                  (L - S) % Bq == 0 and L % c == 0 (Bq >= 1, S % Bq == 0 stay); windows,
                                  candidates (closed chunks wholly before the local window), selection
                                  and attention are unchanged.  Summary buffers then hold
                                  floor(L/c) / floor(L/g) rows (or summary_len/c, summary_len/g), and
                                  hga_build_summaries still takes chunk-aligned ranges: call it when a
                                  chunk closes.  Forward only: hga_attn_bwd, hga_step_host and
                                  hga_tbptt_walk return HGA_ERR_UNSUPPORTED with this flag. */
#define HGA_FLAG_BWD_BF16_GRADS 64 /* hga_attn_bwd / hga_tbptt_walk: dK and dV are written as bf16
                                  [B,Hkv,S,d] (the dtype of K and V, so the call is a drop-in autograd
                                  node) instead of fp32.  The sums over query blocks still run in fp32,
                                  in the workspace (hga_workspace_bytes grows accordingly), and are
                                  rounded once at the end (one conversion launch for both tensors,
                                  released early by the last attention kernel).  Not with
                                  HGA_FLAG_BWD_ACCUMULATE, not in hga_step_host (HGA_ERR_UNSUPPORTED). */

/* bits OR-ed into *status_word by the attention kernels */
#define HGA_STATUS_BAD_INDEX 1     /* a group_idx entry was out of range, inside the sink or
                                      local window, or not ascending: that entry was skipped */
#define HGA_STATUS_WAIT_TIMEOUT 2  /* a bounded on-chip wait gave up; outputs are invalid */

typedef struct hga_params {
  int32_t batch, n_q_heads, n_kv_heads, head_dim; /* Hq % Hkv == 0; head_dim in {64, 128}      */
  int32_t total_len, seg_len;                      /* L >= S >= 1                                */
  int32_t chunk, group, q_block;                   /* c % g == 0; Bq % c == 0; S % Bq == 0;
                                                      (L - S) % Bq == 0; L % c == 0 (but see
                                                      HGA_FLAG_DECODE)                         */
  int32_t topk_chunks, topk_groups;                /* k_c >= 0; k_g >= 1 (per opened chunk)      */
  int32_t sink, local;                             /* tokens, multiples of c                     */
  float   softmax_scale;                           /* <= 0 selects 1/sqrt(head_dim)              */
  int32_t flags;                                   /* HGA_FLAG_*                                 */
  int32_t summary_len;                             /* token length the summary buffers are laid
                                                      out for (>= total_len, multiple of chunk);
                                                      0 means total_len.  Lets one pair of buffers
                                                      [B,Hkv,summary_len/c,d], [B,Hkv,summary_len/g,d]
                                                      serve a sequence walked segment by segment */
  /* element strides of the (batch, head, token) axes; all-zero means dense.  q_stride
   * also describes dQ; o_stride describes O and dO; k_stride / v_stride describe K / V. */
  int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3];
} hga_params;

/* Section 2.1, first paragraph (chunk-level and group-level summaries are derived from the
 * keys the model already projects): for every chunk and group inside the token range [tok_begin, tok_end)
 * (chunk aligned) of every (batch, kv head), write the arithmetic mean of its keys, rounded
 * once to bf16 (the mean is accumulated exactly).  Summaries outside the range are left
 * untouched, so a caller extends resident history summaries segment by segment. */
HGA_API int hga_build_summaries(const hga_params* p, const void* K, int32_t tok_begin, int32_t tok_end,
                        void* chunk_sum, void* group_sum, void* stream);

/* Section 2.1 items 1-2 (chunk selection, group selection), run without gradients.
 * Per item: the score of a summary is the maximum over the item's G*Bq query rows of the
 * raw dot product (bf16 products, fp32 accumulation); the min(k_c, #candidates) best
 * candidate chunks are selected, then inside each selected chunk the kg_eff best groups;
 * ties go to the lowest index.  Outputs as laid out above.
 * chunk_scores (optional, may be NULL) fp32 [B,Hkv,NQB,L/c]: scores, -inf off-candidate.
 * group_scores (optional, may be NULL) fp32 [B,Hkv,NQB,k_c*(c/g)]: slot (r,u) = group u
 *   of the r-th selected chunk, -inf where unused.
 * workspace: device scratch of at least hga_workspace_bytes().route bytes (16-byte
 *   aligned); contents are overwritten.  Calls that share a workspace must not overlap. 
 * An item whose routing could not be completed (a bounded on-chip wait gave up: never in normal
 * operation) gets n_groups = -1; the attention calls then attend to its sink and local window only
 * and report HGA_STATUS_BAD_INDEX. */
HGA_API int hga_route(const hga_params* p, const void* Q, const void* chunk_sum, const void* group_sum,
              int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, float* chunk_scores,
              float* group_scores, void* workspace, size_t workspace_bytes, void* stream);

/* hga_route without a caller-provided workspace (the paper has no counterpart: this entry
 * point exists for deployment reasons only).  It is for callers that cannot allocate device
 * memory at all -- code that runs while its host framework's allocator is locked or has
 * claimed the whole device, loops that must never enter cudaMalloc because it synchronises
 * the device, processes whose device memory is budgeted at start-up.  The scratch hga_route
 * would take from `workspace` lives in a fixed array inside the library image instead
 * (HGA_ROUTE_STATIC_SCRATCH_BYTES per GPU, held until the process exits), and the call itself
 * calls no allocating or freeing routine.
 *   - Same inputs, outputs and selection rule as hga_route (no optional score outputs), and the
 *     same kernels: the fused tensor-core router where the shape qualifies (it keeps the scores
 *     on chip and leaves the array untouched), else the CUDA-core router, whose chunk scores go
 *     to the array.
 *   - Size limit: hga_workspace_bytes().route must not exceed HGA_ROUTE_STATIC_SCRATCH_BYTES.
 *     That is batch * n_kv_heads * (seg_len / q_block) * per_item * 4 bytes + 16 with
 *     per_item = total_len / chunk, plus k_c * (chunk / group) with HGA_FLAG_GLOBAL_GROUP_BUDGET.
 *     A larger problem returns HGA_ERR_WORKSPACE and launches nothing.  All five benchmark
 *     configurations fit.
 *   - The FIRST call on each device looks up the array's device address.  CUDA loads a module's
 *     device data lazily, so it is this look-up that makes the driver place the array in device
 *     memory: make that first call at start-up, while device memory is still available and
 *     outside any stream capture (on a device with no memory left it returns HGA_ERR_CUDA).
 *     Later calls on the same device do no set-up and leave the amount of free device memory
 *     unchanged.
 *   - All calls on a device share the one array and it keeps the last call's contents (the
 *     kernels overwrite what they read, nothing needs clearing).  Two calls that overlap on
 *     the GPU (different streams, no ordering between them) race on it: order them. */
#define HGA_ROUTE_STATIC_SCRATCH_BYTES (4u << 20)
HGA_API int hga_route_static(const hga_params* p, const void* Q, const void* chunk_sum,
                             const void* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                             int32_t* n_groups, void* stream);

/* Section 2.1 item 3 (attention reads the exact K/V rows of the selected groups; summaries
 * only select and never act as values): for every query row i at position
 * pos, O_i = sum over routed keys k <= pos of softmax(scale * q_i.k) v_k (bf16 MMA inputs,
 * fp32 accumulation) and LSE_i.  Accepts any valid index list, not only hga_route's.
 * status_word (optional device int32) receives HGA_STATUS_* bits by atomic OR. */
HGA_API int hga_attn_fwd(const hga_params* p, const void* Q, const void* K, const void* V,
                 const int32_t* group_idx, const int32_t* n_groups, void* O, float* LSE,
                 int32_t* status_word, void* stream);

/* Backward of hga_attn_fwd with the routing frozen (Section 2.1, last paragraph: selection
 * carries no gradient, the gather and the attention do) under segment-wise TBPTT
 * (Section 2.2: history K/V is detached at the segment boundary, so no gradient reaches an
 * earlier segment): writes dQ for all S rows and dK/dV for the
 * S active rows only; history keys contribute to dQ but receive no gradient.
 * O and LSE are hga_attn_fwd's outputs, dO the upstream gradient (layout of O).
 * dK/dV are fp32 [B,Hkv,S,d] (bf16 with HGA_FLAG_BWD_BF16_GRADS) and are overwritten unless
 * HGA_FLAG_BWD_ACCUMULATE is set.  The sum over query blocks
 * uses floating-point atomics: results may differ in the last bits from run to run.
 * workspace: device scratch of at least hga_workspace_bytes().bwd bytes. */
HGA_API int hga_attn_bwd(const hga_params* p, const void* Q, const void* K, const void* V, const void* O,
                 const float* LSE, const void* dO, const int32_t* group_idx,
                 const int32_t* n_groups, void* dQ, void* dK, void* dV, void* workspace,
                 size_t workspace_bytes, int32_t* status_word, void* stream);

/* Scratch sizes (bytes) the two calls above need for `p`; either output may be NULL. */
HGA_API int hga_workspace_bytes(const hga_params* p, size_t* route_bytes, size_t* bwd_bytes);

/* One whole layer step from HOST buffers (pinned memory recommended), for callers that
 * keep the step's tensors on the host: copies Q, dO (host [B,Hq,S,d]) and the active
 * segment's K/V rows (host [B,Hkv,S,d]) into the caller's device arena, appends them to the
 * resident device K/V (device [B,Hkv,L,d] dense, history already in place), runs
 * build_summaries(active range) -> route -> attn_fwd -> attn_bwd, and copies O (bf16),
 * dQ (bf16), dK, dV (fp32) back to the host buffers.  dO_host == NULL runs the forward half
 * only.  The step runs as a pipeline over the (batch, kv head) pairs, which are independent
 * problems: one pair's kernels overlap the next pair's host->device copies and the previous
 * pair's device->host copies.  The copies run on two streams the library creates once per
 * device (on the first call there); they start after the work already queued on `stream`,
 * and `stream` waits for the last of them, so the host buffers are valid after the caller
 * synchronises `stream`.  arena: device scratch of hga_step_arena_bytes() bytes.
 * chunk_sum / group_sum: resident device summaries (history part already built). */
HGA_API int hga_step_host(const hga_params* p, const void* Q_host, const void* Kseg_host,
                  const void* Vseg_host, const void* dO_host, void* K_dev, void* V_dev,
                  void* chunk_sum, void* group_sum, void* O_host, void* dQ_host, float* dK_host,
                  float* dV_host, void* arena, size_t arena_bytes, int32_t* status_word,
                  void* stream);
HGA_API int hga_step_arena_bytes(const hga_params* p, size_t* bytes);

/* Section 2.2 (training walks a long sequence in fixed-size segments; the K/V of earlier
 * segments are kept as detached history, gradients never cross a segment boundary): one layer's
 * forward and backward over a WHOLE sequence, segment by segment, on device buffers.
 * `p` describes the sequence: total_len = its length L, seg_len = the segment length S
 * (L % S == 0); strides, where given, are those of the full-length tensors.  Segment s
 * (s = 0 .. L/S - 1) has history s*S and runs build_summaries([s*S, (s+1)*S)) -> route ->
 * attn_fwd -> attn_bwd exactly as the four calls above would with total_len = (s+1)*S.
 *   Q, dO (in), O, dQ (out)  bf16 [B,Hq,L,d]      K, V  bf16 [B,Hkv,L,d]
 *   chunk_sum, group_sum     bf16 [B,Hkv,L/c,d], [B,Hkv,L/g,d]: written segment by segment
 *   chunk_idx [L/S,B,Hkv,S/Bq,k_c], group_idx [L/S,B,Hkv,S/Bq,k_c*kg_eff], n_groups [L/S,B,Hkv,S/Bq]
 *   LSE fp32 [L/S,B,Hq,S]    dK, dV fp32 [L/S,B,Hkv,S,d] (segment s holds the rows of its own tokens)
 * dO == NULL runs the forward half only (dQ, dK, dV may then be NULL).  p->summary_len is
 * ignored (the summary buffers are laid out for L).  workspace: device scratch of at least
 * route_bytes + bwd_bytes as hga_workspace_bytes(p) reports them.  The forward chain of every
 * segment is queued on `stream`; the backward calls (each depends only on its own segment's forward)
 * are queued on a second stream the library creates once per device, which starts after the work
 * already queued on `stream` and is joined back into `stream` before the call returns, so later work
 * on `stream` sees every result.  The call itself never synchronises. */
HGA_API int hga_tbptt_walk(const hga_params* p, const void* Q, const void* K, const void* V, const void* dO,
                   void* chunk_sum, void* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                   int32_t* n_groups, void* O, float* LSE, void* dQ, void* dK, void* dV,
                   void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream);

/* Variable-length batches (packed sequences with prefix sums, the usual "cu_seqlens" convention): one
 * layer step for n_seq sequences of different lengths that share one set of buffers, tokens packed
 * back to back, token-major.  Sequence i has S_i = cu_q[i+1] - cu_q[i] active tokens (its queries)
 * and L_i = cu_k[i+1] - cu_k[i] resident tokens (history H_i = L_i - S_i first), and must obey the
 * shape rules of hga_params on its own (S_i % Bq == 0, H_i % Bq == 0, L_i % c == 0).
 *   cu_q, cu_k               HOST int32 [n_seq + 1], non-decreasing, cu[0] = 0
 *   Q, dO (in), O, dQ (out)  bf16 [sum S_i, Hq, d]         K, V  bf16 [sum L_i, Hkv, d]
 *   chunk_sum, group_sum     bf16 [Hkv, sum L_i / c, d], [Hkv, sum L_i / g, d]; sequence i's rows start
 *                            at cu_k[i]/c and cu_k[i]/g; history rows already built, the active range
 *                            of every sequence is built here
 *   chunk_idx, group_idx, n_groups   the per-sequence arrays [Hkv, S_i/Bq, ...] of the four calls
 *                            above, sequence after sequence (sequence i starts at item Hkv * cu_q[i] / Bq)
 *   LSE fp32                 sequence i's [Hq, S_i] block at element Hq * cu_q[i]
 *   dK, dV                   sequence i's [Hkv, S_i, d] block at element Hkv * d * cu_q[i]; fp32, or bf16
 *                            with HGA_FLAG_BWD_BF16_GRADS
 * p gives the head counts, head_dim, chunk/group/q_block, budgets, windows, scale and flags; its
 * batch, total_len, seg_len, summary_len and strides are ignored.  dO == NULL runs the forward half
 * only.  Every sequence runs build_summaries(active range) -> route -> attn_fwd -> attn_bwd as a
 * batch-1 problem (host logic only: the kernels are the ones above).  The sequences are independent, so
 * they go alternately to two streams the library creates once per device, and the kernels of two
 * sequences run side by side; both streams start behind the work already queued on `stream` and are
 * joined back into it before the call returns.  workspace: device scratch of
 * hga_varlen_workspace_bytes() bytes (one half per stream). */
HGA_API int hga_varlen_step(const hga_params* p, int32_t n_seq, const int32_t* cu_q, const int32_t* cu_k,
                    const void* Q, const void* K, const void* V, const void* dO, void* chunk_sum,
                    void* group_sum, int32_t* chunk_idx, int32_t* group_idx, int32_t* n_groups, void* O,
                    float* LSE, void* dQ, void* dK, void* dV, void* workspace, size_t workspace_bytes,
                    int32_t* status_word, void* stream);
HGA_API int hga_varlen_workspace_bytes(const hga_params* p, int32_t n_seq, const int32_t* cu_q,
                               const int32_t* cu_k, size_t* bytes);

HGA_API const char* hga_status_string(int status);
HGA_API int hga_version(void);
/* the cudaError_t (as int) of the most recent failed CUDA call made by this library */
HGA_API int hga_last_cuda_error(void);
/* number of kernels this library has launched since it was loaded (all calls, all streams) */
HGA_API int64_t hga_kernel_launch_count(void);

/* The same count per kernel family, so that a caller (or a test) can tell which implementation a
 * call took: every step has a tensor-core kernel (tcgen05 / TMEM / TMA) for the shapes that qualify
 * and a shape-generic CUDA-core kernel for the rest (and for HGA_FLAG_GENERIC_KERNELS).
 * An unknown family returns -1. */
#define HGA_KERNELS_SUMMARIES 0      /* hga_build_summaries */
#define HGA_KERNELS_ROUTE_TENSOR 1   /* hga_route, fused tensor-core router */
#define HGA_KERNELS_ROUTE_GENERIC 2  /* hga_route / hga_route_static, CUDA-core router (three launches) */
#define HGA_KERNELS_FWD_TENSOR 3     /* hga_attn_fwd, tensor-core kernel */
#define HGA_KERNELS_FWD_GENERIC 4    /* hga_attn_fwd, one warp per query row */
#define HGA_KERNELS_BWD_TENSOR 5     /* hga_attn_bwd, tensor-core kernels (local band + routed sweep, and
                                        the delta pre-pass where one is launched) */
#define HGA_KERNELS_BWD_GENERIC 6    /* hga_attn_bwd, CUDA-core kernels (delta, dQ, dK/dV) */
#define HGA_KERNELS_AUX 7            /* conversions (bf16 gradient outputs) and the self-test kernel */
#define HGA_KERNELS_FAMILIES 8
HGA_API int64_t hga_kernel_launch_count_by_family(int family);

/* Self-test of the bounded on-chip waits (no counterpart in the paper).  Every wait on an mbarrier
 * inside the tensor-core kernels is a poll loop with a time limit; a wait that runs out makes its CTA
 * leave cleanly and OR-s HGA_STATUS_WAIT_TIMEOUT into the status word instead of hanging the GPU.
 * This call launches one tiny kernel (one CTA, no TMA, no tensor memory) that waits with a limit of
 * `cycle_limit` SM cycles (1 <= cycle_limit <= 2^24) on a barrier that nothing ever completes, and
 * then reports exactly as the product kernels do: *status_word (device int32, required) receives
 * HGA_STATUS_WAIT_TIMEOUT, waited_cycles (device int64, optional) the cycles the wait lasted.
 * The context stays usable. */
HGA_API int hga_selftest_bounded_wait(uint32_t cycle_limit, int32_t* status_word, long long* waited_cycles,
                                      void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HGA_H */
