/*
 * CPU oracle for Hierarchical Global Attention (HGA) -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of the method of Section 2.1 ("Exact-token
 * hierarchical routing") and Section 2.2 ("Segment-wise backward") of
 * "Long-Context Fine-Tuning with Limited VRAM".  It exists to check the CUDA
 * library; only tests, the smoke check and the benchmark's CPU-baseline leg may
 * use it.  It shares no code with the CUDA path.
 *
 * All pointers are HOST pointers to dense, contiguous arrays:
 *   Q        bf16 bits  [B, Hq,  S, d]   row t of the segment is position H + t
 *   K, V     bf16 bits  [B, Hkv, L, d]   history rows first, active rows last
 *   chunk_sum bf16 bits [B, Hkv, L/c, d] group_sum bf16 bits [B, Hkv, L/g, d]
 *   chunk_idx int32 [B, Hkv, NQB, k_c]          ascending, -1 padded
 *   group_idx int32 [B, Hkv, NQB, k_c*kg_eff]   ascending global group ids, -1 padded,
 *                                               kg_eff = min(k_g, c/g)
 *   n_groups  int32 [B, Hkv, NQB]
 * An "item" is (b, kv head h, query block qb), id = (b*Hkv + h)*NQB + qb.
 * Functions taking (items, n_items) process only the listed items; items == NULL
 * means all of them.  Return 0 on success, a negative code on a bad argument.
 */
#ifndef HGA_ORACLE_H
#define HGA_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hga_ref_params {
  int32_t batch, n_q_heads, n_kv_heads, head_dim;
  int32_t total_len, seg_len;          /* L, S ; H = L - S */
  int32_t chunk, group, q_block;       /* c, g, Bq */
  int32_t topk_chunks, topk_groups;    /* k_c, k_g (per opened chunk) */
  int32_t sink, local;                 /* tokens */
  double  softmax_scale;               /* <= 0 : 1/sqrt(d) */
  int32_t global_group_budget;         /* 0: the k_g best groups inside EACH selected chunk;
                                          1: the other reading of Section 2.1 item 2 ("the best groups
                                          inside the chosen chunks"): the (selected chunks * kg_eff)
                                          best groups over ALL selected chunks together */
  int32_t score_agg;                   /* how the block's G*Bq per-row dot products with one summary become
                                          the block's score of it (Section 2.1 item 1 says only that the
                                          query block scores the summaries; Section 5 that scores come from
                                          several query positions): 0 = maximum over the rows;
                                          1 = mean over the rows (equal to the mean query row's dot
                                          product); 2 = ln sum_rows exp(dot) */
  int32_t decode;                      /* generation-shaped use (Sections 1 and 5: the same routed attention
                                          serves retrieval and generation): the query block is the few
                                          newest tokens.  Lifts the rules q_block % chunk == 0,
                                          history % q_block == 0 and total_len % chunk == 0 (q_block >= 1,
                                          any history); nothing else changes: same windows, same
                                          candidates (closed chunks wholly before the local window),
                                          same selection, same attention.  Summary arrays then hold
                                          floor(L/c) and floor(L/g) rows. */
} hga_ref_params;

/* Round a double to bf16, nearest-even, directly (single rounding). */
uint16_t hga_ref_f64_to_bf16(double x);
double   hga_ref_bf16_to_f64(uint16_t b);

/* Window geometry of query block qb (Section 2.1, item 1: sink and local windows):
 * local start ls, sink end se; candidate chunks are [se/c, ls/c). */
int hga_ref_window(const hga_ref_params* p, int32_t qb, int32_t* ls, int32_t* se);

/* Routed token set R(qb) = sink U groups U local, ascending.  out must hold
 * sink + n_groups*g + local + q_block + chunk entries.  Returns the count or <0. */
int hga_ref_routed_tokens(const hga_ref_params* p, int32_t qb, const int32_t* group_idx_item,
                          int32_t n_groups_item, int32_t* out);

/* Section 2.1: two levels of key summaries (mean of the keys, rounded once to bf16)
 * for the chunks/groups inside [tok_begin, tok_end) (chunk aligned). */
int hga_ref_build_summaries(const hga_ref_params* p, const uint16_t* K, int32_t tok_begin,
                            int32_t tok_end, uint16_t* chunk_sum, uint16_t* group_sum);

/* Section 2.1 items 1-2: chunk scores -> top-k chunks -> group scores -> top-k groups.
 * chunk_scores (optional) double [B,Hkv,NQB,L/c], -inf outside the candidates;
 * group_scores (optional) double [B,Hkv,NQB,k_c*(c/g)], slot (r, u) = group u of the
 * r-th selected chunk (ascending chunk order), -inf where unused. */
int hga_ref_route(const hga_ref_params* p, const uint16_t* Q, const uint16_t* chunk_sum,
                  const uint16_t* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                  int32_t* n_groups, double* chunk_scores, double* group_scores,
                  const int32_t* items, int32_t n_items);

/* Section 2.1 item 3: exact softmax attention over the routed exact-token K/V.
 * O double [B,Hq,S,d], LSE double [B,Hq,S] (natural log). */
int hga_ref_attn_fwd(const hga_ref_params* p, const uint16_t* Q, const uint16_t* K,
                     const uint16_t* V, const int32_t* group_idx, const int32_t* n_groups,
                     double* O, double* LSE, const int32_t* items, int32_t n_items);

/* Section 2.1 (gather + attention differentiable, routing frozen) and Section 2.2
 * (history detached): dQ double [B,Hq,S,d]; dK, dV double [B,Hkv,S,d] for the active
 * rows only (row t is position H + t).  dK/dV are ACCUMULATED into (caller zeroes). */
int hga_ref_attn_bwd(const hga_ref_params* p, const uint16_t* Q, const uint16_t* K,
                     const uint16_t* V, const uint16_t* dO, const int32_t* group_idx,
                     const int32_t* n_groups, double* dQ, double* dK, double* dV,
                     const int32_t* items, int32_t n_items);

/* The two attention entry points with real-valued (double) Q, K, V, dO of the same shapes:
 * the same code, used by finite-difference tests. */
int hga_ref_attn_fwd_f64(const hga_ref_params* p, const double* Q, const double* K,
                         const double* V, const int32_t* group_idx, const int32_t* n_groups,
                         double* O, double* LSE, const int32_t* items, int32_t n_items);
int hga_ref_attn_bwd_f64(const hga_ref_params* p, const double* Q, const double* K,
                         const double* V, const double* dO, const int32_t* group_idx,
                         const int32_t* n_groups, double* dQ, double* dK, double* dV,
                         const int32_t* items, int32_t n_items);

int hga_ref_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
