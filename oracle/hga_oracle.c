/*
 * CPU oracle for Hierarchical Global Attention (HGA) -- TEST INFRASTRUCTURE ONLY.
 * fp64 arithmetic, no blocking or fusion: each function takes the steps of the method
 * in the order the paper states them (Section 2.1 items 1-3, Section 2.2).
 * See hga_oracle.h for layouts.  Shares no code with the CUDA library.
 *
 * Readings adopted where the paper is silent (it defers the definition of HGA to a
 * companion work):
 *   - a summary is the arithmetic mean of the keys of the chunk / group, stored in the
 *     key dtype (one round-to-nearest-even of the exact mean);
 *   - a query block scores a summary by the maximum, over all its rows (positions x the
 *     GQA group's heads), of the raw dot product;
 *   - one routing decision per (sequence, kv head, query block);
 *   - candidates are the closed chunks between the sink and the local window;
 *   - the local window starts `local` tokens before the block, rounded down to a chunk;
 *   - top-k_g groups inside each selected chunk; ties go to the lowest index.
 */
#include "hga_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ERR_ARG (-1)
#define ERR_INDEX (-2)
#define ERR_MEM (-3)

double hga_ref_bf16_to_f64(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

uint16_t hga_ref_f64_to_bf16(double x) {
  uint64_t bits;
  memcpy(&bits, &x, 8);
  uint16_t sign = (uint16_t)((bits >> 63) << 15);
  int eb = (int)((bits >> 52) & 0x7ff);
  uint64_t frac = bits & ((1ull << 52) - 1);
  if (eb == 0x7ff) return (uint16_t)(sign | (frac ? 0x7fc0 : 0x7f80));
  if (eb == 0) return sign; /* zero or a double subnormal: far below bf16's range */
  uint64_t sig = frac | (1ull << 52);    /* x = sig * 2^(eb - 1023 - 52) */
  int E = eb - 1023 + 127;               /* bf16 biased exponent if normal */
  int shift = 52 - 7;                    /* keep 1 + 7 bits */
  int normal = 1;
  if (E <= 0) { shift += 1 - E; normal = 0; }
  if (shift >= 63) return sign;          /* below half the smallest subnormal */
  uint64_t q = sig >> shift;
  uint64_t rem = sig & ((1ull << shift) - 1);
  uint64_t half = 1ull << (shift - 1);
  if (rem > half || (rem == half && (q & 1))) q++;
  /* normal: q in [128, 256]; adding q to (E-1)<<7 carries into the exponent by itself */
  uint32_t out = normal ? (uint32_t)(((uint32_t)(E - 1) << 7) + q) : (uint32_t)q;
  if (out >= 0x7f80) out = 0x7f80;       /* overflow to infinity */
  return (uint16_t)(sign | out);
}

/* element load: bf16 bits, or (for the *_f64 entry points) doubles */
static inline double ld(const void* base, int is_f64, long i) {
  return is_f64 ? ((const double*)base)[i] : hga_ref_bf16_to_f64(((const uint16_t*)base)[i]);
}

static double scale_of(const hga_ref_params* p) {
  return p->softmax_scale > 0 ? p->softmax_scale : 1.0 / sqrt((double)p->head_dim);
}

static int check(const hga_ref_params* p) {
  if (!p) return ERR_ARG;
  if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->head_dim < 1) return ERR_ARG;
  if (p->n_q_heads % p->n_kv_heads) return ERR_ARG;
  if (p->seg_len < 1 || p->total_len < p->seg_len) return ERR_ARG;
  if (p->group < 1 || p->chunk < p->group || p->chunk % p->group) return ERR_ARG;
  if (p->q_block < 1 || p->seg_len % p->q_block) return ERR_ARG;
  if (!p->decode) {
    if (p->q_block < p->chunk || p->q_block % p->chunk) return ERR_ARG;
    if ((p->total_len - p->seg_len) % p->q_block) return ERR_ARG;
    if (p->total_len % p->chunk) return ERR_ARG;
  }
  if (p->topk_chunks < 0 || p->topk_groups < 1) return ERR_ARG;
  if (p->sink < 0 || p->local < 0 || p->sink % p->chunk || p->local % p->chunk) return ERR_ARG;
  if (p->score_agg < 0 || p->score_agg > 2) return ERR_ARG;
  return 0;
}

static int kg_eff(const hga_ref_params* p) {
  int per = p->chunk / p->group;
  return p->topk_groups < per ? p->topk_groups : per;
}

int hga_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

int hga_ref_window(const hga_ref_params* p, int32_t qb, int32_t* ls, int32_t* se) {
  int rc = check(p);
  if (rc) return rc;
  int H = p->total_len - p->seg_len;
  int p0 = H + qb * p->q_block;
  int l = p0 - p->local;
  l = l <= 0 ? 0 : (l / p->chunk) * p->chunk;
  *ls = l;
  *se = p->sink < l ? p->sink : l;
  return 0;
}

int hga_ref_routed_tokens(const hga_ref_params* p, int32_t qb, const int32_t* gi, int32_t ng,
                          int32_t* out) {
  int32_t ls, se;
  int rc = hga_ref_window(p, qb, &ls, &se);
  if (rc) return rc;
  int H = p->total_len - p->seg_len, g = p->group;
  int end = H + (qb + 1) * p->q_block;
  int n = 0, prev = -1;
  for (int t = 0; t < se; ++t) out[n++] = t;
  for (int i = 0; i < ng; ++i) {
    int m = gi[i];
    if (m <= prev) return ERR_INDEX;                       /* ascending, unique */
    if (m * g < se || (m + 1) * g > ls) return ERR_INDEX;  /* between sink and local */
    prev = m;
    for (int t = m * g; t < (m + 1) * g; ++t) out[n++] = t;
  }
  for (int t = ls; t < end; ++t) out[n++] = t;
  return n;
}

int hga_ref_build_summaries(const hga_ref_params* p, const uint16_t* K, int32_t tb, int32_t te,
                            uint16_t* chunk_sum, uint16_t* group_sum) {
  int rc = check(p);
  if (rc) return rc;
  if (!K || !chunk_sum || !group_sum) return ERR_ARG;
  int L = p->total_len, d = p->head_dim, c = p->chunk, g = p->group;
  if (tb < 0 || te > L || tb > te || tb % c || te % c) return ERR_ARG;
  long BH = (long)p->batch * p->n_kv_heads;
#pragma omp parallel for schedule(static)
  for (long bh = 0; bh < BH; ++bh) {
    const uint16_t* Kb = K + bh * (long)L * d;
    for (int m = tb / g; m < te / g; ++m)
      for (int e = 0; e < d; ++e) {
        double s = 0;
        for (int t = m * g; t < (m + 1) * g; ++t) s += hga_ref_bf16_to_f64(Kb[(long)t * d + e]);
        group_sum[(bh * (L / g) + m) * d + e] = hga_ref_f64_to_bf16(s / g);
      }
    for (int j = tb / c; j < te / c; ++j)
      for (int e = 0; e < d; ++e) {
        double s = 0;
        for (int t = j * c; t < (j + 1) * c; ++t) s += hga_ref_bf16_to_f64(Kb[(long)t * d + e]);
        chunk_sum[(bh * (L / c) + j) * d + e] = hga_ref_f64_to_bf16(s / c);
      }
  }
  return 0;
}

/* the block's score of one summary from its rows' dot products (row . summary):
 * agg 0 maximum, 1 mean, 2 log-sum-exp */
static double block_score(const double* rows, int n_rows, int d, const uint16_t* summary, int agg) {
  double* s = (double*)malloc(sizeof(double) * (size_t)n_rows);
  if (!s) return NAN;
  double best = -INFINITY;
  for (int r = 0; r < n_rows; ++r) {
    s[r] = 0;
    for (int e = 0; e < d; ++e) s[r] += rows[(long)r * d + e] * hga_ref_bf16_to_f64(summary[e]);
    if (s[r] > best) best = s[r];
  }
  double out = best;
  if (agg == 1) {
    out = 0;
    for (int r = 0; r < n_rows; ++r) out += s[r];
    out /= (double)n_rows;
  } else if (agg == 2) {
    double z = 0;
    for (int r = 0; r < n_rows; ++r) z += exp(s[r] - best);
    out = best + log(z);
  }
  free(s);
  return out;
}

/* choose the k best of ids[0..n) by (score descending, id ascending); mark them in taken[] */
static void top_k(const double* score, int n, int k, char* taken) {
  memset(taken, 0, (size_t)n);
  for (int r = 0; r < k && r < n; ++r) {
    int best = -1;
    for (int i = 0; i < n; ++i)
      if (!taken[i] && (best < 0 || score[i] > score[best])) best = i; /* first wins ties */
    taken[best] = 1;
  }
}

int hga_ref_route(const hga_ref_params* p, const uint16_t* Q, const uint16_t* chunk_sum,
                  const uint16_t* group_sum, int32_t* chunk_idx, int32_t* group_idx,
                  int32_t* n_groups, double* chunk_scores, double* group_scores,
                  const int32_t* items, int32_t n_items) {
  int rc = check(p);
  if (rc) return rc;
  if (!Q || !chunk_sum || !group_sum || !chunk_idx || !group_idx || !n_groups) return ERR_ARG;
  int Hkv = p->n_kv_heads, G = p->n_q_heads / Hkv, d = p->head_dim;
  int L = p->total_len, S = p->seg_len, c = p->chunk, g = p->group, Bq = p->q_block;
  int NQB = S / Bq, Nc = L / c, Ng = L / g, per = c / g, kc = p->topk_chunks, kge = kg_eff(p);
  long total = (long)p->batch * Hkv * NQB;
  long count = items ? n_items : total;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long it = 0; it < count; ++it) {
    long item = items ? items[it] : it;
    int qb = (int)(item % NQB);
    long bh = item / NQB;
    int h = (int)(bh % Hkv);
    long b = bh / Hkv;
    int32_t ls, se;
    hga_ref_window(p, qb, &ls, &se);
    int j0 = se / c, n_cand = (ls - se) / c;
    int n_rows = G * Bq;
    double* rows = (double*)malloc(sizeof(double) * (size_t)n_rows * d);
    /* room for the candidate chunk scores, or for the group scores of all selected chunks */
    size_t n_sc = (size_t)(n_cand > kc * per ? n_cand : kc * per) + 8;
    double* sc = (double*)malloc(sizeof(double) * n_sc);
    char* taken = (char*)malloc(n_sc);
    if (!rows || !sc || !taken) { failed = 1; free(rows); free(sc); free(taken); continue; }
    for (int a = 0; a < G; ++a)
      for (int t = 0; t < Bq; ++t)
        for (int e = 0; e < d; ++e)
          rows[((long)a * Bq + t) * d + e] = hga_ref_bf16_to_f64(
              Q[(((long)b * p->n_q_heads + h * G + a) * S + (long)qb * Bq + t) * d + e]);
    int32_t* ci = chunk_idx + item * kc;
    int32_t* gi = group_idx + item * (long)kc * kge;
    for (int i = 0; i < kc; ++i) ci[i] = -1;
    for (int i = 0; i < kc * kge; ++i) gi[i] = -1;
    if (chunk_scores)
      for (int j = 0; j < Nc; ++j) chunk_scores[item * Nc + j] = -INFINITY;
    if (group_scores)
      for (int i = 0; i < kc * per; ++i) group_scores[item * (long)kc * per + i] = -INFINITY;
    /* item 1: score every candidate chunk summary, keep the k_c best */
    for (int i = 0; i < n_cand; ++i) {
      sc[i] = block_score(rows, n_rows, d, chunk_sum + (bh * Nc + j0 + i) * (long)d, p->score_agg);
      if (chunk_scores) chunk_scores[item * Nc + j0 + i] = sc[i];
    }
    top_k(sc, n_cand, kc, taken);
    int nsel = 0;
    for (int i = 0; i < n_cand; ++i)
      if (taken[i]) ci[nsel++] = j0 + i; /* ascending */
    int ng = 0;
    if (!p->global_group_budget) {
      /* item 2: open each selected chunk, keep its k_g best groups */
      for (int r = 0; r < nsel; ++r) {
        int m0 = ci[r] * per;
        for (int u = 0; u < per; ++u) {
          sc[u] = block_score(rows, n_rows, d, group_sum + (bh * Ng + m0 + u) * (long)d, p->score_agg);
          if (group_scores) group_scores[item * (long)kc * per + (long)r * per + u] = sc[u];
        }
        top_k(sc, per, kge, taken);
        for (int u = 0; u < per; ++u)
          if (taken[u]) gi[ng++] = m0 + u;
      }
    } else {
      /* item 2, global budget: the groups of all selected chunks compete for nsel * kg_eff places;
       * slots are in ascending group order (chunks ascend), so "first wins ties" = lowest group id */
      for (int r = 0; r < nsel; ++r)
        for (int u = 0; u < per; ++u) {
          sc[r * per + u] = block_score(rows, n_rows, d, group_sum + (bh * Ng + (long)ci[r] * per + u) * (long)d,
                                        p->score_agg);
          if (group_scores) group_scores[item * (long)kc * per + (long)r * per + u] = sc[r * per + u];
        }
      top_k(sc, nsel * per, nsel * kge, taken);
      for (int i = 0; i < nsel * per; ++i)
        if (taken[i]) gi[ng++] = ci[i / per] * per + i % per;
    }
    n_groups[item] = ng;
    free(rows); free(sc); free(taken);
  }
  return failed ? ERR_MEM : 0;
}

/* Gathered copy of one item's routed K/V rows as doubles. */
typedef struct {
  int n;          /* routed tokens */
  int32_t* tok;   /* positions, ascending */
  double* k;      /* [n, d] */
  double* v;      /* [n, d] */
} routed_t;

static int gather_item(const hga_ref_params* p, long bh, int qb, const void* K, const void* V,
                       int f64, const int32_t* gi, int ng, routed_t* r) {
  int d = p->head_dim, L = p->total_len;
  int cap = p->sink + ng * p->group + p->local + p->q_block + p->chunk;
  r->tok = (int32_t*)malloc(sizeof(int32_t) * (size_t)cap);
  if (!r->tok) return ERR_MEM;
  int n = hga_ref_routed_tokens(p, qb, gi, ng, r->tok);
  if (n < 0) { free(r->tok); r->tok = NULL; return n; }
  r->n = n;
  r->k = (double*)malloc(sizeof(double) * (size_t)n * d);
  r->v = (double*)malloc(sizeof(double) * (size_t)n * d);
  if (!r->k || !r->v) { free(r->tok); free(r->k); free(r->v); return ERR_MEM; }
  for (int i = 0; i < n; ++i)
    for (int e = 0; e < d; ++e) {
      long src = (bh * L + r->tok[i]) * (long)d + e;
      r->k[(long)i * d + e] = ld(K, f64, src);
      r->v[(long)i * d + e] = ld(V, f64, src);
    }
  return 0;
}

static void free_routed(routed_t* r) { free(r->tok); free(r->k); free(r->v); }

/* softmax row: fills prob[0..n_vis) for the keys with position <= pos; returns LSE */
static double softmax_row(const double* q, const routed_t* r, int d, int pos, double scale,
                          double* prob, int* n_vis_out) {
  int n_vis = 0;
  double mx = -INFINITY;
  for (int i = 0; i < r->n && r->tok[i] <= pos; ++i) {
    double s = 0;
    for (int e = 0; e < d; ++e) s += q[e] * r->k[(long)i * d + e];
    prob[i] = s * scale;
    if (prob[i] > mx) mx = prob[i];
    n_vis = i + 1;
  }
  double z = 0;
  for (int i = 0; i < n_vis; ++i) z += exp(prob[i] - mx);
  double lse = mx + log(z);
  for (int i = 0; i < n_vis; ++i) prob[i] = exp(prob[i] - lse);
  *n_vis_out = n_vis;
  return lse;
}

static int attn_fwd(const hga_ref_params* p, const void* Q, const void* K, const void* V, int f64,
                    const int32_t* group_idx, const int32_t* n_groups, double* O, double* LSE,
                    const int32_t* items, int32_t n_items) {
  int rc = check(p);
  if (rc) return rc;
  if (!Q || !K || !V || !group_idx || !n_groups || !O || !LSE) return ERR_ARG;
  int Hkv = p->n_kv_heads, Hq = p->n_q_heads, G = Hq / Hkv, d = p->head_dim;
  int S = p->seg_len, Bq = p->q_block, NQB = S / Bq, H = p->total_len - S;
  int width = p->topk_chunks * kg_eff(p);
  double scale = scale_of(p);
  long total = (long)p->batch * Hkv * NQB, count = items ? n_items : total;
  int status = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long it = 0; it < count; ++it) {
    long item = items ? items[it] : it;
    int qb = (int)(item % NQB);
    long bh = item / NQB;
    int h = (int)(bh % Hkv);
    long b = bh / Hkv;
    routed_t r;
    int e0 = gather_item(p, bh, qb, K, V, f64, group_idx + item * width, n_groups[item], &r);
    if (e0) { status = e0; continue; }
    double* prob = (double*)malloc(sizeof(double) * (size_t)r.n);
    double* q = (double*)malloc(sizeof(double) * (size_t)d);
    for (int a = 0; a < G; ++a)
      for (int t = 0; t < Bq; ++t) {
        long row = ((long)b * Hq + h * G + a) * S + (long)qb * Bq + t;
        for (int e = 0; e < d; ++e) q[e] = ld(Q, f64, row * d + e);
        int n_vis;
        LSE[row] = softmax_row(q, &r, d, H + qb * Bq + t, scale, prob, &n_vis);
        for (int e = 0; e < d; ++e) {
          double o = 0;
          for (int i = 0; i < n_vis; ++i) o += prob[i] * r.v[(long)i * d + e];
          O[row * d + e] = o;
        }
      }
    free(prob); free(q);
    free_routed(&r);
  }
  return status;
}

static int attn_bwd(const hga_ref_params* p, const void* Q, const void* K, const void* V,
                    const void* dO, int f64, const int32_t* group_idx, const int32_t* n_groups,
                    double* dQ, double* dK, double* dV, const int32_t* items, int32_t n_items) {
  int rc = check(p);
  if (rc) return rc;
  if (!Q || !K || !V || !dO || !group_idx || !n_groups || !dQ || !dK || !dV) return ERR_ARG;
  int Hkv = p->n_kv_heads, Hq = p->n_q_heads, G = Hq / Hkv, d = p->head_dim;
  int S = p->seg_len, Bq = p->q_block, NQB = S / Bq, H = p->total_len - S;
  int width = p->topk_chunks * kg_eff(p);
  double scale = scale_of(p);
  long total = (long)p->batch * Hkv * NQB, count = items ? n_items : total;
  int status = 0;
#pragma omp parallel for ordered schedule(dynamic, 1)
  for (long it = 0; it < count; ++it) {
    long item = items ? items[it] : it;
    int qb = (int)(item % NQB);
    long bh = item / NQB;
    int h = (int)(bh % Hkv);
    long b = bh / Hkv;
    routed_t r;
    int e0 = gather_item(p, bh, qb, K, V, f64, group_idx + item * width, n_groups[item], &r);
    if (e0) { status = e0; continue; }
    double* prob = (double*)malloc(sizeof(double) * (size_t)r.n);
    double* q = (double*)malloc(sizeof(double) * (size_t)d * 4);
    double *go = q + d, *o = q + 2 * d, *dq = q + 3 * d;
    double* dk = (double*)calloc((size_t)r.n * d, sizeof(double)); /* this item's share */
    double* dv = (double*)calloc((size_t)r.n * d, sizeof(double));
    for (int a = 0; a < G; ++a)
      for (int t = 0; t < Bq; ++t) {
        long row = ((long)b * Hq + h * G + a) * S + (long)qb * Bq + t;
        for (int e = 0; e < d; ++e) {
          q[e] = ld(Q, f64, row * d + e);
          go[e] = ld(dO, f64, row * d + e);
          dq[e] = 0;
        }
        int n_vis;
        softmax_row(q, &r, d, H + qb * Bq + t, scale, prob, &n_vis);
        /* O, then D = sum_e dO_e O_e */
        double D = 0;
        for (int e = 0; e < d; ++e) {
          double acc = 0;
          for (int i = 0; i < n_vis; ++i) acc += prob[i] * r.v[(long)i * d + e];
          o[e] = acc;
          D += go[e] * acc;
        }
        for (int i = 0; i < n_vis; ++i) {
          double dP = 0;
          for (int e = 0; e < d; ++e) dP += go[e] * r.v[(long)i * d + e];
          double dS = prob[i] * (dP - D);
          for (int e = 0; e < d; ++e) {
            dv[(long)i * d + e] += prob[i] * go[e];
            dq[e] += scale * dS * r.k[(long)i * d + e];
            dk[(long)i * d + e] += scale * dS * q[e];
          }
        }
        for (int e = 0; e < d; ++e) dQ[row * d + e] = dq[e];
      }
    /* Section 2.2: only active-segment rows (position >= H) receive dK/dV;
     * items add their shares in item order, so the result does not depend on threads */
#pragma omp ordered
    for (int i = 0; i < r.n; ++i) {
      int pos = r.tok[i];
      if (pos < H) continue;
      long dst = (bh * S + (pos - H)) * (long)d;
      for (int e = 0; e < d; ++e) {
        dK[dst + e] += dk[(long)i * d + e];
        dV[dst + e] += dv[(long)i * d + e];
      }
    }
    free(prob); free(q); free(dk); free(dv);
    free_routed(&r);
  }
  return status;
}

int hga_ref_attn_fwd(const hga_ref_params* p, const uint16_t* Q, const uint16_t* K,
                     const uint16_t* V, const int32_t* group_idx, const int32_t* n_groups,
                     double* O, double* LSE, const int32_t* items, int32_t n_items) {
  return attn_fwd(p, Q, K, V, 0, group_idx, n_groups, O, LSE, items, n_items);
}

int hga_ref_attn_bwd(const hga_ref_params* p, const uint16_t* Q, const uint16_t* K,
                     const uint16_t* V, const uint16_t* dO, const int32_t* group_idx,
                     const int32_t* n_groups, double* dQ, double* dK, double* dV,
                     const int32_t* items, int32_t n_items) {
  return attn_bwd(p, Q, K, V, dO, 0, group_idx, n_groups, dQ, dK, dV, items, n_items);
}

/* Same arithmetic with real-valued (double) inputs: lets tests take finite differences. */
int hga_ref_attn_fwd_f64(const hga_ref_params* p, const double* Q, const double* K,
                         const double* V, const int32_t* group_idx, const int32_t* n_groups,
                         double* O, double* LSE, const int32_t* items, int32_t n_items) {
  return attn_fwd(p, Q, K, V, 1, group_idx, n_groups, O, LSE, items, n_items);
}

int hga_ref_attn_bwd_f64(const hga_ref_params* p, const double* Q, const double* K,
                         const double* V, const double* dO, const int32_t* group_idx,
                         const int32_t* n_groups, double* dQ, double* dK, double* dV,
                         const int32_t* items, int32_t n_items) {
  return attn_bwd(p, Q, K, V, dO, 1, group_idx, n_groups, dQ, dK, dV, items, n_items);
}
