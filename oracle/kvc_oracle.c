/*
 * KVCompose compression pass -- reference oracle (TEST INFRASTRUCTURE ONLY).
 *
 * A plain, slow, double-precision CPU restatement of the method, one function per
 * step, each in the paper's order and notation.  It exists so that the CUDA library
 * can be checked against something that can be verified against the paper by eye.
 * It is not part of the product: only the test-suite, the smoke check and the
 * benchmark's cpu-baseline leg may call it.  It shares no code with the CUDA path.
 *
 * Conventions used by every function here:
 *   - 0-based indices (the paper is 1-based).
 *   - Equation numbers count every numbered display of the paper in order: (3) attention,
 *     (14) Agg_task, (15) Agg_group, (16) head-mean term, (17) argsort, (18) S', (19)
 *     composite score, (20) pool, (21) B_total, (22) N_l, (23)-(24) compressed K', V'.
 *   - One sequence, one layer at a time unless stated; tensors are dense,
 *     row-major, last dimension contiguous.
 *   - Q and K arrive as float (fp32, or bf16 widened exactly to fp32); all
 *     arithmetic is done in double.
 *   - Aggregators: 0 = max-pooling, 1 = average-pooling (Sec. 4 "Experiments":
 *     max for Agg_task, average for the others, is the paper's default).
 *
 * Readings of points the paper leaves open (each also listed in the design notes):
 *   - the scoring ("task") queries are given by the caller, w rows per query head;
 *   - window row m sits at absolute position q_pos0 + m and sees key c iff
 *     c <= q_pos0 + m (the model's own causal mask); q_pos0 >= N disables masking;
 *   - the softmax of Eq. (3) runs over the visible cached keys only; a masked
 *     entry has attention weight 0 and still takes part in an average over m;
 *   - query head j belongs to KV head q_to_kv[j] (default floor(j / G));
 *   - argsort ties: the smaller original position comes first;
 *   - top-B_total ties: total order (I descending, layer ascending, k ascending).
 *
 * Parity status: every function below is pinned by tests against closed forms,
 * invariants, library-routine special cases and brute force.  The one thing that
 * cannot be pinned is agreement with the authors' own implementation (the paper
 * prints no worked numeric example): end-to-end vs. the authors -- parity unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_AGG_MAX 0
#define ORACLE_AGG_MEAN 1

/* Number of worker threads used by the *_layer / compress loops (1 = serial). */
static int g_threads = 1;

void oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }

int oracle_get_threads(void) { return g_threads; }

int oracle_has_openmp(void) {
#ifdef _OPENMP
  return 1;
#else
  return 0;
#endif
}

/* ------------------------------------------------------------------------- */
/* Step 1: attention rows.  Sec. 2.1, Eq. (3): A = softmax(q K^T / sqrt(d_h)). */
/* ------------------------------------------------------------------------- */

/*
 * One query head: q [w, d], k [N, d]  ->  A [w, N] (double).
 * Row m attends to the keys c <= q_pos0 + m; entries beyond that are 0.
 * A row that sees no key at all (q_pos0 + m < 0) is all zeros.
 */
void oracle_attention_rows(const float* q, const float* k, int64_t N, int32_t d,
                           int32_t w, double scale, int64_t q_pos0, double* A) {
  for (int32_t m = 0; m < w; ++m) {
    double* row = A + (int64_t)m * N;
    int64_t last = q_pos0 + m; /* last visible key */
    int64_t n_vis = last >= N - 1 ? N : last + 1;
    if (n_vis < 0) n_vis = 0;
    /* logits s_c = scale * <q_m, k_c> */
    double s_max = -INFINITY;
    for (int64_t c = 0; c < n_vis; ++c) {
      double s = 0.0;
      for (int32_t t = 0; t < d; ++t)
        s += (double)q[(int64_t)m * d + t] * (double)k[c * d + t];
      s *= scale;
      row[c] = s;
      if (s > s_max) s_max = s;
    }
    double denom = 0.0;
    for (int64_t c = 0; c < n_vis; ++c) {
      row[c] = exp(row[c] - s_max);
      denom += row[c];
    }
    for (int64_t c = 0; c < n_vis; ++c) row[c] /= denom;
    for (int64_t c = n_vis; c < N; ++c) row[c] = 0.0;
  }
}

/* ------------------------------------------------------------------------- */
/* Steps 2-4: Eq. (14) Agg_task, Eq. (15) Agg_group, Eq. (16) mean augmentation */
/* ------------------------------------------------------------------------- */

/*
 * One layer of one sequence.
 *   q [Hq, w, d], k [Hkv, N, d]  ->  S [Hkv, N]
 * q_to_kv: Hq entries or NULL (then floor(j / (Hq/Hkv))).
 * S_task [j, c]  = Agg_task over the w window rows of A_j[m, c]      (Eq. 14)
 * S_group[h, c]  = Agg_group over the query heads j of KV head h     (Eq. 15)
 * S[h, c]        = S_group[h, c] + (1/Hkv) sum_i S_group[i, c]       (Eq. 16)
 * Returns 0, or -1 on allocation failure / a KV head without query heads.
 */
static int score_layer_impl(const float* q, const float* k, const float* v, int32_t Hq,
                            int32_t Hkv, int64_t N, int32_t d, int32_t w, double scale,
                            int64_t q_pos0, int32_t agg_task, int32_t agg_group,
                            int32_t augment, const int32_t* q_to_kv, double* S) {
  int32_t G = Hq / Hkv;
  double* S_task = (double*)malloc(sizeof(double) * (size_t)Hq * (size_t)N);
  if (!S_task) return -1;
  int failed = 0;

  /* Eq. (14): per query head */
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(dynamic, 1)
#endif
  for (int32_t j = 0; j < Hq; ++j) {
    int32_t h = q_to_kv ? q_to_kv[j] : j / G;
    double* A = (double*)malloc(sizeof(double) * (size_t)w * (size_t)N);
    if (!A) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
      failed = 1;
      continue;
    }
    oracle_attention_rows(q + (int64_t)j * w * d, k + (int64_t)h * N * d, N, d, w,
                          scale, q_pos0, A);
    if (v) {
      /* App. A.1.3, the v-norm variant: every entry of A is multiplied by the Euclidean
         norm of the value row of its token (in the KV head this query head reads). */
      for (int64_t c = 0; c < N; ++c) {
        double nn = 0.0;
        for (int32_t t = 0; t < d; ++t) {
          double x = (double)v[((int64_t)h * N + c) * d + t];
          nn += x * x;
        }
        nn = sqrt(nn);
        for (int32_t m = 0; m < w; ++m) A[(int64_t)m * N + c] *= nn;
      }
    }
    for (int64_t c = 0; c < N; ++c) {
      double acc = (agg_task == ORACLE_AGG_MAX) ? -INFINITY : 0.0;
      for (int32_t m = 0; m < w; ++m) {
        double a = A[(int64_t)m * N + c];
        if (agg_task == ORACLE_AGG_MAX)
          acc = a > acc ? a : acc;
        else
          acc += a;
      }
      if (agg_task == ORACLE_AGG_MEAN) acc /= (double)w;
      S_task[(int64_t)j * N + c] = acc;
    }
    free(A);
  }
  if (failed) {
    free(S_task);
    return -1;
  }

  /* Eq. (15): per KV head, over its query heads */
  for (int32_t h = 0; h < Hkv; ++h) {
    int32_t members = 0;
    for (int32_t j = 0; j < Hq; ++j)
      if ((q_to_kv ? q_to_kv[j] : j / G) == h) ++members;
    if (members == 0) {
      free(S_task);
      return -1;
    }
    for (int64_t c = 0; c < N; ++c) {
      double acc = (agg_group == ORACLE_AGG_MAX) ? -INFINITY : 0.0;
      for (int32_t j = 0; j < Hq; ++j) {
        if ((q_to_kv ? q_to_kv[j] : j / G) != h) continue;
        double a = S_task[(int64_t)j * N + c];
        if (agg_group == ORACLE_AGG_MAX)
          acc = a > acc ? a : acc;
        else
          acc += a;
      }
      if (agg_group == ORACLE_AGG_MEAN) acc /= (double)members;
      S[(int64_t)h * N + c] = acc;
    }
  }
  free(S_task);

  /* Eq. (16): add the mean over the KV heads of the same layer and token */
  if (augment) {
    for (int64_t c = 0; c < N; ++c) {
      double mean = 0.0;
      for (int32_t i = 0; i < Hkv; ++i) mean += S[(int64_t)i * N + c];
      mean /= (double)Hkv;
      for (int32_t h = 0; h < Hkv; ++h) S[(int64_t)h * N + c] += mean;
    }
  }
  return 0;
}

int oracle_score_layer(const float* q, const float* k, int32_t Hq, int32_t Hkv,
                       int64_t N, int32_t d, int32_t w, double scale,
                       int64_t q_pos0, int32_t agg_task, int32_t agg_group,
                       int32_t augment, const int32_t* q_to_kv, double* S) {
  return score_layer_impl(q, k, NULL, Hq, Hkv, N, d, w, scale, q_pos0, agg_task, agg_group,
                          augment, q_to_kv, S);
}

/*
 * The v-norm variant of App. A.1.3 ("Effect of Value Norms on Token Scores"): the weighted
 * attention matrix A^(w)[m, c] = A[m, c] * ||v_c|| replaces A in Eqs. (14)-(16).
 * v [Hkv, N, d]: the value rows; the norm is the Euclidean norm over the d entries of a row.
 */
int oracle_score_layer_vnorm(const float* q, const float* k, const float* v, int32_t Hq,
                             int32_t Hkv, int64_t N, int32_t d, int32_t w, double scale,
                             int64_t q_pos0, int32_t agg_task, int32_t agg_group,
                             int32_t augment, const int32_t* q_to_kv, double* S) {
  if (!v) return -1;
  return score_layer_impl(q, k, v, Hq, Hkv, N, d, w, scale, q_pos0, agg_task, agg_group,
                          augment, q_to_kv, S);
}

/* ------------------------------------------------------------------------- */
/* Step 5: Eq. (17) per-head argsort, descending; Eq. (18) S'[k] = S[idx[k]]    */
/* ------------------------------------------------------------------------- */

typedef struct {
  double s;
  int64_t c;
} rank_item;

static int rank_cmp(const void* a, const void* b) {
  const rank_item* x = (const rank_item*)a;
  const rank_item* y = (const rank_item*)b;
  if (x->s > y->s) return -1; /* larger score first */
  if (x->s < y->s) return 1;
  if (x->c < y->c) return -1; /* equal scores: smaller position first */
  if (x->c > y->c) return 1;
  return 0;
}

/* One (layer, head): S [N] -> idx [N] (int32), S_sorted [N] (nullable). */
int oracle_rank(const double* S, int64_t N, int32_t* idx, double* S_sorted) {
  rank_item* it = (rank_item*)malloc(sizeof(rank_item) * (size_t)(N > 0 ? N : 1));
  if (!it) return -1;
  for (int64_t c = 0; c < N; ++c) {
    it[c].s = S[c];
    it[c].c = c;
  }
  qsort(it, (size_t)N, sizeof(rank_item), rank_cmp); /* key (s, c) is a total order */
  for (int64_t kk = 0; kk < N; ++kk) {
    idx[kk] = (int32_t)it[kk].c;
    if (S_sorted) S_sorted[kk] = it[kk].s;
  }
  free(it);
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Step 6: Eq. (19) composite score I[k] = Agg_head over h of S'[h, k]         */
/* ------------------------------------------------------------------------- */

/* One layer: S_sorted [Hkv, N] -> I [N], double arithmetic. */
void oracle_compose(const double* S_sorted, int32_t Hkv, int64_t N, int32_t agg_head,
                    double* I) {
  for (int64_t kk = 0; kk < N; ++kk) {
    double acc = (agg_head == ORACLE_AGG_MAX) ? -INFINITY : 0.0;
    for (int32_t h = 0; h < Hkv; ++h) {
      double a = S_sorted[(int64_t)h * N + kk];
      if (agg_head == ORACLE_AGG_MAX)
        acc = a > acc ? a : acc;
      else
        acc += a;
    }
    if (agg_head == ORACLE_AGG_MEAN) acc /= (double)Hkv;
    I[kk] = acc;
  }
}

/*
 * The same step in single precision with a fixed evaluation order
 * (h = 0, 1, ... left to right, then one division by Hkv).  Used where a
 * float decides an integer downstream (the allocation): both sides then take
 * the decision from bit-identical composite scores.
 */
void oracle_compose_f32(const float* S_sorted, int32_t Hkv, int64_t N, int32_t agg_head,
                        float* I) {
  for (int64_t kk = 0; kk < N; ++kk) {
    volatile float acc = S_sorted[kk];
    for (int32_t h = 1; h < Hkv; ++h) {
      float a = S_sorted[(int64_t)h * N + kk];
      if (agg_head == ORACLE_AGG_MAX)
        acc = a > acc ? a : acc;
      else
        acc = acc + a;
    }
    if (agg_head == ORACLE_AGG_MEAN) acc = acc / (float)Hkv;
    I[kk] = acc;
  }
}

/* ------------------------------------------------------------------------- */
/* Step 7: Eq. (20) global pool, Eq. (21) B_total, Eq. (22) per-layer N_l       */
/* ------------------------------------------------------------------------- */

/*
 * B_total = floor((1 - r_target) * L * N).  r_target is a decimal such as 0.8 that a
 * double cannot hold exactly; the product is therefore nudged up by a relative 1e-12
 * before the floor, so that 0.2 * 163840 gives 32768 as in exact arithmetic and not 32767.
 */
int64_t oracle_budget_from_ratio(int32_t L, int64_t N, double r_target) {
  double x = (1.0 - r_target) * (double)L * (double)N;
  double b = floor(x + fabs(x) * 1e-12 + 1e-9);
  if (b < 0.0) b = 0.0;
  if (b > (double)L * (double)N) b = (double)L * (double)N;
  return (int64_t)b;
}

typedef struct {
  double v;
  int32_t l;
  int64_t k;
} pool_item;

static int pool_cmp(const void* a, const void* b) {
  const pool_item* x = (const pool_item*)a;
  const pool_item* y = (const pool_item*)b;
  if (x->v > y->v) return -1;
  if (x->v < y->v) return 1;
  if (x->l < y->l) return -1;
  if (x->l > y->l) return 1;
  if (x->k < y->k) return -1;
  if (x->k > y->k) return 1;
  return 0;
}

/*
 * I [L, N] -> n_keep [L], offsets [L+1].
 * Pool every I[l, k], order by (I desc, l asc, k asc), keep the first B;
 * n_keep[l] = how many of the kept ones lie in layer l; offsets = exclusive
 * prefix sum (offsets[L] = B).
 */
int oracle_allocate(const double* I, int32_t L, int64_t N, int64_t B, int32_t* n_keep,
                    int64_t* offsets) {
  int64_t total = (int64_t)L * N;
  if (B < 0 || B > total) return -2;
  pool_item* P = (pool_item*)malloc(sizeof(pool_item) * (size_t)(total > 0 ? total : 1));
  if (!P) return -1;
  for (int32_t l = 0; l < L; ++l)
    for (int64_t kk = 0; kk < N; ++kk) {
      pool_item* p = &P[(int64_t)l * N + kk];
      p->v = I[(int64_t)l * N + kk];
      p->l = l;
      p->k = kk;
    }
  qsort(P, (size_t)total, sizeof(pool_item), pool_cmp);
  for (int32_t l = 0; l < L; ++l) n_keep[l] = 0;
  for (int64_t i = 0; i < B; ++i) n_keep[P[i].l] += 1;
  free(P);
  offsets[0] = 0;
  for (int32_t l = 0; l < L; ++l) offsets[l + 1] = offsets[l] + n_keep[l];
  return 0;
}

/*
 * Eqs. (20)-(22) with a per-layer minimum (an option the paper does not have: nothing in
 * Sec. 3.3 keeps a layer from getting no slot at all).  Every layer first keeps its
 * min_keep best composite tokens; the remaining B - L * min_keep slots go to the best of
 * all other pooled entries under the same total order.  min_keep = 0 is oracle_allocate.
 */
int oracle_allocate_floor(const double* I, int32_t L, int64_t N, int64_t B, int64_t min_keep,
                          int32_t* n_keep, int64_t* offsets) {
  if (min_keep < 0 || min_keep > N || (int64_t)L * min_keep > B) return -2;
  int64_t rest = N - min_keep;
  int64_t total = (int64_t)L * rest;
  int64_t Brest = B - (int64_t)L * min_keep;
  if (Brest > total) return -2;
  pool_item* P = (pool_item*)malloc(sizeof(pool_item) * (size_t)(total > 0 ? total : 1));
  if (!P) return -1;
  for (int32_t l = 0; l < L; ++l)
    for (int64_t kk = min_keep; kk < N; ++kk) {
      pool_item* p = &P[(int64_t)l * rest + (kk - min_keep)];
      p->v = I[(int64_t)l * N + kk];
      p->l = l;
      p->k = kk;
    }
  qsort(P, (size_t)total, sizeof(pool_item), pool_cmp);
  for (int32_t l = 0; l < L; ++l) n_keep[l] = (int32_t)min_keep;
  for (int64_t i = 0; i < Brest; ++i) n_keep[P[i].l] += 1;
  free(P);
  offsets[0] = 0;
  for (int32_t l = 0; l < L; ++l) offsets[l + 1] = offsets[l] + n_keep[l];
  return 0;
}

/* ------------------------------------------------------------------------- */
/* App. A.2: the unstructured variant                                          */
/* ------------------------------------------------------------------------- */

typedef struct {
  double v;
  int32_t l, h;
  int64_t c;
} entry_item;

/* order: score descending, then layer, head, position ascending */
static int entry_cmp(const void* a, const void* b) {
  const entry_item* x = (const entry_item*)a;
  const entry_item* y = (const entry_item*)b;
  if (x->v > y->v) return -1;
  if (x->v < y->v) return 1;
  if (x->l != y->l) return x->l < y->l ? -1 : 1;
  if (x->h != y->h) return x->h < y->h ? -1 : 1;
  if (x->c < y->c) return -1;
  if (x->c > y->c) return 1;
  return 0;
}

/*
 * App. A.2 ("Discussion on unstructured eviction methods"): the final aggregation over the
 * heads (Eq. 19) is left out and every head keeps its own tokens.  All entries S[l, h, c]
 * of one sequence form one pool; the B best are kept (ties: layer, head, position
 * ascending); n_keep[l, h] = how many of them lie in head h of layer l -- those are the
 * head's n_keep[l, h] best tokens, i.e. the first n_keep[l, h] entries of its ranking
 * (Eq. 17).  offsets = exclusive prefix sum over (l, h) in that order.
 *   S [L, Hkv, N] -> n_keep [L * Hkv], offsets [L * Hkv + 1].
 */
int oracle_select_unstructured(const double* S, int32_t L, int32_t Hkv, int64_t N, int64_t B,
                               int32_t* n_keep, int64_t* offsets) {
  int64_t total = (int64_t)L * Hkv * N;
  if (B < 0 || B > total) return -2;
  entry_item* P = (entry_item*)malloc(sizeof(entry_item) * (size_t)(total > 0 ? total : 1));
  if (!P) return -1;
  for (int32_t l = 0; l < L; ++l)
    for (int32_t h = 0; h < Hkv; ++h)
      for (int64_t c = 0; c < N; ++c) {
        entry_item* p = &P[((int64_t)l * Hkv + h) * N + c];
        p->v = S[((int64_t)l * Hkv + h) * N + c];
        p->l = l;
        p->h = h;
        p->c = c;
      }
  qsort(P, (size_t)total, sizeof(entry_item), entry_cmp);
  for (int32_t r = 0; r < L * Hkv; ++r) n_keep[r] = 0;
  for (int64_t i = 0; i < B; ++i) n_keep[P[i].l * Hkv + P[i].h] += 1;
  free(P);
  offsets[0] = 0;
  for (int32_t r = 0; r < L * Hkv; ++r) offsets[r + 1] = offsets[r] + n_keep[r];
  return 0;
}

static int int32_cmp(const void* a, const void* b) {
  int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
  return x < y ? -1 : (x > y ? 1 : 0);
}

/*
 * Output order option: the kept tokens of a head in their original order.
 * idx [Hkv, N] (Eq. 17), n_keep[h] kept per head -> out [Hkv, N]: out[h, :n_keep[h]] are the
 * positions idx[h, :n_keep[h]] in ascending order; the rest of the row is copied unchanged.
 */
void oracle_sort_kept(const int32_t* idx, int32_t Hkv, int64_t N, const int32_t* n_keep,
                      int32_t* out) {
  memcpy(out, idx, sizeof(int32_t) * (size_t)Hkv * (size_t)N);
  for (int32_t h = 0; h < Hkv; ++h)
    qsort(out + (int64_t)h * N, (size_t)n_keep[h], sizeof(int32_t), int32_cmp);
}

/* ------------------------------------------------------------------------- */
/* Step 8: gather, Eqs. (23)-(24)                                              */
/* ------------------------------------------------------------------------- */

/*
 * One layer, one tensor (K or V), raw bytes:
 *   src [Hkv, N, row_bytes], idx [Hkv, N]  ->  dst [Hkv, n_keep, row_bytes]
 *   dst[h, kk, :] = src[h, idx[h, kk], :]   for kk < n_keep.
 */
void oracle_gather_layer(const uint8_t* src, const int32_t* idx, int32_t Hkv, int64_t N,
                         int64_t row_bytes, int32_t n_keep, uint8_t* dst) {
  for (int32_t h = 0; h < Hkv; ++h)
    for (int32_t kk = 0; kk < n_keep; ++kk) {
      int64_t c = idx[(int64_t)h * N + kk];
      memcpy(dst + ((int64_t)h * n_keep + kk) * row_bytes,
             src + ((int64_t)h * N + c) * row_bytes, (size_t)row_bytes);
    }
}

/* ------------------------------------------------------------------------- */
/* Whole pass for one sequence (used for the end-to-end check and for timing). */
/* ------------------------------------------------------------------------- */

/*
 * q [L, Hq, w, d] float, k [L, Hkv, N, d] float (for scoring),
 * k_raw / v_raw [L, Hkv, N, row_bytes] bytes in the cache's own dtype (for the gather),
 * outputs: S [L, Hkv, N], idx [L, Hkv, N], I [L, N], n_keep [L], offsets [L+1],
 * k_out / v_out [B * Hkv * row_bytes] packed: layer l starts at
 * offsets[l] * Hkv * row_bytes and has shape [Hkv, n_keep[l], row_bytes].
 * Any of S, I, k_out, v_out may be NULL (S and I are then kept internally).
 */
int oracle_compress(const float* q, const float* k, const uint8_t* k_raw,
                    const uint8_t* v_raw, int32_t L, int32_t Hq, int32_t Hkv, int64_t N,
                    int32_t d, int32_t w, int64_t row_bytes, double scale, int64_t q_pos0,
                    int32_t agg_task, int32_t agg_group, int32_t agg_head, int32_t augment,
                    const int32_t* q_to_kv, int64_t B, double* S_out, int32_t* idx,
                    double* I_out, int32_t* n_keep, int64_t* offsets, uint8_t* k_out,
                    uint8_t* v_out) {
  size_t per_layer = (size_t)Hkv * (size_t)N;
  double* S = S_out ? S_out : (double*)malloc(sizeof(double) * per_layer * (size_t)L);
  double* I = I_out ? I_out : (double*)malloc(sizeof(double) * (size_t)N * (size_t)L);
  double* S_sorted = (double*)malloc(sizeof(double) * per_layer);
  int rc = 0;
  if (!S || !I || !S_sorted) rc = -1;
  for (int32_t l = 0; l < L && rc == 0; ++l) {
    rc = oracle_score_layer(q + (int64_t)l * Hq * w * d, k + (int64_t)l * Hkv * N * d, Hq,
                            Hkv, N, d, w, scale, q_pos0, agg_task, agg_group, augment,
                            q_to_kv, S + l * per_layer);
    if (rc) break;
    int bad = 0;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(dynamic, 1)
#endif
    for (int32_t h = 0; h < Hkv; ++h) {
      if (oracle_rank(S + l * per_layer + (int64_t)h * N, N,
                      idx + l * (int64_t)per_layer + (int64_t)h * N,
                      S_sorted + (int64_t)h * N)) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
        bad = 1;
      }
    }
    if (bad) rc = -1;
    if (rc == 0) oracle_compose(S_sorted, Hkv, N, agg_head, I + (int64_t)l * N);
  }
  if (rc == 0) rc = oracle_allocate(I, L, N, B, n_keep, offsets);
  if (rc == 0 && k_out && v_out && k_raw && v_raw) {
    for (int32_t l = 0; l < L; ++l) {
      int64_t src_off = (int64_t)l * Hkv * N * row_bytes;
      int64_t dst_off = offsets[l] * Hkv * row_bytes;
      oracle_gather_layer(k_raw + src_off, idx + l * (int64_t)per_layer, Hkv, N, row_bytes,
                          n_keep[l], k_out + dst_off);
      oracle_gather_layer(v_raw + src_off, idx + l * (int64_t)per_layer, Hkv, N, row_bytes,
                          n_keep[l], v_out + dst_off);
    }
  }
  free(S_sorted);
  if (!S_out) free(S);
  if (!I_out) free(I);
  return rc;
}
