/*
 * CPU oracle for the Lookahead Q-Cache (LAQ) re-eviction step -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what Section 4.3 (Eq. 4) computes, with the steps the
 * equation leaves implicit (scale, softmax, GQA sum, average pooling, retained tail) taken from
 * the "standard KV cache eviction" the paper builds on (Sections 1 and 5.1, SnapKV's average
 * pooling). It shares no code with the CUDA library and must never be called from it: only the
 * tests, the smoke check and the benchmark's cpu_baseline leg may use this file.
 *
 * Inputs are bf16 bit patterns (uint16_t), converted exactly to double. Every loop is the
 * definition written out; there is no blocking, fusion or reordering. OpenMP is used only
 * across independent (layer, batch, KV head) units in laq_oracle_evict.
 *
 * Pins (tests/test_oracle_pins.py): brute-force softmax on tiny inputs, torch.softmax /
 * torch.topk in fp64 as independent library routines, row sums = 1, sum of column sums = M,
 * identical-key closed forms for pooling and tie-break, key-shift invariance, additivity over
 * heads and queries, budget nestedness, planted key kept.
 * Parity unpinned by the paper: the softmax reading of Eq. 4, the sum over the GQA group, the
 * average pool with zero padding and divisor k, and the retained tail are conventions fixed by
 * the problem statement this oracle was written for, not by a value the paper prints.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/*
 * Steps 1-3 of the unit computation (Eq. 4, "sum_{q_i in Q} q_i K^T", read as attention
 * weights): logits, per-row softmax over all L keys, column sums over the G*W rows.
 *   q        [G][W][D] bf16, the lookahead queries of the G query heads that share this KV head
 *   k        [L][D]    bf16, prompt keys of this KV head
 *   c        [L]       out: c[j] = sum_r P[r][j]
 *   row_max  [G*W]     out (may be NULL): m_r
 *   row_sum  [G*W]     out (may be NULL): l_r
 */
void laq_oracle_unit_colsum_local(const uint16_t* q, const uint16_t* k, int G, int W, int W_local,
                                  int D, int L, double scale, double* c, double* row_max,
                                  double* row_sum);

void laq_oracle_unit_colsum(const uint16_t* q, const uint16_t* k, int G, int W, int D, int L,
                            double scale, double* c, double* row_max, double* row_sum) {
  laq_oracle_unit_colsum_local(q, k, G, W, 0, D, L, scale, c, row_max, row_sum);
}

/*
 * The same with the unified observation window of LAQ++ (Eq. 5: the sum runs over W u Q): the
 * first W_local of each head's W queries are the queries of the last W_local prompt positions
 * (query i sits at position L - W_local + i), the remaining W - W_local are lookahead queries.
 * A local query attends causally, to the keys at positions <= its own; a lookahead query sees
 * every prompt key. Keys a row cannot see get probability 0 from that row.
 */
void laq_oracle_unit_colsum_local(const uint16_t* q, const uint16_t* k, int G, int W, int W_local,
                                  int D, int L, double scale, double* c, double* row_max,
                                  double* row_sum) {
  const int M = G * W;
  double* s = (double*)malloc((size_t)L * sizeof(double));
  for (int j = 0; j < L; ++j) c[j] = 0.0;
  for (int r = 0; r < M; ++r) {
    /* logits of row r against every key (Eq. 4: q_i K^T, scaled) */
    for (int j = 0; j < L; ++j) {
      double acc = 0.0;
      for (int d = 0; d < D; ++d)
        acc += bf16_to_double(q[(size_t)r * D + d]) * bf16_to_double(k[(size_t)j * D + d]);
      s[j] = scale * acc;
    }
    /* keys this row can see: all of them for a lookahead query, positions <= its own for a
     * local query (row r is query i = r mod W of head r / W) */
    const int i = r % W;
    const int vis = i < W_local ? L - W_local + i + 1 : L;
    /* softmax over the visible prompt keys */
    double m = s[0];
    for (int j = 1; j < vis; ++j)
      if (s[j] > m) m = s[j];
    double l = 0.0;
    for (int j = 0; j < vis; ++j) l += exp(s[j] - m);
    /* Eq. 4 / Eq. 5: the sum over the window (and over the heads of the group) */
    for (int j = 0; j < vis; ++j) c[j] += exp(s[j] - m) / l;
    if (row_max) row_max[r] = m;
    if (row_sum) row_sum[r] = l;
  }
  free(s);
}

/*
 * Column sums of each query head on its own: c_heads[g][j] = sum_{i<W} P[(g,i)][j]. The rows of
 * different heads do not interact (every row has its own softmax), so head g is the unit
 * computation above with that head's W queries alone. Row g of c_heads starts at g*row_stride.
 */
void laq_oracle_unit_colsum_heads(const uint16_t* q, const uint16_t* k, int G, int W, int W_local,
                                  int D, int L, double scale, double* c_heads, int64_t row_stride) {
  for (int g = 0; g < G; ++g)
    laq_oracle_unit_colsum_local(q + (size_t)g * W * D, k, 1, W, W_local, D, L, scale,
                                 c_heads + g * row_stride, NULL, NULL);
}

/*
 * How the G query heads that share a KV head are combined into one importance per key (the
 * paper does not define it): mode 0 adds them (the reading used throughout), mode 1 takes the
 * largest, so that a key one head attends to strongly is not averaged away by the others.
 */
void laq_oracle_group_reduce(const double* c_heads, int G, int L, int mode, double* c) {
  for (int j = 0; j < L; ++j) {
    double acc = c_heads[j];
    for (int g = 1; g < G; ++g) {
      const double x = c_heads[(size_t)g * L + j];
      if (mode == 1) {
        if (x > acc) acc = x;
      } else {
        acc += x;
      }
    }
    c[j] = acc;
  }
}

/*
 * Step 4: average pooling over the scored positions [0, Ls), stride 1, zero padding of k/2 on
 * both sides, divisor always k (SnapKV-style pooling, Section 5.1 "employs average pooling").
 */
void laq_oracle_pool(const double* c, int Ls, int kernel, double* p) {
  const int h = kernel / 2;
  for (int j = 0; j < Ls; ++j) {
    double acc = 0.0;
    for (int t = -h; t <= h; ++t) {
      const int jj = j + t;
      if (jj >= 0 && jj < Ls) acc += c[jj];
    }
    p[j] = acc / (double)kernel;
  }
}

/*
 * Step 4 with maximum pooling instead (the other pooling the SnapKV-style step is used with):
 * p_j = max of c over the window positions that exist, |t| <= k/2 and 0 <= j+t < Ls. Positions
 * outside [0, Ls) are not candidates (padding with minus infinity).
 */
void laq_oracle_pool_max(const double* c, int Ls, int kernel, double* p) {
  const int h = kernel / 2;
  for (int j = 0; j < Ls; ++j) {
    double best = c[j];
    for (int t = -h; t <= h; ++t) {
      const int jj = j + t;
      if (jj >= 0 && jj < Ls && c[jj] > best) best = c[jj];
    }
    p[j] = best;
  }
}

/*
 * Eq. 4 read literally: the importance of key j is the sum of the raw (scaled) logits
 * "sum_{q_i in Q} q_i K^T" over the window rows, with no softmax. Same arguments as
 * laq_oracle_unit_colsum; c[j] may be negative.
 */
void laq_oracle_unit_rawsum(const uint16_t* q, const uint16_t* k, int G, int W, int D, int L,
                            double scale, double* c) {
  const int M = G * W;
  for (int j = 0; j < L; ++j) {
    double total = 0.0;
    for (int r = 0; r < M; ++r) {
      double acc = 0.0;
      for (int d = 0; d < D; ++d)
        acc += bf16_to_double(q[(size_t)r * D + d]) * bf16_to_double(k[(size_t)j * D + d]);
      total += scale * acc;
    }
    c[j] = total;
  }
}

/*
 * Step 5 (Eq. 4's ArgSort(...)[:B], descending): the Kb = B-R positions of largest p, a tie
 * going to the lower position; written ascending and followed by the tail Ls..L-1.
 * Selection by repeated scan for the best remaining position: O(Ls*Kb), obviously correct.
 */
void laq_oracle_select(const double* p, int L, int R, int B, int32_t* idx) {
  const int Ls = L - R, Kb = B - R;
  unsigned char* taken = (unsigned char*)calloc((size_t)(Ls > 0 ? Ls : 1), 1);
  for (int n = 0; n < Kb; ++n) {
    int best = -1;
    for (int j = 0; j < Ls; ++j) {
      if (taken[j]) continue;
      if (best < 0 || p[j] > p[best]) best = j; /* strict '>' keeps the lower position on ties */
    }
    taken[best] = 1;
  }
  int t = 0;
  for (int j = 0; j < Ls; ++j)
    if (taken[j]) idx[t++] = j;
  for (int j = Ls; j < L; ++j) idx[t++] = j;
  free(taken);
}

/* Same selection in O(Ls log Ls) for the timed baseline and large parity samples: sort positions
 * by (p descending, position ascending), keep the first Kb. Checked against laq_oracle_select. */
typedef struct {
  double p;
  int32_t j;
} laq_oracle_pair;

static int pair_cmp(const void* a, const void* b) {
  const laq_oracle_pair* x = (const laq_oracle_pair*)a;
  const laq_oracle_pair* y = (const laq_oracle_pair*)b;
  if (x->p > y->p) return -1;
  if (x->p < y->p) return 1;
  return (x->j > y->j) - (x->j < y->j);
}

static int int_cmp(const void* a, const void* b) {
  const int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
  return (x > y) - (x < y);
}

void laq_oracle_select_sorted(const double* p, int L, int R, int B, int32_t* idx) {
  const int Ls = L - R, Kb = B - R;
  laq_oracle_pair* a = (laq_oracle_pair*)malloc((size_t)(Ls > 0 ? Ls : 1) * sizeof *a);
  for (int j = 0; j < Ls; ++j) {
    a[j].p = p[j];
    a[j].j = j;
  }
  qsort(a, (size_t)Ls, sizeof *a, pair_cmp);
  for (int t = 0; t < Kb; ++t) idx[t] = a[t].j;
  qsort(idx, (size_t)Kb, sizeof *idx, int_cmp);
  for (int j = Ls; j < L; ++j) idx[Kb + (j - Ls)] = j;
  free(a);
}

/* Step 6: bit copies of the kept rows. src [L][D], dst [B][D], bf16 bit patterns. */
void laq_oracle_compact(const uint16_t* src, const int32_t* idx, int B, int D, uint16_t* dst) {
  for (int t = 0; t < B; ++t)
    for (int d = 0; d < D; ++d) dst[(size_t)t * D + d] = src[(size_t)idx[t] * D + d];
}

/*
 * The whole step for densely packed tensors:
 *   Q [NL][Bt][Hq][W][D], K and V [NL][Bt][Hkv][L][D]  (bf16 bit patterns)
 *   scores [NL][Bt][Hkv][L-R] pooled (may be NULL), colsum [NL][Bt][Hkv][L] (may be NULL),
 *   idx [NL][Bt][Hkv][B] (may be NULL; then k_out/v_out are not written),
 *   k_out, v_out [NL][Bt][Hkv][B][D] (may be NULL).
 * `unit_list` (may be NULL) restricts the work to n_units listed unit numbers
 * u = (layer*Bt + b)*Hkv + h; outputs of other units are left untouched.
 * Query head h*G+g belongs to KV head h. Returns the number of OpenMP threads used.
 */
/*
 * Variants of the step (all off when the structure is zeroed):
 *   W_local    unified window of LAQ++ (Eq. 5), see laq_oracle_unit_colsum_local
 *   pool_mode  0 average pooling, 1 maximum pooling
 *   score_mode 0 attention weights (softmax), 1 raw logit sums (Eq. 4 read literally)
 *   group_mode 0: the G heads of a group are summed (one kept set per KV head); 1: the largest
 *              head counts (one kept set per KV head); 2: every query head selects for itself:
 *              scores are then [NL][Bt][Hq][L-R], idx [NL][Bt][Hq][B], k_out / v_out
 *              [NL][Bt][Hq][B][D], head h*G+g gathering from KV head h (softmax scoring only)
 *   seq_lens   [Bt] or NULL: prompt b holds only its first seq_lens[b] <= L positions. Everything
 *              is then taken relative to that length Lb: keys [0, Lb), local queries at the last
 *              W_local of them, scored positions [0, Lb-R), tail [Lb-R, Lb). Scores and column
 *              sums beyond are written as 0; rows of K/V beyond Lb are never read.
 */
typedef struct {
  int32_t W_local, pool_mode, score_mode, group_mode;
  const int32_t* seq_lens;
} laq_oracle_variant;

int laq_oracle_evict_variant(const uint16_t* q, const uint16_t* k, const uint16_t* v, int NL, int Bt,
                             int Hq, int Hkv, int D, int L, int W, int R, int kernel, int B,
                             double scale, const laq_oracle_variant* var, const int64_t* unit_list,
                             int64_t n_units, double* scores, double* colsum, int32_t* idx,
                             uint16_t* k_out, uint16_t* v_out, int fast_select);

int laq_oracle_evict_local(const uint16_t* q, const uint16_t* k, const uint16_t* v, int NL, int Bt,
                           int Hq, int Hkv, int D, int L, int W, int W_local, int R, int kernel, int B,
                           double scale, const int64_t* unit_list, int64_t n_units, double* scores,
                           double* colsum, int32_t* idx, uint16_t* k_out, uint16_t* v_out,
                           int fast_select) {
  laq_oracle_variant var;
  memset(&var, 0, sizeof var);
  var.W_local = W_local;
  return laq_oracle_evict_variant(q, k, v, NL, Bt, Hq, Hkv, D, L, W, R, kernel, B, scale, &var,
                                  unit_list, n_units, scores, colsum, idx, k_out, v_out, fast_select);
}

int laq_oracle_evict_variant(const uint16_t* q, const uint16_t* k, const uint16_t* v, int NL, int Bt,
                             int Hq, int Hkv, int D, int L, int W, int R, int kernel, int B,
                             double scale, const laq_oracle_variant* var, const int64_t* unit_list,
                             int64_t n_units, double* scores, double* colsum, int32_t* idx,
                             uint16_t* k_out, uint16_t* v_out, int fast_select) {
  const int G = Hq / Hkv;
  const int64_t U = (int64_t)NL * Bt * Hkv;
  const int64_t n = unit_list ? n_units : U;
  int threads = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    threads = omp_get_num_threads();
  }
#pragma omp parallel for schedule(dynamic, 1)
#endif
  for (int64_t t = 0; t < n; ++t) {
    const int64_t u = unit_list ? unit_list[t] : t;
    const int64_t h = u % Hkv;
    const int64_t lb = u / Hkv; /* layer*Bt + b */
    const uint16_t* qu = q + ((lb * Hq + h * G) * (int64_t)W) * D;
    const uint16_t* ku = k + u * (int64_t)L * D;
    /* this prompt's own length, and the scored positions that follow from it */
    const int Lb = var->seq_lens ? var->seq_lens[lb % Bt] : L;
    const int Ls = Lb - R;
    double* c = (double*)calloc((size_t)L, sizeof(double));
    double* p = (double*)calloc((size_t)(L - R > 0 ? L - R : 1), sizeof(double));
    if (var->group_mode != 0 && var->score_mode == 0) {
      /* per-head column sums, then either their maximum or one selection per query head */
      double* ch = (double*)calloc((size_t)G * L, sizeof(double));
      laq_oracle_unit_colsum_heads(qu, ku, G, W, var->W_local, D, Lb, scale, ch, L);
      if (var->group_mode == 2) {
        for (int g = 0; g < G; ++g) {
          const int64_t uh = u * G + g; /* (layer*Bt + b)*Hq + h*G + g */
          const double* cg = ch + (size_t)g * L;
          if (var->pool_mode == 1)
            laq_oracle_pool_max(cg, Ls, kernel, p);
          else
            laq_oracle_pool(cg, Ls, kernel, p);
          if (colsum) memcpy(colsum + uh * (int64_t)L, cg, (size_t)L * sizeof(double));
          if (scores) memcpy(scores + uh * (int64_t)(L - R), p, (size_t)(L - R) * sizeof(double));
          if (idx) {
            int32_t* iu = idx + uh * (int64_t)B;
            if (fast_select)
              laq_oracle_select_sorted(p, Lb, R, B, iu);
            else
              laq_oracle_select(p, Lb, R, B, iu);
            if (k_out) laq_oracle_compact(ku, iu, B, D, k_out + uh * (int64_t)B * D);
            if (v_out) laq_oracle_compact(v + u * (int64_t)L * D, iu, B, D, v_out + uh * (int64_t)B * D);
          }
        }
        free(ch);
        free(c);
        free(p);
        continue;
      }
      laq_oracle_group_reduce(ch, G, L, var->group_mode, c);
      free(ch);
    } else if (var->score_mode == 1)
      laq_oracle_unit_rawsum(qu, ku, G, W, D, Lb, scale, c);
    else
      laq_oracle_unit_colsum_local(qu, ku, G, W, var->W_local, D, Lb, scale, c, NULL, NULL);
    if (var->pool_mode == 1)
      laq_oracle_pool_max(c, Ls, kernel, p);
    else
      laq_oracle_pool(c, Ls, kernel, p);
    if (colsum) memcpy(colsum + u * (int64_t)L, c, (size_t)L * sizeof(double));
    if (scores) memcpy(scores + u * (int64_t)(L - R), p, (size_t)(L - R) * sizeof(double));
    if (idx) {
      int32_t* iu = idx + u * (int64_t)B;
      if (fast_select)
        laq_oracle_select_sorted(p, Lb, R, B, iu);
      else
        laq_oracle_select(p, Lb, R, B, iu);
      if (k_out) laq_oracle_compact(ku, iu, B, D, k_out + u * (int64_t)B * D);
      if (v_out) laq_oracle_compact(v + u * (int64_t)L * D, iu, B, D, v_out + u * (int64_t)B * D);
    }
    free(c);
    free(p);
  }
  return threads;
}

int laq_oracle_evict(const uint16_t* q, const uint16_t* k, const uint16_t* v, int NL, int Bt,
                     int Hq, int Hkv, int D, int L, int W, int R, int kernel, int B,
                     double scale, const int64_t* unit_list, int64_t n_units, double* scores,
                     double* colsum, int32_t* idx, uint16_t* k_out, uint16_t* v_out,
                     int fast_select) {
  return laq_oracle_evict_local(q, k, v, NL, Bt, Hq, Hkv, D, L, W, 0, R, kernel, B, scale, unit_list,
                                n_units, scores, colsum, idx, k_out, v_out, fast_select);
}

/*
 * Recall of a selected index set against a gold one (Section 3, Eq. 1-3):
 * |M_pred n M_gold| / |M_gold|, by comparing every pair. Both sets hold distinct positions;
 * no order is assumed. Returns the size of the intersection through *n_common.
 */
double laq_oracle_recall(const int32_t* pred, int n_pred, const int32_t* gold, int n_gold,
                         int32_t* n_common) {
  int common = 0;
  for (int a = 0; a < n_pred; ++a)
    for (int b = 0; b < n_gold; ++b)
      if (pred[a] == gold[b]) {
        ++common;
        break;
      }
  if (n_common) *n_common = common;
  return n_gold > 0 ? (double)common / (double)n_gold : 0.0;
}
