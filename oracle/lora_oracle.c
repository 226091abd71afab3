/*
 * CPU oracle for batch LoRA inference.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain, per-token definition that the CUDA library is
 * checked against.  It shares no code with the CUDA path and is never used by
 * it.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it.
 *
 * What it computes (paper Section 3.4, the displayed batch equation, taken in
 * the "per-sample" baseline form of Section 4.3, i.e. no grouping, no tiling):
 *
 *     y[t] = W x[t] + s_a * B_a (A_a x[t]),   a = adapter_id[t],
 *     a = -1  =>  y[t] = W x[t].
 *
 * Shapes follow Section 2.1: A_a is r_a x h_in, B_a is h_out x r_a (the paper
 * writes the square case d x d; here W is h_out x h_in).  The paper's equation
 * carries no scale; the per-adapter scalar s_a (alpha / r in common LoRA use)
 * multiplies the low-rank term once.
 *
 * All inputs are bfloat16 bit patterns (uint16), widened exactly to double.
 * All sums are fp64, index ascending, never rounded in between.  The output is
 * kept in fp64.
 *
 * Routing (Section 3.4 "u-batch", Section 4.3 "maps adapter IDs to sample
 * indices"): segments are maximal runs of equal ids in token order; groups are
 * the tokens of one id, ids ascending with -1 first, token order kept inside a
 * group.
 */
#include <stdint.h>
#include <string.h>
#include <stddef.h>

/* bfloat16 is the upper half of an IEEE binary32. */
static double bf16_to_double(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/*
 * Batch LoRA linear, per token.
 *   W        [h_out][h_in]      bf16
 *   x        [T][h_in]          bf16
 *   ids      [T]                slot index or -1
 *   A[a]     [rank[a]][h_in]    bf16, dense (no padding), NULL if slot empty
 *   B[a]     [h_out][rank[a]]   bf16, dense
 *   y        [T][h_out]         fp64 out
 * Returns 0, or -1 if an id is outside [-1, n_slots) or names an empty slot
 * (nothing is written for the offending token or later ones in that case).
 */
int oracle_lora_linear(const uint16_t *W, const uint16_t *x, const int32_t *ids,
                       int32_t T, int32_t h_in, int32_t h_out, int32_t n_slots,
                       const uint16_t *const *A, const uint16_t *const *B,
                       const int32_t *rank, const float *scale, double *y) {
  int bad = 0;
  for (int32_t t = 0; t < T; ++t) {
    int32_t a = ids[t];
    if (a < -1 || a >= n_slots || (a >= 0 && (A[a] == NULL || B[a] == NULL)))
      bad = 1;
  }
  if (bad) return -1;

#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t t = 0; t < T; ++t) {
    const uint16_t *xt = x + (size_t)t * h_in;
    double *yt = y + (size_t)t * h_out;
    int32_t a = ids[t];

    /* base part: y[t][j] = sum_k W[j][k] x[t][k] */
    for (int32_t j = 0; j < h_out; ++j) {
      const uint16_t *Wj = W + (size_t)j * h_in;
      double acc = 0.0;
      for (int32_t k = 0; k < h_in; ++k)
        acc += bf16_to_double(Wj[k]) * bf16_to_double(xt[k]);
      yt[j] = acc;
    }
    if (a < 0) continue;

    /* low-rank part: z = A_a x[t];  y[t] += s_a * B_a z */
    int32_t r = rank[a];
    double s = (double)scale[a];
    double z[1024];
    if (r > 1024) r = 1024; /* caller never passes more; keeps z on the stack */
    for (int32_t i = 0; i < r; ++i) {
      const uint16_t *Ai = A[a] + (size_t)i * h_in;
      double acc = 0.0;
      for (int32_t k = 0; k < h_in; ++k)
        acc += bf16_to_double(Ai[k]) * bf16_to_double(xt[k]);
      z[i] = acc;
    }
    for (int32_t j = 0; j < h_out; ++j) {
      const uint16_t *Bj = B[a] + (size_t)j * rank[a];
      double acc = 0.0;
      for (int32_t i = 0; i < r; ++i) acc += bf16_to_double(Bj[i]) * z[i];
      yt[j] += s * acc;
    }
  }
  return 0;
}

/*
 * Projection form used to check every token of a full-size batch: for a given
 * v[h_out] (fp64) returns p[t] = sum_j v[j] * y[t][j].  By linearity
 *     p[t] = (v^T W) x[t] + s_a (v^T B_a) (A_a x[t]).
 * Pinned against oracle_lora_linear by the CPU tests.
 *   vW   scratch [h_in] fp64;  vB scratch [n_slots][max_rank] fp64
 */
int oracle_lora_projection(const uint16_t *W, const uint16_t *x, const int32_t *ids,
                           int32_t T, int32_t h_in, int32_t h_out, int32_t n_slots,
                           const uint16_t *const *A, const uint16_t *const *B,
                           const int32_t *rank, const float *scale, const double *v,
                           int32_t max_rank, double *vW, double *vB, double *p) {
  for (int32_t t = 0; t < T; ++t) {
    int32_t a = ids[t];
    if (a < -1 || a >= n_slots || (a >= 0 && (A[a] == NULL || B[a] == NULL))) return -1;
  }
  for (int32_t k = 0; k < h_in; ++k) vW[k] = 0.0;
  for (int32_t j = 0; j < h_out; ++j) {
    const uint16_t *Wj = W + (size_t)j * h_in;
    for (int32_t k = 0; k < h_in; ++k) vW[k] += v[j] * bf16_to_double(Wj[k]);
  }
  for (int32_t a = 0; a < n_slots; ++a) {
    double *vBa = vB + (size_t)a * max_rank;
    for (int32_t i = 0; i < max_rank; ++i) vBa[i] = 0.0;
    if (B[a] == NULL) continue;
    for (int32_t j = 0; j < h_out; ++j)
      for (int32_t i = 0; i < rank[a]; ++i)
        vBa[i] += v[j] * bf16_to_double(B[a][(size_t)j * rank[a] + i]);
  }
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t t = 0; t < T; ++t) {
    const uint16_t *xt = x + (size_t)t * h_in;
    int32_t a = ids[t];
    double acc = 0.0;
    for (int32_t k = 0; k < h_in; ++k) acc += vW[k] * bf16_to_double(xt[k]);
    if (a >= 0) {
      double lo = 0.0;
      for (int32_t i = 0; i < rank[a]; ++i) {
        const uint16_t *Ai = A[a] + (size_t)i * h_in;
        double z = 0.0;
        for (int32_t k = 0; k < h_in; ++k) z += bf16_to_double(Ai[k]) * bf16_to_double(xt[k]);
        lo += vB[(size_t)a * max_rank + i] * z;
      }
      acc += (double)scale[a] * lo;
    }
    p[t] = acc;
  }
  return 0;
}

/*
 * Segments: one left-to-right scan.  A new segment starts wherever the id
 * differs from the previous token's.  seg_start has n_seg + 1 entries (the last
 * is T).  Returns n_seg.
 */
int32_t oracle_segments(const int32_t *ids, int32_t T, int32_t *seg_start,
                        int32_t *seg_adapter) {
  int32_t n = 0;
  for (int32_t t = 0; t < T; ++t) {
    if (t == 0 || ids[t] != ids[t - 1]) {
      seg_start[n] = t;
      seg_adapter[n] = ids[t];
      ++n;
    }
  }
  seg_start[n] = T;
  return n;
}

/*
 * Groups (the paper's u-batches): for id = -1, 0, 1, ... in that order, list the
 * tokens carrying that id in token order.  perm[T] is the concatenation;
 * group_start has n_groups + 1 entries; ids with no token make no group.
 * Returns n_groups, or -1 on an id outside [-1, n_slots).
 */
int32_t oracle_groups(const int32_t *ids, int32_t T, int32_t n_slots, int32_t *perm,
                      int32_t *group_start, int32_t *group_adapter) {
  for (int32_t t = 0; t < T; ++t)
    if (ids[t] < -1 || ids[t] >= n_slots) return -1;
  int32_t n = 0, pos = 0;
  for (int32_t a = -1; a < n_slots; ++a) {
    int32_t first = pos;
    for (int32_t t = 0; t < T; ++t)
      if (ids[t] == a) perm[pos++] = t;
    if (pos > first) {
      group_start[n] = first;
      group_adapter[n] = a;
      ++n;
    }
  }
  group_start[n] = T;
  return n;
}
