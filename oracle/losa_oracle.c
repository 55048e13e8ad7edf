/*
 * fp64 CPU oracle for LoSA's attention hot path.  TEST INFRASTRUCTURE ONLY:
 * the tests, the smoke check and the benchmark's CPU-baseline leg may call it;
 * the CUDA library never does, and the two share no code.
 *
 * Everything is the plain definition, in double precision, one query row at a
 * time, with no tiling, no online rescaling and no fusion:
 *
 *   scores   s(q,k) = (Q(q) . K(k)) * scale             ("Measuring Sparse Attention
 *   probs    A(q,k) = exp(s - max_k s) / sum_k exp(..)    by Retained Mass": A = row-wise
 *                                                          softmax(Q K^T / sqrt(d)))
 *   mass     M(i,j) = sum_{q in B^Q_i} sum_{k in B^K_j} A(q,k)            (Eq. 1)
 *            stored divided by the number of valid rows of B^Q_i, so that
 *            sum_j mass(i,j) = 1 and the threshold theta*R of Eq. 3 becomes tau.
 *   top-k    the k heaviest blocks of every row (the fixed-ratio ablation rule)
 *   select   pi = blocks by decreasing mass (equal masses: lower index first),
 *            s = min{ m >= 1 : sum_{r<=m} mass(pi(r)) >= tau },  Omega = pi(1..s)  (Eq. 3)
 *   sparse   O(q) = sum_{k in K(q)} softmax over K(q) only * V(k),
 *            K(q) = union of the retained key blocks of q's query block   (Eq. 4)
 *   dense    O(q) = sum_k A(q,k) V(k)
 *
 * Inputs are float arrays that hold the bf16 input values exactly, laid out
 * [B, H, N, D] contiguous.  N is the number of valid tokens; the last query or
 * key block may be short.  Tokens >= N do not exist: they enter no softmax and
 * no mass, and short query blocks are averaged over their valid rows.
 *
 * Parity pins: every function here is checked by the CPU test-suite against
 * closed forms, brute force on a materialised A, torch's fp64 attention, and
 * subset enumeration (see tests/test_oracle_*.py).  No function is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int losa_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static void widen(const float* src, double* dst, int64_t n) {
  for (int64_t i = 0; i < n; ++i) dst[i] = (double)src[i];
}

/* s_k = (q . K_k) * scale for every key k < N with keep[k] != 0 (keep == NULL: all). */
static void score_row(const double* q, const double* K, int N, int D, double scale, double* s,
                      const unsigned char* keep) {
  for (int k = 0; k < N; ++k) {
    if (keep && !keep[k]) {
      s[k] = 0.0;
      continue;
    }
    const double* kr = K + (int64_t)k * D;
    double acc = 0.0;
#pragma omp simd reduction(+ : acc)
    for (int c = 0; c < D; ++c) acc += q[c] * kr[c];
    s[k] = acc * scale;
  }
}

/* In place: s_k -> softmax probabilities over the keys with keep[k] != 0
 * (keep == NULL: all keys).  Keys that are not kept get probability 0.
 * Returns log(sum exp(s)) over the kept keys (natural log). */
static double softmax_row(double* s, int N, const unsigned char* keep) {
  double m = -INFINITY;
  for (int k = 0; k < N; ++k)
    if ((!keep || keep[k]) && s[k] > m) m = s[k];
  double z = 0.0;
  for (int k = 0; k < N; ++k) {
    if (!keep || keep[k]) {
      s[k] = exp(s[k] - m);
      z += s[k];
    } else {
      s[k] = 0.0;
    }
  }
  for (int k = 0; k < N; ++k) s[k] /= z;
  return m + log(z);
}

/* o_c = sum_k p_k V(k,c) */
static void apply_v(const double* p, const double* V, int N, int D, double* o) {
  for (int c = 0; c < D; ++c) o[c] = 0.0;
  for (int k = 0; k < N; ++k) {
    const double pk = p[k];
    if (pk == 0.0) continue;
    const double* vr = V + (int64_t)k * D;
#pragma omp simd
    for (int c = 0; c < D; ++c) o[c] += pk * vr[c];
  }
}

/* Dense attention, all rows.  o: double [B,H,N,D]. */
int losa_oracle_dense_attn(const float* q, const float* k, const float* v, int B, int H, int N,
                           int D, double scale, double* o) {
  const int64_t hd = (int64_t)N * D;
  double* K = (double*)malloc(sizeof(double) * hd);
  double* V = (double*)malloc(sizeof(double) * hd);
  if (!K || !V) return -1;
  for (int bh = 0; bh < B * H; ++bh) {
    widen(k + bh * hd, K, hd);
    widen(v + bh * hd, V, hd);
#pragma omp parallel
    {
      double* s = (double*)malloc(sizeof(double) * N);
      double* qd = (double*)malloc(sizeof(double) * D);
#pragma omp for schedule(dynamic, 4)
      for (int r = 0; r < N; ++r) {
        widen(q + bh * hd + (int64_t)r * D, qd, D);
        score_row(qd, K, N, D, scale, s, NULL);
        softmax_row(s, N, NULL);
        apply_v(s, V, N, D, o + bh * hd + (int64_t)r * D);
      }
      free(s);
      free(qd);
    }
  }
  free(K);
  free(V);
  return 0;
}

/* Block attention mass (Eq. 1, averaged over the valid rows of the query block)
 * for the query blocks listed in row_ids (flattened (b*H + h)*nQb + i; NULL = all
 * B*H*nQb blocks in order).  mass: double [n_rows, nKb].  lse (may be NULL):
 * double [n_rows, R], natural-log sum-exp of each valid row, 0 for rows >= N. */
int losa_oracle_block_mass(const float* q, const float* k, int B, int H, int N, int D, int R,
                           int C, double scale, int n_rows, const int32_t* row_ids, double* mass,
                           double* lse) {
  const int nQb = (N + R - 1) / R, nKb = (N + C - 1) / C;
  const int64_t hd = (int64_t)N * D;
  double* K = (double*)malloc(sizeof(double) * hd);
  double* rowmass = (double*)malloc(sizeof(double) * (int64_t)R * nKb);
  if (!K || !rowmass) return -1;
  int cached_bh = -1;
  for (int it = 0; it < n_rows; ++it) {
    const int rid = row_ids ? row_ids[it] : it;
    if (rid < 0 || rid >= B * H * nQb) return -2;
    const int bh = rid / nQb, i = rid % nQb;
    if (bh != cached_bh) {
      widen(k + bh * hd, K, hd);
      cached_bh = bh;
    }
    const int r0 = i * R;
    const int nvalid = (N - r0 < R) ? (N - r0) : R;
#pragma omp parallel
    {
      double* s = (double*)malloc(sizeof(double) * N);
      double* qd = (double*)malloc(sizeof(double) * D);
#pragma omp for schedule(dynamic, 1)
      for (int rr = 0; rr < nvalid; ++rr) {
        widen(q + bh * hd + (int64_t)(r0 + rr) * D, qd, D);
        score_row(qd, K, N, D, scale, s, NULL);
        const double l = softmax_row(s, N, NULL);
        if (lse) lse[(int64_t)it * R + rr] = l;
        for (int j = 0; j < nKb; ++j) {
          const int k1 = ((j + 1) * C < N) ? (j + 1) * C : N;
          double acc = 0.0;
          for (int kk = j * C; kk < k1; ++kk) acc += s[kk];
          rowmass[(int64_t)rr * nKb + j] = acc;
        }
      }
      free(s);
      free(qd);
    }
    if (lse)
      for (int rr = nvalid; rr < R; ++rr) lse[(int64_t)it * R + rr] = 0.0;
    for (int j = 0; j < nKb; ++j) {
      double acc = 0.0;
      for (int rr = 0; rr < nvalid; ++rr) acc += rowmass[(int64_t)rr * nKb + j];
      mass[(int64_t)it * nKb + j] = acc / (double)nvalid;
    }
  }
  free(K);
  free(rowmass);
  return 0;
}

typedef struct {
  double m;
  int32_t j;
} mass_key_t;

static int by_mass_desc_then_index(const void* a, const void* b) {
  const mass_key_t* x = (const mass_key_t*)a;
  const mass_key_t* y = (const mass_key_t*)b;
  if (x->m > y->m) return -1;
  if (x->m < y->m) return 1;
  return (x->j > y->j) - (x->j < y->j);
}

static int by_index(const void* a, const void* b) {
  const int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
  return (x > y) - (x < y);
}

/* Retained-mass selection (Eq. 3) on a [rows, nKb] mass matrix.
 *   order  int32 [rows, nKb]: pi, blocks by decreasing mass, equal masses by lower index
 *   cum    double [rows, nKb]: cumulative mass along pi, accumulated left to right
 *   count  int32 [rows]: s = smallest m >= 1 with cum[m-1] >= tau; nKb when tau >= 1
 *          or when no prefix reaches tau
 *   kept   int32 [rows, nKb]: the first count[r] entries of row r are Omega in
 *          ascending block index; the rest is -1 */
int losa_oracle_select(const double* mass, int rows, int nKb, double tau, int32_t* order,
                       double* cum, int32_t* count, int32_t* kept) {
  if (!(tau > 0.0)) return -2;
#pragma omp parallel
  {
    mass_key_t* keys = (mass_key_t*)malloc(sizeof(mass_key_t) * nKb);
#pragma omp for schedule(static)
    for (int r = 0; r < rows; ++r) {
      const double* mr = mass + (int64_t)r * nKb;
      for (int j = 0; j < nKb; ++j) {
        keys[j].m = mr[j];
        keys[j].j = j;
      }
      qsort(keys, nKb, sizeof(mass_key_t), by_mass_desc_then_index);
      double acc = 0.0;
      int s = -1;
      for (int m = 0; m < nKb; ++m) {
        acc += keys[m].m;
        order[(int64_t)r * nKb + m] = keys[m].j;
        cum[(int64_t)r * nKb + m] = acc;
        if (s < 0 && acc >= tau) s = m + 1;
      }
      if (s < 0 || tau >= 1.0) s = nKb;
      count[r] = s;
      int32_t* kr = kept + (int64_t)r * nKb;
      for (int m = 0; m < nKb; ++m) kr[m] = (m < s) ? keys[m].j : -1;
      qsort(kr, s, sizeof(int32_t), by_index);
    }
    free(keys);
  }
  return 0;
}

/* Fixed-ratio selection (the paper's ablation, "Retained mass versus fixed-ratio top-k
 * selection"): every row keeps its k heaviest blocks, equal masses by lower index.
 *   kept  int32 [rows, k]: the kept block indices of each row in ascending order */
int losa_oracle_select_topk(const double* mass, int rows, int nKb, int k, int32_t* kept) {
  if (k < 1 || k > nKb) return -2;
#pragma omp parallel
  {
    mass_key_t* keys = (mass_key_t*)malloc(sizeof(mass_key_t) * nKb);
#pragma omp for schedule(static)
    for (int r = 0; r < rows; ++r) {
      for (int j = 0; j < nKb; ++j) {
        keys[j].m = mass[(int64_t)r * nKb + j];
        keys[j].j = j;
      }
      qsort(keys, nKb, sizeof(mass_key_t), by_mass_desc_then_index);
      int32_t* kr = kept + (int64_t)r * k;
      for (int m = 0; m < k; ++m) kr[m] = keys[m].j;
      qsort(kr, k, sizeof(int32_t), by_index);
    }
    free(keys);
  }
  return 0;
}

/* Retained and total block mass of every row under a CSR pattern (the numerator and
 * denominator of Recall, Eq. 2, before the sum over heads and query blocks). */
int losa_oracle_row_recall(const double* mass, int rows, int nKb, const int32_t* offsets,
                           const int32_t* kv_idx, double* retained, double* total) {
  for (int r = 0; r < rows; ++r) {
    double tot = 0.0, ret = 0.0;
    for (int j = 0; j < nKb; ++j) tot += mass[(int64_t)r * nKb + j];
    for (int p = offsets[r]; p < offsets[r + 1]; ++p) {
      if (kv_idx[p] < 0 || kv_idx[p] >= nKb) return -3;
      ret += mass[(int64_t)r * nKb + kv_idx[p]];
    }
    retained[r] = ret;
    total[r] = tot;
  }
  return 0;
}

/* Attention over the retained key blocks only (Eq. 4), for the query blocks in
 * row_ids (NULL = all).  CSR: row r = (b*H + h)*nQb + i keeps key blocks
 * kv_idx[offsets[r] .. offsets[r+1]).  o: double [n_rows, R, D]; rows >= N are 0. */
int losa_oracle_sparse_attn(const float* q, const float* k, const float* v, int B, int H, int N,
                            int D, int R, int C, double scale, const int32_t* offsets,
                            const int32_t* kv_idx, int n_rows, const int32_t* row_ids,
                            double* o) {
  const int nQb = (N + R - 1) / R, nKb = (N + C - 1) / C;
  const int64_t hd = (int64_t)N * D;
  double* K = (double*)malloc(sizeof(double) * hd);
  double* V = (double*)malloc(sizeof(double) * hd);
  unsigned char* keep = (unsigned char*)malloc(N);
  if (!K || !V || !keep) return -1;
  int cached_bh = -1;
  for (int it = 0; it < n_rows; ++it) {
    const int rid = row_ids ? row_ids[it] : it;
    if (rid < 0 || rid >= B * H * nQb) return -2;
    const int bh = rid / nQb, i = rid % nQb;
    if (bh != cached_bh) {
      widen(k + bh * hd, K, hd);
      widen(v + bh * hd, V, hd);
      cached_bh = bh;
    }
    memset(keep, 0, N);
    if (offsets[rid + 1] <= offsets[rid]) return -4; /* Eq. 3 keeps at least one block */
    for (int p = offsets[rid]; p < offsets[rid + 1]; ++p) {
      const int j = kv_idx[p];
      if (j < 0 || j >= nKb) return -3;
      const int k1 = ((j + 1) * C < N) ? (j + 1) * C : N;
      for (int kk = j * C; kk < k1; ++kk) keep[kk] = 1;
    }
    const int r0 = i * R;
    const int nvalid = (N - r0 < R) ? (N - r0) : R;
    double* ob = o + (int64_t)it * R * D;
    memset(ob, 0, sizeof(double) * (int64_t)R * D);
#pragma omp parallel
    {
      double* s = (double*)malloc(sizeof(double) * N);
      double* qd = (double*)malloc(sizeof(double) * D);
#pragma omp for schedule(dynamic, 1)
      for (int rr = 0; rr < nvalid; ++rr) {
        widen(q + bh * hd + (int64_t)(r0 + rr) * D, qd, D);
        score_row(qd, K, N, D, scale, s, keep);
        softmax_row(s, N, keep);
        apply_v(s, V, N, D, ob + (int64_t)rr * D);
      }
      free(s);
      free(qd);
    }
  }
  free(K);
  free(V);
  free(keep);
  return 0;
}
