/*
 * vosti_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what batch-invariant paged attention
 * computes.  It exists to check the CUDA library; the product never calls it.
 * Only the tests, the smoke check and the benchmark's cpu_baseline / reference
 * arm may load this file.  It shares no code, header or table with the CUDA
 * path.
 *
 * What is computed (the exact result the tiled kernel approximates):
 *
 *   - Causal GQA attention for one query head and its KV head (App. A,
 *     "Properties and Logical Inputs"): query row i of a request whose rows
 *     start at logical position `start` stands at position p = start + i
 *     (Sec. "The causal contract": p = k_len - q_len + i; here start may be
 *     smaller than k_len - q_len, later keys are masked anyway).
 *   - The logical cache read through a page table (App. A):
 *         K[j,:] = K_phys[ pi(floor(j/P)), j mod P, : ]      same for V.
 *   - The mask of App. A, "A Simplified Tile IR":  key j is visible to the
 *     row at p iff  j <= p  and  j < n.
 *   - The result is softmax(scale * q.K^T) V over the visible keys, written
 *     as the plain two-pass definition (maximum, exponentials, sum, divide),
 *     with the z > 0 guard of the paper's output equation
 *         O = U * select(z > 0, 1/z, 0).
 *     No tiling, no online softmax, no splitting: those are properties of
 *     the kernel, not of the result.
 *   - Query head h reads KV head floor(h / G), G = n_q_heads / n_kv_heads.
 *   - Sliding window (App. A, last paragraph: "adds j > p - w for shared window
 *     size w > 0"): with window w > 0 key j is visible iff  p - w < j <= p;
 *     w = 0 means no window.
 *   - The auxiliary log-sum-exp the paper's kernel emits (App. A, after the
 *     output equation): lse = log sum_j exp(scale * q.K_j) over visible keys,
 *     natural logarithm, computed as  max + log(sum exp(s - max)).
 *
 * Inputs are bf16 bit patterns (uint16) widened exactly to double; every
 * sum is a plain left-to-right double sum.
 *
 * Pool layout (part of the library boundary, restated here independently):
 *   pool[page][kv_head][0=K,1=V][slot 0..P-1][e 0..d-1]   bf16
 *
 * Pinned by tests/test_oracle_pins.py (closed forms, brute force, library
 * routine, invariances).  Parity with the paper's own implementation:
 * unpinned -- the paper prints no code output or worked numeric example.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* A view of one request's logical K/V sequence: dense [n][Hkv][d] arrays or a
 * page pool read through one block-table row. */
typedef struct {
  int paged;
  const uint16_t* k_dense; /* dense: [n][Hkv][d] */
  const uint16_t* v_dense;
  const uint16_t* pool; /* paged */
  const int32_t* bt;    /* paged: block-table row of this request */
  int P, Hkv, d;
} kv_view;

/* Row j of K (which=0) or V (which=1) for KV head kappa. */
static const uint16_t* kv_row(const kv_view* w, int64_t j, int kappa, int which) {
  if (!w->paged) {
    const uint16_t* base = which ? w->v_dense : w->k_dense;
    return base + ((size_t)j * w->Hkv + kappa) * (size_t)w->d;
  }
  int64_t page = w->bt[j / w->P];
  int64_t slot = j % w->P;
  size_t chunk = ((size_t)page * w->Hkv + kappa) * 2 + (size_t)which;
  return w->pool + (chunk * w->P + (size_t)slot) * (size_t)w->d;
}

/* One output row: attention of query vector q (d bf16 values) at position p
 * over keys 0..p of KV head kappa.  out receives d doubles.
 * Returns 0, or -1 if memory ran out. */
static int attend_row(const uint16_t* q, const kv_view* w, int64_t p, int kappa, double scale,
                      int64_t window, double* out, double* lse) {
  const int d = w->d;
  const int64_t j0 = (window > 0 && p - window + 1 > 0) ? p - window + 1 : 0; /* first visible key */
  const int64_t nvis = p + 1 - j0;                                             /* keys j0..p are visible */
  double* s = (double*)malloc(sizeof(double) * (size_t)(nvis > 0 ? nvis : 1));
  if (!s) return -1;
  double qd[1024];
  for (int e = 0; e < d; ++e) qd[e] = bf16_to_f64(q[e]);

  /* scores and their maximum */
  double mx = -INFINITY;
  for (int64_t j = 0; j < nvis; ++j) {
    const uint16_t* kr = kv_row(w, j0 + j, kappa, 0);
    double acc = 0.0;
    for (int e = 0; e < d; ++e) acc += qd[e] * bf16_to_f64(kr[e]);
    s[j] = scale * acc;
    if (s[j] > mx) mx = s[j];
  }
  /* weights and normaliser */
  double z = 0.0;
  for (int64_t j = 0; j < nvis; ++j) {
    s[j] = exp(s[j] - mx);
    z += s[j];
  }
  /* weighted values */
  for (int e = 0; e < d; ++e) out[e] = 0.0;
  for (int64_t j = 0; j < nvis; ++j) {
    const uint16_t* vr = kv_row(w, j0 + j, kappa, 1);
    for (int e = 0; e < d; ++e) out[e] += s[j] * bf16_to_f64(vr[e]);
  }
  const double inv = (z > 0.0) ? 1.0 / z : 0.0;
  for (int e = 0; e < d; ++e) out[e] *= inv;
  if (lse) *lse = mx + log(z);
  free(s);
  return 0;
}

int vosti_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Dense front-end, one request.
 *   q   [s][Hq][d] bf16     rows at positions start .. start+s-1
 *   k,v [n][Hkv][d] bf16    the logical sequence, n >= start + s
 *   out [s][Hq][d] double;  lse [s][Hq] double or NULL;  window: 0 = none
 * Returns 0 on success, 1 on bad arguments, 2 if memory ran out. */
int vosti_oracle_attention_dense(const uint16_t* q, const uint16_t* k, const uint16_t* v, int s,
                                 int n, int start, int Hq, int Hkv, int d, double scale,
                                 int64_t window, double* out, double* lse /* [s][Hq] or NULL */) {
  if (s < 0 || n < 0 || start < 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || d > 1024) return 1;
  if (Hq % Hkv != 0 || (int64_t)start + s > n) return 1;
  const int G = Hq / Hkv;
  kv_view w = {0, k, v, NULL, NULL, 0, Hkv, d};
  int fail = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int i = 0; i < s; ++i)
    for (int h = 0; h < Hq; ++h) {
      const size_t row = (size_t)i * Hq + h;
      if (attend_row(q + row * d, &w, (int64_t)start + i, h / G, scale, window, out + row * d,
                     lse ? lse + row : NULL))
        fail = 1;
    }
  return fail ? 2 : 0;
}

/* Paged front-end, a batch.
 *   q            [T][Hq][d] bf16, packed rows: request-major, token-minor
 *   pool         page pool in the boundary's layout
 *   q_lens, start_pos, seq_lens   [B]
 *   block_tables [B][bt_stride]   only entries < ceil(seq_len/P) are read
 *   sel          NULL: compute every row, out is [T][Hq][d];
 *                else n_sel triples (request, token i, head h): out is [n_sel][d]
 *   lse          NULL, or [T][Hq] (resp. [n_sel]) doubles;  window: 0 = none
 * Returns 0 on success, 1 on bad arguments, 2 if memory ran out. */
int vosti_oracle_paged_attention(const uint16_t* q, const uint16_t* pool, const int32_t* q_lens,
                                 const int32_t* start_pos, const int32_t* seq_lens,
                                 const int32_t* block_tables, int bt_stride, int B, int Hq, int Hkv,
                                 int d, int P, int64_t num_pages, double scale, int64_t window,
                                 const int32_t* sel, int64_t n_sel, double* out, double* lse) {
  if (B < 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || d > 1024 || P <= 0 || Hq % Hkv != 0) return 1;
  const int G = Hq / Hkv;
  int64_t* row0 = (int64_t*)malloc(sizeof(int64_t) * (size_t)(B + 1));
  if (!row0) return 2;
  row0[0] = 0;
  for (int r = 0; r < B; ++r) {
    if (q_lens[r] < 0 || start_pos[r] < 0 ||
        (int64_t)start_pos[r] + q_lens[r] > (int64_t)seq_lens[r] ||
        ((int64_t)seq_lens[r] + P - 1) / P > bt_stride) {
      free(row0);
      return 1;
    }
    if (q_lens[r] > 0)
      for (int64_t b = 0; b < ((int64_t)seq_lens[r] + P - 1) / P; ++b) {
        int32_t pg = block_tables[(size_t)r * bt_stride + b];
        if (pg < 0 || pg >= num_pages) {
          free(row0);
          return 1;
        }
      }
    row0[r + 1] = row0[r] + q_lens[r];
  }
  int fail = 0;
  if (sel == NULL) {
    const int64_t T = row0[B];
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t job = 0; job < T * Hq; ++job) {
      const int64_t t = job / Hq;
      const int h = (int)(job % Hq);
      int r = 0;
      while (row0[r + 1] <= t) ++r;
      const int64_t i = t - row0[r];
      kv_view w = {1, NULL, NULL, pool, block_tables + (size_t)r * bt_stride, P, Hkv, d};
      const size_t row = (size_t)t * Hq + h;
      if (attend_row(q + row * d, &w, (int64_t)start_pos[r] + i, h / G, scale, window, out + row * d,
                     lse ? lse + row : NULL))
        fail = 1;
    }
  } else {
    for (int64_t x = 0; x < n_sel; ++x) {
      int r = sel[3 * x], i = sel[3 * x + 1], h = sel[3 * x + 2];
      if (r < 0 || r >= B || i < 0 || i >= q_lens[r] || h < 0 || h >= Hq) {
        free(row0);
        return 1;
      }
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t x = 0; x < n_sel; ++x) {
      const int r = sel[3 * x], i = sel[3 * x + 1], h = sel[3 * x + 2];
      kv_view w = {1, NULL, NULL, pool, block_tables + (size_t)r * bt_stride, P, Hkv, d};
      const size_t row = (size_t)(row0[r] + i) * Hq + h;
      if (attend_row(q + row * d, &w, (int64_t)start_pos[r] + i, h / G, scale, window,
                     out + (size_t)x * d, lse ? lse + x : NULL))
        fail = 1;
    }
  }
  free(row0);
  return fail ? 2 : 0;
}

/* KV write into page slots (Sec. "Separate cache reuse from generation": new
 * K/V go to the request's own suffix slots).  Token i of request r stands at
 * p = start_pos[r] + i and lands in page block_tables[r][p / P], slot p % P.
 *   k_new, v_new [T][Hkv][d] bf16 packed like q.
 * Returns 0 on success, 1 on bad arguments. */
int vosti_oracle_kv_append(uint16_t* pool, const uint16_t* k_new, const uint16_t* v_new,
                           const int32_t* q_lens, const int32_t* start_pos,
                           const int32_t* block_tables, int bt_stride, int B, int Hkv, int d, int P,
                           int64_t num_pages) {
  int64_t t = 0;
  for (int r = 0; r < B; ++r) {
    if (q_lens[r] < 0 || start_pos[r] < 0) return 1;
    for (int i = 0; i < q_lens[r]; ++i, ++t) {
      const int64_t p = (int64_t)start_pos[r] + i;
      if (p / P >= bt_stride) return 1;
      const int64_t page = block_tables[(size_t)r * bt_stride + p / P];
      if (page < 0 || page >= num_pages) return 1;
      const int64_t slot = p % P;
      for (int kh = 0; kh < Hkv; ++kh) {
        const size_t chunk = ((size_t)page * Hkv + kh) * 2;
        uint16_t* kd = pool + ((chunk + 0) * P + slot) * (size_t)d;
        uint16_t* vd = pool + ((chunk + 1) * P + slot) * (size_t)d;
        memcpy(kd, k_new + ((size_t)t * Hkv + kh) * d, sizeof(uint16_t) * (size_t)d);
        memcpy(vd, v_new + ((size_t)t * Hkv + kh) * d, sizeof(uint16_t) * (size_t)d);
      }
    }
  }
  return 0;
}
