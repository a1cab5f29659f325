/*
 * TEST INFRASTRUCTURE -- fp64 CPU oracle for packed variable-length causal GQA attention.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may build, load or call
 * this file. It shares no code, header, table or helper with the CUDA library and never calls it.
 *
 * What it evaluates is the plain definition of the local attention compute phase of an Ulysses-style
 * sequence-parallel backend (paper Sec. 2.1, paragraph "Sequence Parallelism": after the all-to-all every GPU holds
 * complete sequences for a subset of heads and attends locally; Sec. 2.2 "Sequence Packing": packed segments
 * never attend to one another; Sec. 4.1.2 "SP-backend level": the compute phase exists for forward and for
 * backward). The paper delegates the arithmetic to standard softmax attention kernels and prints no
 * formula of its own, so the oracle is the textbook definition written out, in double precision:
 *
 *   S_ij  = scale * <Q[i,h,:], K[j,g,:]>      for j <= i (causal, diagonal included), g = h / (Hq/Hkv)
 *   LSE_i = log sum_{j<=i} exp(S_ij),   P_ij = exp(S_ij - LSE_i),   O[i,h,:] = sum_j P_ij V[j,g,:]
 *   dP_ij = <dO[i,h,:], V[j,g,:]>,      dS_ij = P_ij * (dP_ij - sum_j' P_ij' dP_ij')
 *   dQ[i,h,:] = scale * sum_{j<=i} dS_ij K[j,g,:]
 *   dK[j,g,:] = scale * sum_{h in group g} sum_{i>=j} dS_ij Q[i,h,:]
 *   dV[j,g,:] =         sum_{h in group g} sum_{i>=j} P_ij dO[i,h,:]
 *
 * i.e. the gradients of the scalar sum(O * dO). No tiling, no online softmax, no fusion: one query row at a
 * time (forward, dQ) and one key column at a time (dK, dV), each owned by exactly one loop iteration, so the
 * result does not depend on the number of threads.
 *
 * Packed layout (the library's interface, restated here independently): segment s of Q/O/dO/dQ is a
 * contiguous [L_s, Hq_s, D] block at element offset D * sum_{t<s} L_t*Hq_t; K/V/dK/dV are [L_s, Hkv_s, D]
 * at D * sum_{t<s} L_t*Hkv_t; LSE is [Hq_s, L_s] at sum_{t<s} L_t*Hq_t.
 *
 * Inputs are either raw bf16 bit patterns (widened exactly to double) or doubles (in_dtype 0 / 1).
 * Outputs are always doubles. Pins for every function live in tests/test_oracle_*.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_BAD 1
#define ORC_NOMEM 2

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static inline double load_elem(const void* p, int64_t idx, int dt) {
  if (dt == 1) return ((const double*)p)[idx];
  uint32_t u = ((uint32_t)((const uint16_t*)p)[idx]) << 16; /* bf16 is the top half of an fp32 */
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

typedef struct {
  int n_seg, D;
  const int32_t *cu, *hq, *hkv;
  int64_t *q_off, *kv_off, *lse_off; /* element offsets per segment (+1 entry: totals) */
} layout_t;

static int layout_init(layout_t* lay, const int32_t* cu, const int32_t* hq, const int32_t* hkv, int n_seg, int D) {
  if (n_seg < 0 || D <= 0 || (n_seg > 0 && (!cu || !hq || !hkv))) return ORC_BAD;
  if (n_seg > 0 && cu[0] != 0) return ORC_BAD;
  lay->n_seg = n_seg;
  lay->D = D;
  lay->cu = cu;
  lay->hq = hq;
  lay->hkv = hkv;
  lay->q_off = (int64_t*)calloc((size_t)n_seg + 1, sizeof(int64_t));
  lay->kv_off = (int64_t*)calloc((size_t)n_seg + 1, sizeof(int64_t));
  lay->lse_off = (int64_t*)calloc((size_t)n_seg + 1, sizeof(int64_t));
  if (!lay->q_off || !lay->kv_off || !lay->lse_off) return ORC_NOMEM;
  for (int s = 0; s < n_seg; ++s) {
    int64_t L = (int64_t)cu[s + 1] - cu[s];
    if (L < 0 || hq[s] <= 0 || hkv[s] <= 0 || hq[s] % hkv[s] != 0) return ORC_BAD;
    lay->q_off[s + 1] = lay->q_off[s] + L * hq[s] * D;
    lay->kv_off[s + 1] = lay->kv_off[s] + L * hkv[s] * D;
    lay->lse_off[s + 1] = lay->lse_off[s] + L * hq[s];
  }
  return ORC_OK;
}
static void layout_free(layout_t* lay) {
  free(lay->q_off);
  free(lay->kv_off);
  free(lay->lse_off);
}

/* Copy head g of segment s of a [L, H, D] block into a dense double [L][D] array. */
static double* gather_head(const void* base, int dt, int64_t seg_off, int64_t L, int H, int g, int D) {
  double* out = (double*)malloc((size_t)(L > 0 ? L : 1) * D * sizeof(double));
  if (!out) return NULL;
  for (int64_t i = 0; i < L; ++i)
    for (int d = 0; d < D; ++d) out[i * D + d] = load_elem(base, seg_off + (i * H + g) * D + d, dt);
  return out;
}
static void gather_row(const void* base, int dt, int64_t seg_off, int64_t i, int H, int h, int D, double* out) {
  for (int d = 0; d < D; ++d) out[d] = load_elem(base, seg_off + (i * H + h) * D + d, dt);
}
static inline double dot(const double* a, const double* b, int D) {
  double acc = 0.0;
  for (int d = 0; d < D; ++d) acc += a[d] * b[d];
  return acc;
}

/*
 * One query row i of one head against keys 0..i of its KV head (dense double K, V of that head).
 * p[0..i] receives the softmax row. Outputs: o[D], *lse; and, when dO_row is given, dq[D] and *rowdot
 * (= sum_j P_ij dP_ij, the softmax-Jacobian correction term).
 */
static void attend_row(const double* q, const double* K, const double* V, int64_t i, int D, double scale, double* p,
                       double* o, double* lse, const double* dO_row, double* dq, double* rowdot) {
  double m = -INFINITY;
  for (int64_t j = 0; j <= i; ++j) {
    p[j] = scale * dot(q, K + j * D, D);
    if (p[j] > m) m = p[j];
  }
  double Z = 0.0;
  for (int64_t j = 0; j <= i; ++j) Z += exp(p[j] - m);
  const double l = m + log(Z);
  for (int64_t j = 0; j <= i; ++j) p[j] = exp(p[j] - l);
  if (o) {
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int64_t j = 0; j <= i; ++j)
      for (int d = 0; d < D; ++d) o[d] += p[j] * V[j * D + d];
  }
  if (lse) *lse = l;
  if (dO_row) {
    double rd = 0.0;
    for (int64_t j = 0; j <= i; ++j) rd += p[j] * dot(dO_row, V + j * D, D);
    if (rowdot) *rowdot = rd;
    if (dq) {
      for (int d = 0; d < D; ++d) dq[d] = 0.0;
      for (int64_t j = 0; j <= i; ++j) {
        const double ds = p[j] * (dot(dO_row, V + j * D, D) - rd);
        for (int d = 0; d < D; ++d) dq[d] += ds * K[j * D + d];
      }
      for (int d = 0; d < D; ++d) dq[d] *= scale;
    }
  }
}

/* ------------------------------------------------------------------------------------------------ forward */
int orc_attn_fwd(const void* q, const void* k, const void* v, int in_dtype, const int32_t* cu, const int32_t* hq,
                 const int32_t* hkv, int n_seg, int D, double scale, double* O, double* LSE) {
  layout_t lay;
  int rc = layout_init(&lay, cu, hq, hkv, n_seg, D);
  if (rc) return rc;
  for (int s = 0; s < n_seg && !rc; ++s) {
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    const int Hq = hq[s], Hkv = hkv[s], G = Hq / Hkv;
    for (int g = 0; g < Hkv && !rc; ++g) {
      double* K = gather_head(k, in_dtype, lay.kv_off[s], L, Hkv, g, D);
      double* V = gather_head(v, in_dtype, lay.kv_off[s], L, Hkv, g, D);
      if (!K || !V) rc = ORC_NOMEM;
      if (!rc) {
#pragma omp parallel
        {
          double* p = (double*)malloc((size_t)(L > 0 ? L : 1) * sizeof(double));
          double* qr = (double*)malloc((size_t)D * sizeof(double));
#pragma omp for schedule(dynamic, 8) collapse(2)
          for (int hh = 0; hh < G; ++hh)
            for (int64_t i = 0; i < L; ++i) {
              const int h = g * G + hh;
              gather_row(q, in_dtype, lay.q_off[s], i, Hq, h, D, qr);
              attend_row(qr, K, V, i, D, scale, p, O + lay.q_off[s] + (i * Hq + h) * D,
                         LSE ? LSE + lay.lse_off[s] + (int64_t)h * L + i : NULL, NULL, NULL, NULL);
            }
          free(p);
          free(qr);
        }
      }
      free(K);
      free(V);
    }
  }
  layout_free(&lay);
  return rc;
}

/* ------------------------------------------------------------------------------------------------ backward
 * Pass A (row-owned): LSE_i, rowdot_i and dQ_i for every active row.  Pass B (column-owned): dK_j, dV_j.
 *
 * rows_seg / rows_idx (n_rows entries, may be NULL): restrict every sum over query rows i to the listed
 * (segment, row) pairs. With NULL all rows take part and the result is the full gradient. With a list the
 * result equals the full gradient whenever dO is zero on every unlisted row (those rows contribute nothing:
 * dP = 0 so dS = 0, and P*dO = 0); dQ is then written for listed rows only (other rows of dQ are set to 0).
 */
int orc_attn_bwd(const void* q, const void* k, const void* v, const void* d_o, int in_dtype, const int32_t* cu,
                 const int32_t* hq, const int32_t* hkv, int n_seg, int D, double scale, const int32_t* rows_seg,
                 const int32_t* rows_idx, int64_t n_rows, double* dQ, double* dK, double* dV) {
  layout_t lay;
  int rc = layout_init(&lay, cu, hq, hkv, n_seg, D);
  if (rc) return rc;
  if (dQ) memset(dQ, 0, (size_t)lay.q_off[n_seg] * sizeof(double));
  memset(dK, 0, (size_t)lay.kv_off[n_seg] * sizeof(double));
  memset(dV, 0, (size_t)lay.kv_off[n_seg] * sizeof(double));
  for (int s = 0; s < n_seg && !rc; ++s) {
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    const int Hq = hq[s], Hkv = hkv[s], G = Hq / Hkv;
    if (L == 0) continue;
    /* active rows of this segment, ascending */
    int64_t n_act = 0;
    int64_t* act = (int64_t*)malloc((size_t)L * sizeof(int64_t));
    if (!act) {
      rc = ORC_NOMEM;
      break;
    }
    if (!rows_seg) {
      for (int64_t i = 0; i < L; ++i) act[n_act++] = i;
    } else {
      char* mark = (char*)calloc((size_t)L, 1);
      if (!mark) {
        free(act);
        rc = ORC_NOMEM;
        break;
      }
      for (int64_t r = 0; r < n_rows; ++r)
        if (rows_seg[r] == s && rows_idx[r] >= 0 && rows_idx[r] < L) mark[rows_idx[r]] = 1;
      for (int64_t i = 0; i < L; ++i)
        if (mark[i]) act[n_act++] = i;
      free(mark);
    }
    for (int g = 0; g < Hkv && !rc; ++g) {
      double* K = gather_head(k, in_dtype, lay.kv_off[s], L, Hkv, g, D);
      double* V = gather_head(v, in_dtype, lay.kv_off[s], L, Hkv, g, D);
      double* lse = (double*)malloc((size_t)G * (n_act > 0 ? n_act : 1) * sizeof(double));
      double* rdot = (double*)malloc((size_t)G * (n_act > 0 ? n_act : 1) * sizeof(double));
      double* Qa = (double*)malloc((size_t)G * (n_act > 0 ? n_act : 1) * D * sizeof(double));  /* active Q rows */
      double* dOa = (double*)malloc((size_t)G * (n_act > 0 ? n_act : 1) * D * sizeof(double)); /* active dO rows */
      if (!K || !V || !lse || !rdot || !Qa || !dOa) rc = ORC_NOMEM;
      if (!rc) {
        /* pass A */
#pragma omp parallel
        {
          double* p = (double*)malloc((size_t)L * sizeof(double));
          double* dq = (double*)malloc((size_t)D * sizeof(double));
#pragma omp for schedule(dynamic, 4) collapse(2)
          for (int hh = 0; hh < G; ++hh)
            for (int64_t a = 0; a < n_act; ++a) {
              const int h = g * G + hh;
              const int64_t i = act[a];
              double* qr = Qa + ((int64_t)hh * n_act + a) * D;
              double* dor = dOa + ((int64_t)hh * n_act + a) * D;
              gather_row(q, in_dtype, lay.q_off[s], i, Hq, h, D, qr);
              gather_row(d_o, in_dtype, lay.q_off[s], i, Hq, h, D, dor);
              attend_row(qr, K, V, i, D, scale, p, NULL, &lse[(int64_t)hh * n_act + a], dor, dQ ? dq : NULL,
                         &rdot[(int64_t)hh * n_act + a]);
              if (dQ) memcpy(dQ + lay.q_off[s] + (i * Hq + h) * D, dq, (size_t)D * sizeof(double));
            }
          free(p);
          free(dq);
        }
        /* pass B: column j sums over active rows i >= j of every head in the group */
#pragma omp parallel for schedule(dynamic, 16)
        for (int64_t j = 0; j < L; ++j) {
          double* dk = dK + lay.kv_off[s] + (j * Hkv + g) * D;
          double* dv = dV + lay.kv_off[s] + (j * Hkv + g) * D;
          const double* kj = K + j * D;
          const double* vj = V + j * D;
          for (int hh = 0; hh < G; ++hh)
            for (int64_t a = 0; a < n_act; ++a) {
              const int64_t i = act[a];
              if (i < j) continue;
              const double* qr = Qa + ((int64_t)hh * n_act + a) * D;
              const double* dor = dOa + ((int64_t)hh * n_act + a) * D;
              const double pij = exp(scale * dot(qr, kj, D) - lse[(int64_t)hh * n_act + a]);
              const double ds = pij * (dot(dor, vj, D) - rdot[(int64_t)hh * n_act + a]);
              for (int d = 0; d < D; ++d) {
                dk[d] += ds * qr[d];
                dv[d] += pij * dor[d];
              }
            }
          for (int d = 0; d < D; ++d) dk[d] *= scale;
        }
      }
      free(K);
      free(V);
      free(lse);
      free(rdot);
      free(Qa);
      free(dOa);
    }
    free(act);
  }
  layout_free(&lay);
  return rc;
}

/* ------------------------------------------------------------------------------------------------ samples
 * Query-row samples: O, LSE and (when d_o is given) dQ for n listed (segment, q head, row) triples.
 * Outputs are dense [n][D], [n], [n][D]. Each row costs O(row * D).
 */
int orc_attn_rows(const void* q, const void* k, const void* v, const void* d_o, int in_dtype, const int32_t* cu,
                  const int32_t* hq, const int32_t* hkv, int n_seg, int D, double scale, int64_t n,
                  const int32_t* s_seg, const int32_t* s_head, const int32_t* s_row, double* O, double* LSE,
                  double* dQ) {
  layout_t lay;
  int rc = layout_init(&lay, cu, hq, hkv, n_seg, D);
  if (rc) return rc;
  for (int64_t t = 0; t < n; ++t) {
    const int s = s_seg[t];
    if (s < 0 || s >= n_seg) { rc = ORC_BAD; break; }
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    if (s_head[t] < 0 || s_head[t] >= hq[s] || s_row[t] < 0 || s_row[t] >= L) { rc = ORC_BAD; break; }
  }
  /* group by (segment, kv head) so each K/V head is gathered once */
  for (int s = 0; s < n_seg && !rc; ++s) {
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    const int Hq = hq[s], Hkv = hkv[s], G = Hq / Hkv;
    for (int g = 0; g < Hkv && !rc; ++g) {
      int64_t cnt = 0, need = 0;
      for (int64_t t = 0; t < n; ++t)
        if (s_seg[t] == s && s_head[t] / G == g) {
          ++cnt;
          if (s_row[t] + 1 > need) need = s_row[t] + 1;
        }
      if (!cnt) continue;
      double* K = gather_head(k, in_dtype, lay.kv_off[s], need, Hkv, g, D);
      double* V = gather_head(v, in_dtype, lay.kv_off[s], need, Hkv, g, D);
      if (!K || !V) rc = ORC_NOMEM;
      if (!rc) {
#pragma omp parallel
        {
          double* p = (double*)malloc((size_t)need * sizeof(double));
          double* qr = (double*)malloc((size_t)D * sizeof(double));
          double* dor = (double*)malloc((size_t)D * sizeof(double));
#pragma omp for schedule(dynamic, 1)
          for (int64_t t = 0; t < n; ++t) {
            if (s_seg[t] != s || s_head[t] / G != g) continue;
            const int h = s_head[t];
            const int64_t i = s_row[t];
            gather_row(q, in_dtype, lay.q_off[s], i, Hq, h, D, qr);
            if (d_o) gather_row(d_o, in_dtype, lay.q_off[s], i, Hq, h, D, dor);
            attend_row(qr, K, V, i, D, scale, p, O + t * D, LSE + t, d_o ? dor : NULL, (d_o && dQ) ? dQ + t * D : NULL,
                       NULL);
          }
          free(p);
          free(qr);
          free(dor);
        }
      }
      free(K);
      free(V);
    }
  }
  layout_free(&lay);
  return rc;
}

/*
 * Key-column samples: dK and dV (dense [n][D] each) for n listed (segment, kv head, column) triples, under
 * the full dO. Column j needs LSE_i and rowdot_i of every row i >= j of the G heads in its group, each
 * O(i * D), so this is affordable for columns near the end of a segment.
 */
int orc_attn_cols(const void* q, const void* k, const void* v, const void* d_o, int in_dtype, const int32_t* cu,
                  const int32_t* hq, const int32_t* hkv, int n_seg, int D, double scale, int64_t n,
                  const int32_t* s_seg, const int32_t* s_kvhead, const int32_t* s_col, double* dK, double* dV) {
  layout_t lay;
  int rc = layout_init(&lay, cu, hq, hkv, n_seg, D);
  if (rc) return rc;
  for (int64_t t = 0; t < n; ++t) {
    const int s = s_seg[t];
    if (s < 0 || s >= n_seg) { rc = ORC_BAD; break; }
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    if (s_kvhead[t] < 0 || s_kvhead[t] >= hkv[s] || s_col[t] < 0 || s_col[t] >= L) { rc = ORC_BAD; break; }
  }
  for (int s = 0; s < n_seg && !rc; ++s) {
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    const int Hq = hq[s], Hkv = hkv[s], G = Hq / Hkv;
    for (int g = 0; g < Hkv && !rc; ++g) {
      int64_t cnt = 0, jmin = L;
      for (int64_t t = 0; t < n; ++t)
        if (s_seg[t] == s && s_kvhead[t] == g) {
          ++cnt;
          if (s_col[t] < jmin) jmin = s_col[t];
        }
      if (!cnt) continue;
      const int64_t nr = L - jmin; /* rows jmin..L-1 */
      double* K = gather_head(k, in_dtype, lay.kv_off[s], L, Hkv, g, D);
      double* V = gather_head(v, in_dtype, lay.kv_off[s], L, Hkv, g, D);
      double* lse = (double*)malloc((size_t)G * nr * sizeof(double));
      double* rdot = (double*)malloc((size_t)G * nr * sizeof(double));
      double* Qa = (double*)malloc((size_t)G * nr * D * sizeof(double));
      double* dOa = (double*)malloc((size_t)G * nr * D * sizeof(double));
      if (!K || !V || !lse || !rdot || !Qa || !dOa) rc = ORC_NOMEM;
      if (!rc) {
#pragma omp parallel
        {
          double* p = (double*)malloc((size_t)L * sizeof(double));
#pragma omp for schedule(dynamic, 1) collapse(2)
          for (int hh = 0; hh < G; ++hh)
            for (int64_t a = 0; a < nr; ++a) {
              const int h = g * G + hh;
              const int64_t i = jmin + a;
              double* qr = Qa + ((int64_t)hh * nr + a) * D;
              double* dor = dOa + ((int64_t)hh * nr + a) * D;
              gather_row(q, in_dtype, lay.q_off[s], i, Hq, h, D, qr);
              gather_row(d_o, in_dtype, lay.q_off[s], i, Hq, h, D, dor);
              attend_row(qr, K, V, i, D, scale, p, NULL, &lse[(int64_t)hh * nr + a], dor, NULL,
                         &rdot[(int64_t)hh * nr + a]);
            }
          free(p);
        }
#pragma omp parallel for schedule(dynamic, 1)
        for (int64_t t = 0; t < n; ++t) {
          if (s_seg[t] != s || s_kvhead[t] != g) continue;
          const int64_t j = s_col[t];
          double* dk = dK + t * D;
          double* dv = dV + t * D;
          for (int d = 0; d < D; ++d) dk[d] = dv[d] = 0.0;
          for (int hh = 0; hh < G; ++hh)
            for (int64_t i = j; i < L; ++i) {
              const int64_t a = i - jmin;
              const double* qr = Qa + ((int64_t)hh * nr + a) * D;
              const double* dor = dOa + ((int64_t)hh * nr + a) * D;
              const double pij = exp(scale * dot(qr, K + j * D, D) - lse[(int64_t)hh * nr + a]);
              const double ds = pij * (dot(dor, V + j * D, D) - rdot[(int64_t)hh * nr + a]);
              for (int d = 0; d < D; ++d) {
                dk[d] += ds * qr[d];
                dv[d] += pij * dor[d];
              }
            }
          for (int d = 0; d < D; ++d) dk[d] *= scale;
        }
      }
      free(K);
      free(V);
      free(lse);
      free(rdot);
      free(Qa);
      free(dOa);
    }
  }
  layout_free(&lay);
  return rc;
}

/* ------------------------------------------------------------------------------------------------ tile plan
 * Work list of the in-GPU schedule (the paper balances load across GPUs and issues a GPU's nodes one after
 * the other, Sec. 4.2.1; the in-GPU list is this build's reading). Tile sizes bm (query rows), bn (key rows).
 *   pass 0 (forward):  one item per (segment s, q head h, q tile m);  cost = ceil(min(L, (m+1)*bm) / bn),
 *                      the number of key tiles the q tile visits.
 *   pass 1 (backward): one item per (segment s, kv head g, key tile n); cost = G * (Mt - floor(n*bn / bm)),
 *                      the number of (q head, q tile) visits of the key tile.
 * Order: cost descending, then segment, tile, head ascending -- a total order, so the list is unique.
 *   pass 2 (backward, as executed): the items of pass 1 in the order the backward pass walks them: the groups
 *                      (segment, kv head) by segment length descending, then segment ascending, then kv head
 *                      ascending; inside a group the key tiles ascending. Also a total order.
 * Each item is four int32 {seg, head, tile, cost}. Returns the item count in *n_items; writes at most cap.
 */
typedef struct { int32_t seg, head, tile, cost; } item_t;

/* order of pass 2; the segment lengths are reached through this file-scope pointer while qsort runs */
static const int32_t* g_cmp_cu = 0;
static int item_cmp_exec(const void* a, const void* b) {
  const item_t* x = (const item_t*)a;
  const item_t* y = (const item_t*)b;
  const int64_t lx = (int64_t)g_cmp_cu[x->seg + 1] - g_cmp_cu[x->seg], ly = (int64_t)g_cmp_cu[y->seg + 1] - g_cmp_cu[y->seg];
  if (lx != ly) return lx > ly ? -1 : 1;
  if (x->seg != y->seg) return x->seg < y->seg ? -1 : 1;
  if (x->head != y->head) return x->head < y->head ? -1 : 1;
  if (x->tile != y->tile) return x->tile < y->tile ? -1 : 1;
  return 0;
}

static int item_cmp(const void* a, const void* b) {
  const item_t* x = (const item_t*)a;
  const item_t* y = (const item_t*)b;
  if (x->cost != y->cost) return x->cost > y->cost ? -1 : 1;
  if (x->seg != y->seg) return x->seg < y->seg ? -1 : 1;
  if (x->tile != y->tile) return x->tile < y->tile ? -1 : 1;
  if (x->head != y->head) return x->head < y->head ? -1 : 1;
  return 0;
}

int orc_plan_tiles(const int32_t* cu, const int32_t* hq, const int32_t* hkv, int n_seg, int bm, int bn, int pass,
                   int32_t* out, int64_t cap, int64_t* n_items) {
  if (n_seg < 0 || bm <= 0 || bn <= 0 || pass < 0 || pass > 2 || !n_items) return ORC_BAD;
  int64_t total = 0;
  for (int s = 0; s < n_seg; ++s) {
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    if (L < 0 || hq[s] <= 0 || hkv[s] <= 0 || hq[s] % hkv[s]) return ORC_BAD;
    const int64_t Mt = (L + bm - 1) / bm, Nt = (L + bn - 1) / bn;
    total += pass == 0 ? Mt * hq[s] : Nt * hkv[s];
  }
  *n_items = total;
  if (!out || cap < total) return ORC_OK; /* size query */
  item_t* it = (item_t*)out;
  int64_t w = 0;
  for (int s = 0; s < n_seg; ++s) {
    const int64_t L = (int64_t)cu[s + 1] - cu[s];
    const int64_t Mt = (L + bm - 1) / bm, Nt = (L + bn - 1) / bn;
    const int G = hq[s] / hkv[s];
    if (pass == 0) {
      for (int h = 0; h < hq[s]; ++h)
        for (int64_t m = 0; m < Mt; ++m) {
          int64_t hi = (m + 1) * bm < L ? (m + 1) * bm : L;
          it[w++] = (item_t){s, h, (int32_t)m, (int32_t)((hi + bn - 1) / bn)};
        }
    } else {
      for (int g = 0; g < hkv[s]; ++g)
        for (int64_t n = 0; n < Nt; ++n) it[w++] = (item_t){s, g, (int32_t)n, (int32_t)(G * (Mt - (n * bn) / bm))};
    }
  }
  if (pass == 2) {
    g_cmp_cu = cu; /* not re-entrant: the Python front end calls this from one thread */
    qsort(it, (size_t)total, sizeof(item_t), item_cmp_exec);
  } else {
    qsort(it, (size_t)total, sizeof(item_t), item_cmp);
  }
  return ORC_OK;
}
