/*
 * MoGA routed group-attention forward: reference oracle (TEST INFRASTRUCTURE ONLY).
 *
 * A plain, slow, fp64 CPU statement of what the path computes, written from the
 * paper's equations.  It shares no code with the CUDA library and is imported
 * only by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Inputs are float arrays holding exactly the values the GPU sees (bf16 or fp32,
 * widened without rounding); every sum, exponential and division is in double.
 *
 * Steps, in the paper's order (Sec. 3.2 "Mixture-of-Groups Attention"):
 *   route : r = x W_r (+ bias)                          Eq. 2
 *           p(i|x) = softmax(r)_i                       Eq. 3
 *           g(x) = argmax_i p(i|x)  (top-k: k largest)  Eq. 4
 *   sort  : the "permute" of Alg. 1 line 2: tokens listed group by group,
 *           ascending token index inside a group; cumulative group lengths.
 *   attn  : SA(q, K_g, V_g) = softmax(q K_g^T * scale) V_g   Eq. 1 inside group g
 *   out   : MoGA(x) = sum_j gate_j * SA(q, K_{g_j}, V_{g_j})  Eq. 5 (k = 1 in the paper)
 *
 * Readings where the paper is silent: ties go to the lower group index; the gate
 * is either the softmax over all M logits (Eq. 3-5) or over the k selected ones
 * (gate_mode 1); an empty group does no work; rows are independent.
 *
 * Pinned by tests (not by itself): M = 1 equals textbook full attention computed
 * with library matmul/softmax; pure-Python brute force on tiny inputs; closed
 * forms (equal V rows, zero Q); permutation and independence invariants.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_GATE_SOFTMAX_ALL 0
#define ORACLE_GATE_SOFTMAX_TOPK 1

int moga_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Eq. 2-4 for one token: logits r[M], the k selected groups, their gates. */
static void route_token(int C, int M, int k, int gate_mode, const float* x, const float* Wr,
                        const float* bias, double* r, int32_t* sel, double* gate) {
  for (int i = 0; i < M; ++i) {
    double acc = 0.0;
    for (int c = 0; c < C; ++c) acc += (double)x[c] * (double)Wr[(size_t)c * M + i];
    if (bias) acc += (double)bias[i];
    r[i] = acc;
  }
  /* k largest logits, descending; a tie goes to the lower index. */
  for (int j = 0; j < k; ++j) {
    int best = -1;
    for (int i = 0; i < M; ++i) {
      int taken = 0;
      for (int t = 0; t < j; ++t) taken |= (sel[t] == i);
      if (taken) continue;
      if (best < 0 || r[i] > r[best]) best = i;
    }
    sel[j] = best;
  }
  /* softmax gate, max-subtracted; r[sel[0]] is the global maximum. */
  double mx = r[sel[0]];
  double Z = 0.0;
  if (gate_mode == ORACLE_GATE_SOFTMAX_ALL) {
    for (int i = 0; i < M; ++i) Z += exp(r[i] - mx);
  } else {
    for (int j = 0; j < k; ++j) Z += exp(r[sel[j]] - mx);
  }
  for (int j = 0; j < k; ++j) gate[j] = exp(r[sel[j]] - mx) / Z;
}

int moga_oracle_route(int B, int N, int C, int M, int k, int gate_mode, const float* X,
                      const float* Wr, const float* bias, int32_t* gid, double* gate,
                      double* logits) {
  if (B < 1 || N < 0 || C < 1 || M < 1 || k < 1 || k > M) return 1;
  long long total = (long long)B * N;
#pragma omp parallel
  {
    double* r = (double*)malloc(sizeof(double) * (size_t)M);
#pragma omp for schedule(static)
    for (long long t = 0; t < total; ++t) {
      route_token(C, M, k, gate_mode, X + (size_t)t * C, Wr, bias, r, gid + (size_t)t * k,
                  gate + (size_t)t * k);
      if (logits) memcpy(logits + (size_t)t * M, r, sizeof(double) * (size_t)M);
    }
    free(r);
  }
  return 0;
}

/* Alg. 1 line 2 (index part): group lists in ascending token order, prefix sums. */
int moga_oracle_sort(int B, int N, int M, int k, const int32_t* gid, int32_t* offsets,
                     int32_t* perm, int32_t* inv) {
  if (B < 1 || N < 0 || M < 1 || k < 1) return 1;
  size_t T = (size_t)N * k;
  for (int b = 0; b < B; ++b) {
    const int32_t* g = gid + (size_t)b * T;
    int32_t* off = offsets + (size_t)b * (M + 1);
    int32_t* pm = perm + (size_t)b * T;
    int32_t* iv = inv + (size_t)b * T;
    int32_t pos = 0;
    for (int grp = 0; grp < M; ++grp) {
      off[grp] = pos;
      for (int n = 0; n < N; ++n)
        for (int j = 0; j < k; ++j)
          if (g[(size_t)n * k + j] == grp) {
            pm[pos] = n;
            iv[(size_t)n * k + j] = pos;
            ++pos;
          }
    }
    off[M] = pos;
    if ((size_t)pos != T) return 2; /* a group id was outside [0, M) */
  }
  return 0;
}

/* Eq. 1 inside one group, then Eq. 5's gate-weighted sum, for one (b, h, n). */
static void attn_row(int H, int N, int D, int M, int k, double scale, const float* Q,
                     const float* K, const float* V, const int32_t* gid, const double* gate,
                     const int32_t* offsets, const int32_t* perm, int b, int h, int n, double* out,
                     double* a /* scratch, >= max group size */) {
  size_t T = (size_t)N * k;
  const float* Qh = Q + ((size_t)b * H + h) * (size_t)N * D;
  const float* Kh = K + ((size_t)b * H + h) * (size_t)N * D;
  const float* Vh = V + ((size_t)b * H + h) * (size_t)N * D;
  const float* q = Qh + (size_t)n * D;
  for (int d = 0; d < D; ++d) out[d] = 0.0;
  for (int j = 0; j < k; ++j) {
    int g = gid[(size_t)b * T + (size_t)n * k + j];
    int lo = offsets[(size_t)b * (M + 1) + g], hi = offsets[(size_t)b * (M + 1) + g + 1];
    const int32_t* members = perm + (size_t)b * T;
    double mx = -INFINITY;
    for (int p = lo; p < hi; ++p) {
      const float* kr = Kh + (size_t)members[p] * D;
      double s = 0.0;
      for (int d = 0; d < D; ++d) s += (double)q[d] * (double)kr[d];
      a[p - lo] = s * scale;
      if (a[p - lo] > mx) mx = a[p - lo];
    }
    double Z = 0.0;
    for (int p = lo; p < hi; ++p) {
      a[p - lo] = exp(a[p - lo] - mx);
      Z += a[p - lo];
    }
    double gt = gate[(size_t)b * T + (size_t)n * k + j];
    for (int p = lo; p < hi; ++p) {
      const float* vr = Vh + (size_t)members[p] * D;
      double w = gt * (a[p - lo] / Z);
      for (int d = 0; d < D; ++d) out[d] += w * (double)vr[d];
    }
  }
}

/* rows: nrows triples (b, h, n); out: [nrows, D] doubles. */
int moga_oracle_attn_rows(int B, int H, int N, int D, int M, int k, double scale, const float* Q,
                          const float* K, const float* V, const int32_t* gid, const double* gate,
                          const int32_t* offsets, const int32_t* perm, long long nrows,
                          const int32_t* rows, double* out) {
  if (B < 1 || H < 1 || N < 0 || D < 1 || M < 1 || k < 1) return 1;
  size_t T = (size_t)N * k;
  int bad = 0;
#pragma omp parallel
  {
    double* a = (double*)malloc(sizeof(double) * (T ? T : 1));
#pragma omp for schedule(dynamic, 16)
    for (long long r = 0; r < nrows; ++r) {
      int b = rows[r * 3 + 0], h = rows[r * 3 + 1], n = rows[r * 3 + 2];
      if (b < 0 || b >= B || h < 0 || h >= H || n < 0 || n >= N) {
        bad = 1;
        continue;
      }
      attn_row(H, N, D, M, k, scale, Q, K, V, gid, gate, offsets, perm, b, h, n,
               out + (size_t)r * D, a);
    }
    free(a);
  }
  return bad ? 3 : 0;
}

/* The whole forward.  O is [B,H,N,D] doubles; the index outputs may each be NULL. */
int moga_oracle_forward(int B, int H, int N, int C, int D, int M, int k, int gate_mode,
                        double scale, const float* X, const float* Wr, const float* bias,
                        const float* Q, const float* K, const float* V, double* O,
                        int32_t* gid_out, double* gate_out, int32_t* offsets_out,
                        int32_t* perm_out, int32_t* inv_out) {
  size_t T = (size_t)N * k;
  int32_t* gid = (int32_t*)malloc(sizeof(int32_t) * (size_t)B * (T ? T : 1));
  double* gate = (double*)malloc(sizeof(double) * (size_t)B * (T ? T : 1));
  int32_t* offsets = (int32_t*)malloc(sizeof(int32_t) * (size_t)B * (M + 1));
  int32_t* perm = (int32_t*)malloc(sizeof(int32_t) * (size_t)B * (T ? T : 1));
  int32_t* inv = (int32_t*)malloc(sizeof(int32_t) * (size_t)B * (T ? T : 1));
  int rc = moga_oracle_route(B, N, C, M, k, gate_mode, X, Wr, bias, gid, gate, NULL);
  if (!rc) rc = moga_oracle_sort(B, N, M, k, gid, offsets, perm, inv);
  if (!rc) {
    long long total = (long long)B * H * N;
#pragma omp parallel
    {
      double* a = (double*)malloc(sizeof(double) * (T ? T : 1));
#pragma omp for schedule(dynamic, 16)
      for (long long r = 0; r < total; ++r) {
        int n = (int)(r % N);
        int h = (int)((r / N) % H);
        int b = (int)(r / ((long long)N * H));
        attn_row(H, N, D, M, k, scale, Q, K, V, gid, gate, offsets, perm, b, h, n,
                 O + (size_t)r * D, a);
      }
      free(a);
    }
  }
  if (gid_out) memcpy(gid_out, gid, sizeof(int32_t) * (size_t)B * T);
  if (gate_out) memcpy(gate_out, gate, sizeof(double) * (size_t)B * T);
  if (offsets_out) memcpy(offsets_out, offsets, sizeof(int32_t) * (size_t)B * (M + 1));
  if (perm_out) memcpy(perm_out, perm, sizeof(int32_t) * (size_t)B * T);
  if (inv_out) memcpy(inv_out, inv, sizeof(int32_t) * (size_t)B * T);
  free(gid);
  free(gate);
  free(offsets);
  free(perm);
  free(inv);
  return rc;
}
