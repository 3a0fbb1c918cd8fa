// CPU oracle for the DAM (Dynamic Attention Mask) prefill path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, float64 statement of
// what the hot path computes.  It shares no code with the CUDA library, is never
// linked into it, and may only be called from tests, the smoke check and the
// benchmark's CPU-baseline leg.
//
// Every function follows one passage of the paper (cited by section / equation
// in the comment above it) in the paper's own order; there is no blocking,
// tiling or fusion here.  OpenMP parallelises independent rows only.
//
// Pins (see tests/test_oracle_*.py): Table 2's Box-Cox maximum, closed forms for
// uniform attention, injected band / sink score tensors, brute force from the
// literal pattern matrices, float64 library attention, invariants.
//
// Build: g++ -O2 -fopenmp -ffp-contract=off -shared -fPIC (no fast-math: the
// fp32 threshold chain below relies on IEEE single operations, unfused).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// ---------------------------------------------------------------------------
// Sec. 3 ("Preliminaries"): S = Q K^T / sqrt(d_k), softmax over keys.
// Sec. 4.2.1: only the first L tokens (the pattern-capture window) take part.
// Causal map: P[i][j] = softmax_{j<=i}(scale * q_i . k_j), and 0 for j > i.
// Q, K point at (first token of the sequence, this head); consecutive tokens
// are q_stride / k_stride floats apart.  P is [L][L] float64, row-major.
// ---------------------------------------------------------------------------
int oracle_window_probs(const float* Q, const float* K, int L, int d,
                        int64_t q_stride, int64_t k_stride, double scale,
                        double* P) {
  if (!Q || !K || !P || L < 0 || d <= 0) return 1;
#pragma omp parallel for schedule(dynamic, 8)
  for (int i = 0; i < L; ++i) {
    std::vector<double> s(i + 1);
    double m = -std::numeric_limits<double>::infinity();
    for (int j = 0; j <= i; ++j) {
      double acc = 0.0;
      for (int t = 0; t < d; ++t)
        acc += (double)Q[i * q_stride + t] * (double)K[j * k_stride + t];
      s[j] = acc * scale;
      if (s[j] > m) m = s[j];
    }
    double l = 0.0;
    for (int j = 0; j <= i; ++j) l += std::exp(s[j] - m);
    for (int j = 0; j <= i; ++j) P[(int64_t)i * L + j] = std::exp(s[j] - m) / l;
    for (int j = i + 1; j < L; ++j) P[(int64_t)i * L + j] = 0.0;
  }
  return 0;
}

// ---------------------------------------------------------------------------
// Sec. 4.2.2: X = max(Abar, eps);  B = (X^lambda - 1)/lambda  (ln X if
// lambda = 0);  B* = B - min B.  The minimum runs over every cell of every
// map, and every map has cells above the diagonal where Abar = 0, so the
// minimum is the constant B(eps).  Sec. 4.2.3: m_ij = [B*_ij >= tau].
// Float64 version (the map itself was computed in float64).
// ---------------------------------------------------------------------------
static double boxcox64(double x, double lambda) {
  if (lambda != 0.0) return (std::pow(x, lambda) - 1.0) / lambda;
  return std::log(x);
}

int oracle_amplify_f64(const double* P, int64_t n, double lambda, double eps,
                       double* A_tilde) {
  if (!P || !A_tilde || n < 0 || !(eps > 0.0)) return 1;
  const double bmin = boxcox64(eps, lambda);
  for (int64_t t = 0; t < n; ++t) {
    double x = P[t] > eps ? P[t] : eps;
    A_tilde[t] = boxcox64(x, lambda) - bmin;
  }
  return 0;
}

int oracle_true_mask_f64(const double* P, int L, double tau, double lambda,
                         double eps, uint8_t* M) {
  if (!P || !M || L < 0 || !(eps > 0.0)) return 1;
  const double bmin = boxcox64(eps, lambda);
  for (int i = 0; i < L; ++i)
    for (int j = 0; j < L; ++j) {
      double p = P[(int64_t)i * L + j];
      double x = p > eps ? p : eps;
      double a = boxcox64(x, lambda) - bmin;
      M[(int64_t)i * L + j] = (a >= tau) ? 1 : 0;
    }
  return 0;
}

// Same rule on an fp32 score tensor, lambda = 0.5, every operation an IEEE
// single-precision operation in this order (no fused multiply-add):
//   x = max(p, eps); b = (sqrt(x) - 1) * 2; bmin = (sqrt(eps) - 1) * 2;
//   a = b - bmin; active = a >= tau.
// This is the form both sides evaluate when masks must agree bit for bit.
int oracle_true_mask_f32(const float* P, int L, float tau, float eps,
                         uint8_t* M) {
  if (!P || !M || L < 0 || !(eps > 0.0f)) return 1;
  volatile float se = std::sqrt(eps);
  volatile float bmin_v = (se - 1.0f) * 2.0f;
  const float bmin = bmin_v;
#pragma omp parallel for schedule(static)
  for (int i = 0; i < L; ++i)
    for (int j = 0; j < L; ++j) {
      float p = P[(int64_t)i * L + j];
      float x = p > eps ? p : eps;
      float r = std::sqrt(x);
      float b = (r - 1.0f) * 2.0f;
      float a = b - bmin;
      M[(int64_t)i * L + j] = (a >= tau) ? 1 : 0;
    }
  return 0;
}

// ---------------------------------------------------------------------------
// Sec. 4.2.4: pattern pool.  Diagonal r: cells (i, i-r), i in [r, L).
// Vertical c: cells (i, c), i in [c, L).  The match score's numerator is the
// number of mask cells on the pattern; its denominator the pattern's size.
// ---------------------------------------------------------------------------
int oracle_pattern_counts(const uint8_t* M, int L, int32_t* cntD,
                          int32_t* cntV) {
  if (!M || !cntD || !cntV || L < 0) return 1;
  for (int r = 0; r < L; ++r) {
    int32_t c = 0;
    for (int i = r; i < L; ++i) c += M[(int64_t)i * L + (i - r)] ? 1 : 0;
    cntD[r] = c;
  }
  for (int c = 0; c < L; ++c) {
    int32_t n = 0;
    for (int i = c; i < L; ++i) n += M[(int64_t)i * L + c] ? 1 : 0;
    cntV[c] = n;
  }
  return 0;
}

// gamma_k >= mu, with gamma_k = cnt / size, decided without a division as
// (float)cnt >= mu * (float)size in single precision (one multiply, one
// compare).  Patterns of fewer than min_support cells are ignored
// (min_support = 1 is the paper's rule: every pattern takes part).
int oracle_match(const int32_t* cntD, const int32_t* cntV, int L, float mu,
                 int min_support, uint8_t* D, uint8_t* V) {
  if (!cntD || !cntV || !D || !V || L < 0) return 1;
  for (int k = 0; k < L; ++k) {
    int size = L - k;
    volatile float need = mu * (float)size;
    bool ok = size >= min_support;
    D[k] = (ok && (float)cntD[k] >= need) ? 1 : 0;
    V[k] = (ok && (float)cntV[k] >= need) ? 1 : 0;
  }
  return 0;
}

// ---------------------------------------------------------------------------
// Sec. 4.3: Case 1 (S <= L): the true mask.  Case 2 (S > L): the L x L block
// keeps the true mask; every later row i >= L attends j iff (i, j) lies on a
// matched pattern extended to the full length: a matched vertical c (j = c)
// or a matched diagonal r (i - j = r).  Nothing above the diagonal.
// out is [nrows][S] bytes for the requested rows.
// ---------------------------------------------------------------------------
int oracle_extended_rows(const uint8_t* M, const uint8_t* D, const uint8_t* V,
                         int L, int S, const int32_t* rows, int nrows,
                         uint8_t* out) {
  if (!M || !D || !V || !rows || !out || L < 0 || S < L) return 1;
  for (int a = 0; a < nrows; ++a) {
    int i = rows[a];
    if (i < 0 || i >= S) return 2;
    uint8_t* o = out + (int64_t)a * S;
    for (int j = 0; j < S; ++j) {
      uint8_t bit = 0;
      if (j <= i) {
        if (i < L) {
          bit = M[(int64_t)i * L + j];
        } else {
          bool vert = (j < L) && V[j];
          bool diag = (i - j < L) && D[i - j];
          bit = (vert || diag) ? 1 : 0;
        }
      }
      o[j] = bit;
    }
  }
  return 0;
}

// ---------------------------------------------------------------------------
// Sec. 4.3 (last paragraph) and Sec. 3: logits q_i . k_j / sqrt(d_k); masked
// positions are set to -inf before the softmax; O = softmax(.) V.
// Computed for the requested rows over ALL S keys of the sequence.
// mask_rows: [nrows][S] bytes (1 = attend) or NULL for "attend everything".
// causal != 0 additionally removes j > i.
// LSE_i = max + ln(sum exp(s - max)) over the active keys (natural log).
// A row with no active key gives O = 0 and LSE = -inf.
// ---------------------------------------------------------------------------
int oracle_attention_rows(const float* Q, const float* K, const float* V,
                          int S, int d, int64_t q_stride, int64_t k_stride,
                          int64_t v_stride, double scale, const int32_t* rows,
                          int nrows, const uint8_t* mask_rows, int causal,
                          double* O, double* lse) {
  if (!Q || !K || !V || !rows || !O || !lse || S < 0 || d <= 0) return 1;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 4) reduction(| : bad)
  for (int a = 0; a < nrows; ++a) {
    int i = rows[a];
    if (i < 0 || i >= S) { bad |= 1; continue; }
    const uint8_t* mrow = mask_rows ? mask_rows + (int64_t)a * S : nullptr;
    std::vector<double> s(S);
    const double ninf = -std::numeric_limits<double>::infinity();
    double m = ninf;
    for (int j = 0; j < S; ++j) {
      bool active = (!mrow || mrow[j]) && !(causal && j > i);
      if (!active) { s[j] = ninf; continue; }
      double acc = 0.0;
      for (int t = 0; t < d; ++t)
        acc += (double)Q[i * q_stride + t] * (double)K[j * k_stride + t];
      s[j] = acc * scale;
      if (s[j] > m) m = s[j];
    }
    double* o = O + (int64_t)a * d;
    for (int t = 0; t < d; ++t) o[t] = 0.0;
    if (m == ninf) { lse[a] = ninf; continue; }
    double l = 0.0;
    for (int j = 0; j < S; ++j)
      if (s[j] != ninf) l += std::exp(s[j] - m);
    for (int j = 0; j < S; ++j) {
      if (s[j] == ninf) continue;
      double w = std::exp(s[j] - m) / l;
      for (int t = 0; t < d; ++t) o[t] += w * (double)V[j * v_stride + t];
    }
    lse[a] = m + std::log(l);
  }
  return bad ? 2 : 0;
}

int oracle_num_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
#endif
  return n;
}

}  // extern "C"
