// Timed twin of the CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// The same float64 restatement as oracle/kvswap_oracle.py (steps O2..O7: Eq. 1, "Scoring and
// selection" of Sec. 4.3, the decode attention of Sec. 4.4 / 4.4.1 / 4.4.4), written as plain loops
// with one OpenMP pragma per step so that the benchmark can time the method on all host cores
// instead of timing the Python interpreter.  No blocking, no fusion, no pre-summing: every step
// materialises its result and the next step reads it, in the paper's order.  It shares no code
// with the CUDA library and is checked against the numpy oracle (which stays the parity
// authority) by tests/test_oracle_omp.py.
//
// Inputs are float arrays holding the exact values of the stored types (bf16 / fp16 / fp32
// widen to float without rounding); all arithmetic is double.
//   q [B, H_q, d]   proj [H_kv, d, r]   meta [B, H_m, N, r]   K, V [B, H_kv, N, d]
//   scope: 0 = one selection per (sequence, KV head), 1 = one per sequence (all heads summed)
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <numeric>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

int kvo_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// O2..O6.  idx [B, S, M'] (M' = min(M, floor(N / G))), ascending; R_opt NULL or [B, S, NG].
int kvo_score_select(const float* q, const float* proj, const float* meta, int B, int Hq, int Hkv, int d, int r,
                     int Hm, int N, int G, int M, int scope, int32_t* idx, double* R_opt) {
  if (Hq % Hkv != 0 || (Hm != 1 && Hm != Hkv) || G < 1 || M < 1) return 1;
  const int rho = Hq / Hkv;
  const int S = scope == 0 ? Hkv : 1;
  const int NG = N / G;
  const int Mp = std::min(M, NG);
  // O2: low-rank query Q_h A_g(h)   (Eq. 1)
  std::vector<double> q_lr(size_t(B) * Hq * r);
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < Hq; ++h) {
      const float* A = proj + size_t(h / rho) * d * r;
      for (int j = 0; j < r; ++j) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += double(q[(size_t(b) * Hq + h) * d + c]) * double(A[size_t(c) * r + j]);
        q_lr[(size_t(b) * Hq + h) * r + j] = acc;
      }
    }
  // O3: per-head scores (Q_h A_g(h)) K_lr^T   (Eq. 1): raw logits
  std::vector<double> s(size_t(B) * Hq * N);
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < Hq; ++h) {
      const int m = Hm == 1 ? 0 : h / rho;
      const float* Mrow = meta + (size_t(b) * Hm + m) * N * r;
      const double* u = &q_lr[(size_t(b) * Hq + h) * r];
      for (int n = 0; n < N; ++n) {
        double acc = 0.0;
        for (int j = 0; j < r; ++j) acc += u[j] * double(Mrow[size_t(n) * r + j]);
        s[(size_t(b) * Hq + h) * N + n] = acc;
      }
    }
  // O4: sum over the heads of a scope   (Sec. 4.3)
  std::vector<double> T(size_t(B) * S * N);
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int sc = 0; sc < S; ++sc) {
      const int h0 = scope == 0 ? sc * rho : 0, h1 = scope == 0 ? (sc + 1) * rho : Hq;
      for (int n = 0; n < N; ++n) {
        double acc = 0.0;
        for (int h = h0; h < h1; ++h) acc += s[(size_t(b) * Hq + h) * N + n];
        T[(size_t(b) * S + sc) * N + n] = acc;
      }
    }
  // O5: ReduceMax over groups of G consecutive tokens; the N mod G newest tokens form no group
  std::vector<double> R(size_t(B) * S * std::max(NG, 1));
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int sc = 0; sc < S; ++sc)
      for (int j = 0; j < NG; ++j) {
        double mx = T[(size_t(b) * S + sc) * N + size_t(j) * G];
        for (int t = 1; t < G; ++t) mx = std::max(mx, T[(size_t(b) * S + sc) * N + size_t(j) * G + t]);
        R[(size_t(b) * S + sc) * NG + j] = mx;
      }
  // O6: TopK: the M' largest, the lower index first among equal scores; written in ascending index order
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int sc = 0; sc < S; ++sc) {
      const double* Rr = &R[(size_t(b) * S + sc) * NG];
      std::vector<int32_t> order(NG);
      std::iota(order.begin(), order.end(), 0);
      std::sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return Rr[x] > Rr[y] || (Rr[x] == Rr[y] && x < y); });
      std::sort(order.begin(), order.begin() + Mp);
      for (int i = 0; i < Mp; ++i) idx[(size_t(b) * S + sc) * Mp + i] = order[i];
    }
  if (R_opt != nullptr) std::copy(R.begin(), R.begin() + size_t(B) * S * NG, R_opt);
  return 0;
}

// O7.  idx [B, S, Mp]; out [B, H_q, d], lse [B, H_q] (double).
int kvo_attend(const float* q, const float* K, const float* V, const int32_t* idx, int Mp, int B, int Hq, int Hkv, int d,
               int N, int G, int scope, double* out, double* lse) {
  if (Hq % Hkv != 0 || G < 1) return 1;
  const int rho = Hq / Hkv;
  const int S = scope == 0 ? Hkv : 1;
  const int NG = N / G;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < Hq; ++h) {
      const int g = h / rho, sc = scope == 0 ? g : 0;
      std::vector<int64_t> tokens;
      for (int i = 0; i < Mp; ++i)
        for (int t = 0; t < G; ++t) tokens.push_back(int64_t(idx[(size_t(b) * S + sc) * Mp + i]) * G + t);
      for (int n = NG * G; n < N; ++n) tokens.push_back(n);          // the rolling-buffer tail is always attended
      const float* qh = q + (size_t(b) * Hq + h) * d;
      const float* Kg = K + (size_t(b) * Hkv + g) * N * d;
      const float* Vg = V + (size_t(b) * Hkv + g) * N * d;
      std::vector<double> logit(tokens.size());
      const double scale = 1.0 / std::sqrt(double(d));
      for (size_t i = 0; i < tokens.size(); ++i) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += double(qh[c]) * double(Kg[size_t(tokens[i]) * d + c]);
        logit[i] = acc * scale;
      }
      double* o = out + (size_t(b) * Hq + h) * d;
      if (tokens.empty()) {                                           // nothing attended
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        lse[size_t(b) * Hq + h] = -INFINITY;
        continue;
      }
      // two-pass softmax with max subtraction
      double mx = logit[0];
      for (double v : logit) mx = std::max(mx, v);
      double denom = 0.0;
      for (double& v : logit) { v = std::exp(v - mx); denom += v; }
      for (int c = 0; c < d; ++c) o[c] = 0.0;
      for (size_t i = 0; i < tokens.size(); ++i) {
        const double pw = logit[i] / denom;
        for (int c = 0; c < d; ++c) o[c] += pw * double(Vg[size_t(tokens[i]) * d + c]);
      }
      lse[size_t(b) * Hq + h] = mx + std::log(denom);
    }
  return 0;
}

}  // extern "C"
