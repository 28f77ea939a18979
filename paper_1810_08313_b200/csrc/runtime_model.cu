// Runtime / delay model of local-update SGD (Sections 2-4 of the paper): host code only.
//
//   ls_delay            D = D_0 s(m)                                   (Section 2, delay model)
//   ls_speedup          (1 + alpha) / (1 + alpha / tau), alpha = D / Y  (Section 3.2)
//   ls_error_bound      Theorem 1, the error bound after wall-clock time T
//   ls_tau_star         Theorem 2, the period that minimises it
//   ls_simulate_runtime Monte-Carlo means of T_sync = max_i Y_i + D and T_P-Avg = max_i Ybar_i + D / tau
//                       (Section 3.1) for exponential or constant compute times
//
// The random compute times come from Philox4x32-10 (Salmon et al., SC'11), written here from its
// published definition: counter = (period lo, period hi, local step, worker), key = the seed.
#include <math.h>
#include <stdint.h>

#include <vector>

#include "ls.h"

namespace {

struct Block { uint32_t v[4]; };

inline void mulhilo(uint32_t a, uint32_t b, uint32_t* hi, uint32_t* lo) {
  const uint64_t p = (uint64_t)a * (uint64_t)b;
  *hi = (uint32_t)(p >> 32);
  *lo = (uint32_t)p;
}

Block philox4x32_10(Block c, uint32_t k0, uint32_t k1) {
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo(0xD2511F53u, c.v[0], &hi0, &lo0);
    mulhilo(0xCD9E8D57u, c.v[2], &hi1, &lo1);
    const Block n = {{hi1 ^ c.v[1] ^ k0, lo1, hi0 ^ c.v[3] ^ k1, lo0}};
    c = n;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

inline double compute_time(uint64_t seed, uint64_t period, uint32_t k, uint32_t worker, double y, bool exponential) {
  if (!exponential) return y;
  const Block c = {{(uint32_t)period, (uint32_t)(period >> 32), k, worker}};
  const uint32_t x = philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32)).v[0];
  const double u = ((double)x + 0.5) / 4294967296.0;      // in (0, 1)
  return -y * log(u);
}

}  // namespace

extern "C" {

int ls_philox4x32_10(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4]) {
  if (counter == nullptr || key == nullptr || out == nullptr) return LS_ERR_INVALID_ARG;
  const Block c = {{counter[0], counter[1], counter[2], counter[3]}};
  const Block r = philox4x32_10(c, key[0], key[1]);
  for (int i = 0; i < 4; ++i) out[i] = r.v[i];
  return LS_OK;
}

int ls_delay(double D0, int m, int scaling, double* D) {
  if (D == nullptr || m < 1 || !isfinite(D0) || D0 < 0.0) return LS_ERR_INVALID_ARG;
  double s;
  switch (scaling) {
    case LS_DELAY_CONSTANT: s = 1.0; break;
    case LS_DELAY_LOG2: s = log2((double)m); break;
    case LS_DELAY_TREE: s = 2.0 * log2((double)m); break;
    case LS_DELAY_LINEAR: s = (double)m; break;
    default: return LS_ERR_INVALID_ARG;
  }
  *D = D0 * s;
  return LS_OK;
}

int ls_speedup(double alpha, int tau, double* speedup) {
  if (speedup == nullptr || tau < 1 || !isfinite(alpha) || alpha < 0.0) return LS_ERR_INVALID_ARG;
  *speedup = (1.0 + alpha) / (1.0 + alpha / (double)tau);
  return LS_OK;
}

int ls_error_bound(double T, double F1, double Finf, double lr, double L, double sigma2, int m, int tau, double Y,
                   double D, double* bound) {
  if (bound == nullptr || m < 1 || tau < 1) return LS_ERR_INVALID_ARG;
  if (!(T > 0.0) || !(lr > 0.0) || !(L >= 0.0) || !(sigma2 >= 0.0) || !(Y >= 0.0) || !(D >= 0.0) || !isfinite(F1) ||
      !isfinite(Finf) || !isfinite(T) || !isfinite(lr) || !isfinite(L) || !isfinite(sigma2) || !isfinite(Y) || !isfinite(D))
    return LS_ERR_INVALID_ARG;
  *bound = 2.0 * (F1 - Finf) / (lr * T) * (Y + D / (double)tau) + lr * L * sigma2 / (double)m +
           lr * lr * L * L * sigma2 * (double)(tau - 1);
  return LS_OK;
}

int ls_tau_star(double F1, double Finf, double D, double lr, double L, double sigma2, double T, double* tau) {
  if (tau == nullptr) return LS_ERR_INVALID_ARG;
  if (!(T > 0.0) || !(lr > 0.0) || !(L > 0.0) || !(sigma2 > 0.0) || !(D >= 0.0) || !(F1 >= Finf) || !isfinite(F1) ||
      !isfinite(Finf) || !isfinite(T) || !isfinite(lr) || !isfinite(L) || !isfinite(sigma2) || !isfinite(D))
    return LS_ERR_INVALID_ARG;
  *tau = sqrt(2.0 * (F1 - Finf) * D / (lr * lr * lr * L * L * sigma2 * T));
  return LS_OK;
}

int ls_simulate_runtime(int m, int tau, int64_t n_periods, double y_mean, double D, uint64_t seed, int exponential,
                        double* t_sync_mean, double* t_pavg_mean) {
  if (m < 1 || tau < 1 || n_periods < 1 || t_sync_mean == nullptr || t_pavg_mean == nullptr) return LS_ERR_INVALID_ARG;
  if (!(y_mean >= 0.0) || !(D >= 0.0) || !isfinite(y_mean) || !isfinite(D)) return LS_ERR_INVALID_ARG;
  std::vector<double> ybar((size_t)m);
  double sum_sync = 0.0, sum_pavg = 0.0;
  for (int64_t p = 0; p < n_periods; ++p) {
    for (int i = 0; i < m; ++i) ybar[(size_t)i] = 0.0;
    for (int k = 0; k < tau; ++k) {
      // this local step taken as one iteration of fully synchronous SGD: T = max_i Y_i + D
      double mx = 0.0;
      for (int i = 0; i < m; ++i) {
        const double yv = compute_time(seed, (uint64_t)p, (uint32_t)k, (uint32_t)i, y_mean, exponential != 0);
        if (i == 0 || yv > mx) mx = yv;
        ybar[(size_t)i] += yv;
      }
      sum_sync += mx + D;
    }
    // the same draws as one period of PASGD: T = max_i (sum_k Y_ik / tau) + D / tau
    double mx = 0.0;
    for (int i = 0; i < m; ++i) {
      const double v = ybar[(size_t)i] / (double)tau;
      if (i == 0 || v > mx) mx = v;
    }
    sum_pavg += mx + D / (double)tau;
  }
  *t_sync_mean = sum_sync / ((double)n_periods * (double)tau);
  *t_pavg_mean = sum_pavg / (double)n_periods;
  return LS_OK;
}

}  // extern "C"
