#include "generator.h"

#include <atomic>
#include <cmath>
#include <complex>
#include <thread>
#include <vector>

namespace dft3d {
namespace gen {

namespace {

constexpr double kHalfPi = 1.57079632679489661923132169163975144;

// (cos, sin) of quadrant*pi/2 + frac_of_quadrant*pi/2 with 0 <= frac_of_quadrant < 1.
// The angle handed to cos/sin never exceeds pi/4, and the quadrant is applied by exact swaps / sign flips.
void quadrant_phasor(int quadrant, double frac_of_quadrant, double* c, double* s) {
  double cc, ss;
  if (frac_of_quadrant <= 0.5) {
    const double th = frac_of_quadrant * kHalfPi;
    cc = std::cos(th);
    ss = std::sin(th);
  } else {
    const double th = (1.0 - frac_of_quadrant) * kHalfPi;
    cc = std::sin(th);
    ss = std::cos(th);
  }
  switch (quadrant & 3) {
    case 0: *c = cc; *s = ss; break;
    case 1: *c = -ss; *s = cc; break;
    case 2: *c = -cc; *s = -ss; break;
    default: *c = ss; *s = -cc; break;
  }
}

// exp(sign*2*pi*i*a*t) for an integer-valued a and any finite t: a*t is reduced modulo 1 with the
// rounding error of the product recovered by a fused multiply-add.
void node_phasor(double a, double t, int sign, double* re, double* im) {
  const double prod = a * t;
  const double err = std::fma(a, t, -prod);
  double f = prod - std::floor(prod);
  f += err;
  f -= std::floor(f);
  const double f4 = 4.0 * f;
  double qd = std::floor(f4);
  if (qd >= 4.0) qd = 3.0;
  double c, s;
  quadrant_phasor(static_cast<int>(qd), f4 - qd, &c, &s);
  *re = c;
  *im = sign < 0 ? -s : s;
}

}  // namespace

void root_of_unity(int64_t num, int64_t den, int sign, double* re, double* im) {
  const __int128 four = static_cast<__int128>(4) * num;
  const int quadrant = static_cast<int>(four / den);
  const int64_t rem = static_cast<int64_t>(four % den);
  double c, s;
  if (rem == 0) {
    quadrant_phasor(quadrant, 0.0, &c, &s);
  } else {
    quadrant_phasor(quadrant, static_cast<double>(rem) / static_cast<double>(den), &c, &s);
  }
  *re = c;
  *im = sign < 0 ? -s : s;
  if (*im == 0.0) *im = 0.0;  // no negative zero
}

void axis_matrix(int64_t n, int sign, double scale, const double* nodes, bool nodes_on_output, double* M) {
  for (int64_t k = 0; k < n; ++k) {
    for (int64_t j = 0; j < n; ++j) {
      double re, im;
      if (!nodes) {
        const int64_t m = static_cast<int64_t>((static_cast<__int128>(k) * j) % n);
        root_of_unity(m, n, sign, &re, &im);
      } else if (!nodes_on_output) {
        node_phasor(static_cast<double>(k), nodes[j], sign, &re, &im);
      } else {
        node_phasor(static_cast<double>(j), nodes[k], sign, &re, &im);
      }
      M[2 * (k * n + j)] = scale * re;
      M[2 * (k * n + j) + 1] = scale * im;
    }
  }
}

namespace {

// all threads of a team meet here; sense-reversing spin barrier (the waits are microseconds long)
struct SpinBarrier {
  explicit SpinBarrier(int n) : count(n), waiting(0), sense(0) {}
  void wait() {
    const int my = sense.load(std::memory_order_acquire);
    if (waiting.fetch_add(1, std::memory_order_acq_rel) + 1 == count) {
      waiting.store(0, std::memory_order_relaxed);
      sense.store(my ^ 1, std::memory_order_release);
    } else {
      while (sense.load(std::memory_order_acquire) == my) std::this_thread::yield();
    }
  }
  const int count;
  std::atomic<int> waiting, sense;
};

}  // namespace

bool invert_matrix(int64_t n, double* Mraw, double* growth) {
  using cd = std::complex<double>;
  cd* A = reinterpret_cast<cd*>(Mraw);
  double amax = 0.0;
  for (int64_t i = 0; i < n * n; ++i) amax = std::fmax(amax, std::abs(A[i]));
  std::vector<int64_t> perm(n);
  int threads = int(std::thread::hardware_concurrency());
  if (threads < 1) threads = 1;
  if (threads > 16) threads = 16;
  if (n < 128) threads = 1;
  SpinBarrier barrier(threads);
  std::atomic<int> singular(0);
  // Gauss-Jordan in place: after step k column k holds column k of the inverse of the row-permuted matrix
  auto worker = [&](int tid) {
    for (int64_t k = 0; k < n; ++k) {
      if (tid == 0) {
        int64_t piv = k;
        double best = std::abs(A[k * n + k]);
        for (int64_t i = k + 1; i < n; ++i) {
          const double v = std::abs(A[i * n + k]);
          if (v > best) { best = v; piv = i; }
        }
        perm[k] = piv;
        if (!(best > 0.0) || !std::isfinite(best)) {
          singular.store(1);
        } else {
          if (piv != k)
            for (int64_t j = 0; j < n; ++j) std::swap(A[k * n + j], A[piv * n + j]);
          const cd inv = 1.0 / A[k * n + k];
          A[k * n + k] = 1.0;
          for (int64_t j = 0; j < n; ++j) A[k * n + j] *= inv;
        }
      }
      barrier.wait();
      if (singular.load()) return;
      const cd* rk = A + k * n;
      for (int64_t i = tid; i < n; i += threads) {
        if (i == k) continue;
        cd* ri = A + i * n;
        const cd f = ri[k];
        ri[k] = 0.0;
        for (int64_t j = 0; j < n; ++j) ri[j] -= f * rk[j];
      }
      barrier.wait();
    }
  };
  std::vector<std::thread> team;
  for (int t = 1; t < threads; ++t) team.emplace_back(worker, t);
  worker(0);
  for (auto& t : team) t.join();
  if (singular.load()) return false;
  // undo the row exchanges: they become column exchanges of the inverse, in reverse order
  for (int64_t k = n - 1; k >= 0; --k)
    if (perm[k] != k)
      for (int64_t i = 0; i < n; ++i) std::swap(A[i * n + k], A[i * n + perm[k]]);
  double imax = 0.0;
  for (int64_t i = 0; i < n * n; ++i) imax = std::fmax(imax, std::abs(A[i]));
  if (!std::isfinite(imax)) return false;
  if (growth) *growth = imax * amax;
  return true;
}

void twiddle(int64_t N1, int64_t N2, int sign, double* T) {
  const int64_t N = N1 * N2;
  for (int64_t k1 = 0; k1 < N1; ++k1)
    for (int64_t b = 0; b < N2; ++b) {
      double re, im;
      root_of_unity((k1 * b) % N, N, sign, &re, &im);
      T[2 * (k1 * N2 + b)] = re;
      T[2 * (k1 * N2 + b) + 1] = im;
    }
}

float round_to_tf32(double v) {
  if (v == 0.0 || !std::isfinite(v)) return static_cast<float>(v);
  if (std::fabs(v) < 1e-30) return 0.0f;  // far below anything a DFT table holds; avoids float subnormals
  int e;
  const double m = std::frexp(v, &e);             // v = m * 2^e, 0.5 <= |m| < 1
  const double r = std::nearbyint(std::ldexp(m, 11));  // 11 significant bits, ties to even
  return static_cast<float>(std::ldexp(r, e - 11));
}

double round_to_fp16(double v) {
  if (v == 0.0 || !std::isfinite(v)) return v;
  const double a = std::fabs(v);
  if (a < 6.103515625e-05) {                       // below 2^-14: subnormal grid, spacing 2^-24
    return std::nearbyint(v * 16777216.0) / 16777216.0;
  }
  int e;
  const double m = std::frexp(v, &e);
  return std::ldexp(std::nearbyint(std::ldexp(m, 11)), e - 11);
}

void real_table_from_matrix(int64_t n, const double* M, float* hi, float* lo) {
  const int64_t ld = 2 * n;
  for (int64_t k = 0; k < n; ++k)
    for (int64_t j = 0; j < n; ++j) {
      const double re = M[2 * (k * n + j)], im = M[2 * (k * n + j) + 1];
      const int64_t r0 = (2 * k) * ld + 2 * j, r1 = (2 * k + 1) * ld + 2 * j;
      split_tf32(re, &hi[r0], &lo[r0]);
      split_tf32(-im, &hi[r0 + 1], &lo[r0 + 1]);
      split_tf32(im, &hi[r1], &lo[r1]);
      split_tf32(re, &hi[r1 + 1], &lo[r1 + 1]);
    }
}

}  // namespace gen
}  // namespace dft3d
