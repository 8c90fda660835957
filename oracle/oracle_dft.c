/*
 * Oracle for the 3D complex DFT -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, float64 direct-summation evaluation of the transform that the
 * GPU library computes.  It exists only so that tests, the smoke check and the
 * bench's CPU-baseline leg have something independent to compare against; the
 * product path never calls it and shares no code, table or constant with it.
 *
 * What it evaluates (paper Eq. 11, the 3D DFT on a rectangular grid, written
 * per axis as in Eq. 12-13 with one Vandermonde matrix per axis):
 *
 *   X[k0,k1,k2] = sum_{n0,n1,n2} x[n0,n1,n2] M_0[k0,n0] M_1[k1,n1] M_2[k2,n2]
 *   M_a[k,j]    = c_a * exp(sign * 2*pi*i * k * t_a[j])
 *
 * with t_a[j] = j/n_a on the uniform grid (Eq. 14 fixes the kernel and the
 * negative exponent of the forward transform) or t_a[j] = the caller's node
 * x_j for a nonuniform axis (the Vandermonde matrix of Eq. 3 with its sample
 * points taken on the unit circle).  c_a = 1, or 1/n_a when the caller asks
 * for the scaled inverse.  With `nodes_on_output` the roles swap and
 * M_a[k,j] = exp(sign*2*pi*i * w_k * j): Eq. 1 read literally (arbitrary
 * evaluation points z_k, integer powers n).
 *
 * No FFT, no BLAS, no blocking: each output of each axis pass is an O(n_a)
 * sum in double precision.  Phases are reduced exactly before sin/cos:
 * (k*j) mod n in integers on the uniform grid, and the fractional part of
 * k*x_j with the product's rounding error recovered by fma for nodes.
 *
 * Every function here is pinned by tests/test_oracle_pins.py (closed forms,
 * brute force, invariants, library special cases).
 *
 * Layout everywhere: row-major [n0][n1][n2], interleaved complex (re, im).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_TWO_PI 6.283185307179586476925286766559

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* exp(sign*2*pi*i*frac) for frac already reduced to [0,1) */
static void unit_phasor(double frac, int sign, double* re, double* im) {
  double ang = ORACLE_TWO_PI * frac;
  *re = cos(ang);
  *im = (sign < 0) ? -sin(ang) : sin(ang);
}

/*
 * One entry of the per-axis matrix (Eq. 3 / Eq. 13 with unit-circle points;
 * Eq. 14's kernel when nodes == NULL).
 *   nodes == NULL         : phase = k*j/n, reduced as ((k*j) mod n)/n
 *   nodes, on input  (0)  : phase = k * nodes[j]
 *   nodes, on output (1)  : phase = nodes[k] * j
 */
static void matrix_entry(int64_t n, int64_t k, int64_t j, int sign, const double* nodes,
                         int nodes_on_output, double* re, double* im) {
  double frac;
  if (!nodes) {
    int64_t m = (int64_t)(((__int128)k * (__int128)j) % (__int128)n);
    frac = (double)m / (double)n;
    /* exact values at the quarter turns, so that structured pins stay exact */
    if (4 * m == 0) { *re = 1.0; *im = 0.0; return; }
    if (4 * m == n) { *re = 0.0; *im = (sign < 0) ? -1.0 : 1.0; return; }
    if (4 * m == 2 * n) { *re = -1.0; *im = 0.0; return; }
    if (4 * m == 3 * n) { *re = 0.0; *im = (sign < 0) ? 1.0 : -1.0; return; }
  } else {
    double a = nodes_on_output ? (double)j : (double)k; /* the integer factor  */
    double t = nodes_on_output ? nodes[k] : nodes[j];   /* the real-valued one */
    double p = a * t;
    double e = fma(a, t, -p); /* p + e == a*t exactly */
    frac = (p - floor(p)) + e;
    frac -= floor(frac);
  }
  unit_phasor(frac, sign, re, im);
}

/*
 * Fill the dense n x n complex matrix M[k][j] (row-major, interleaved) for one
 * axis, times `scale`.  Exposed so tests can pin it directly.
 */
void oracle_axis_matrix(int64_t n, int sign, double scale, const double* nodes,
                        int nodes_on_output, double* M) {
  for (int64_t k = 0; k < n; ++k)
    for (int64_t j = 0; j < n; ++j) {
      double re, im;
      matrix_entry(n, k, j, sign, nodes, nodes_on_output, &re, &im);
      M[2 * (k * n + j)] = scale * re;
      M[2 * (k * n + j) + 1] = scale * im;
    }
}

/*
 * One axis of the transform by direct summation (the mode-`axis` product of
 * Eq. 12; Eq. 5 shows which side multiplies: axis 0 is V1 from the left,
 * the last axis is V^T from the right):
 *   out[.., k, ..] = sum_j M[k,j] * in[.., j, ..]
 * in/out: n0*n1*n2 complex doubles, distinct buffers.
 */
void oracle_dft_axis(const double* in, double* out, int64_t n0, int64_t n1, int64_t n2,
                     int axis, int sign, double scale, const double* nodes,
                     int nodes_on_output) {
  int64_t dims[3] = {n0, n1, n2};
  int64_t n = dims[axis];
  double* M = (double*)malloc(sizeof(double) * 2 * (size_t)n * (size_t)n);
  oracle_axis_matrix(n, sign, scale, nodes, nodes_on_output, M);
  int64_t outer = 1, inner = 1;
  for (int a = 0; a < axis; ++a) outer *= dims[a];
  for (int a = axis + 1; a < 3; ++a) inner *= dims[a];
  /* element (o, j, c) lives at ((o*n + j)*inner + c) */
  if (inner == 1) {
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < outer; ++o) {
      const double* x = in + 2 * o * n;
      double* y = out + 2 * o * n;
      for (int64_t k = 0; k < n; ++k) {
        const double* m = M + 2 * k * n;
        double sr = 0.0, si = 0.0;
        for (int64_t j = 0; j < n; ++j) {
          sr += m[2 * j] * x[2 * j] - m[2 * j + 1] * x[2 * j + 1];
          si += m[2 * j] * x[2 * j + 1] + m[2 * j + 1] * x[2 * j];
        }
        y[2 * k] = sr;
        y[2 * k + 1] = si;
      }
    }
  } else {
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t o = 0; o < outer; ++o)
      for (int64_t k = 0; k < n; ++k) {
        double* y = out + 2 * ((o * n + k) * inner);
        for (int64_t c = 0; c < 2 * inner; ++c) y[c] = 0.0;
        for (int64_t j = 0; j < n; ++j) {
          const double mr = M[2 * (k * n + j)], mi = M[2 * (k * n + j) + 1];
          const double* x = in + 2 * ((o * n + j) * inner);
          for (int64_t c = 0; c < inner; ++c) {
            y[2 * c] += mr * x[2 * c] - mi * x[2 * c + 1];
            y[2 * c + 1] += mr * x[2 * c + 1] + mi * x[2 * c];
          }
        }
      }
  }
  free(M);
}

/*
 * The whole 3D transform: three successive axis passes (the operators of
 * Eq. 12 commute; the order here is last axis first).
 * sign: -1 forward, +1 conjugate kernel.  scaled_inverse != 0 multiplies the
 * axis matrices by 1/n_a.  nodesA may be NULL (uniform axis).
 * Returns 0, or -1 when out of memory.
 */
int oracle_dft3d(const double* in, double* out, int64_t n0, int64_t n1, int64_t n2, int sign,
                 int scaled_inverse, const double* nodes0, const double* nodes1,
                 const double* nodes2, int nodes_on_output) {
  size_t P = (size_t)n0 * (size_t)n1 * (size_t)n2;
  double* tmp = (double*)malloc(sizeof(double) * 2 * P);
  if (!tmp) return -1;
  double s0 = scaled_inverse ? 1.0 / (double)n0 : 1.0;
  double s1 = scaled_inverse ? 1.0 / (double)n1 : 1.0;
  double s2 = scaled_inverse ? 1.0 / (double)n2 : 1.0;
  oracle_dft_axis(in, out, n0, n1, n2, 2, sign, s2, nodes2, nodes_on_output);
  oracle_dft_axis(out, tmp, n0, n1, n2, 1, sign, s1, nodes1, nodes_on_output);
  oracle_dft_axis(tmp, out, n0, n1, n2, 0, sign, s0, nodes0, nodes_on_output);
  free(tmp);
  return 0;
}

/* Same, for the float32 samples the GPU saw (widened exactly to double). */
int oracle_dft3d_f32(const float* in, double* out, int64_t n0, int64_t n1, int64_t n2, int sign,
                     int scaled_inverse, const double* nodes0, const double* nodes1,
                     const double* nodes2, int nodes_on_output) {
  size_t P = (size_t)n0 * (size_t)n1 * (size_t)n2;
  double* wide = (double*)malloc(sizeof(double) * 2 * P);
  if (!wide) return -1;
  for (size_t i = 0; i < 2 * P; ++i) wide[i] = (double)in[i];
  int rc = oracle_dft3d(wide, out, n0, n1, n2, sign, scaled_inverse, nodes0, nodes1, nodes2,
                        nodes_on_output);
  free(wide);
  return rc;
}

/*
 * One coefficient by the literal triple sum of Eq. 11 (no shared partial
 * sums, matrix entries evaluated on the fly).  Slow: O(n0*n1*n2) per call.
 */
void oracle_coeff_triple_f32(const float* in, int64_t n0, int64_t n1, int64_t n2, int sign,
                             int scaled_inverse, const double* nodes0, const double* nodes1,
                             const double* nodes2, int nodes_on_output, int64_t k0, int64_t k1,
                             int64_t k2, double* out_re, double* out_im) {
  double sr = 0.0, si = 0.0;
#pragma omp parallel for reduction(+ : sr, si) schedule(static)
  for (int64_t a = 0; a < n0; ++a) {
    double e0r, e0i;
    matrix_entry(n0, k0, a, sign, nodes0, nodes_on_output, &e0r, &e0i);
    for (int64_t b = 0; b < n1; ++b) {
      double e1r, e1i;
      matrix_entry(n1, k1, b, sign, nodes1, nodes_on_output, &e1r, &e1i);
      double pr = e0r * e1r - e0i * e1i, pi = e0r * e1i + e0i * e1r;
      for (int64_t c = 0; c < n2; ++c) {
        double e2r, e2i;
        matrix_entry(n2, k2, c, sign, nodes2, nodes_on_output, &e2r, &e2i);
        double wr = pr * e2r - pi * e2i, wi = pr * e2i + pi * e2r;
        const float* x = in + 2 * ((a * n1 + b) * n2 + c);
        sr += wr * (double)x[0] - wi * (double)x[1];
        si += wr * (double)x[1] + wi * (double)x[0];
      }
    }
  }
  double s = scaled_inverse ? 1.0 / ((double)n0 * (double)n1 * (double)n2) : 1.0;
  *out_re = s * sr;
  *out_im = s * si;
}

/*
 * Coefficients on a product grid S0 x S1 x S2 of output indices, streaming the
 * input one slab of n0-planes at a time (so a cube that does not fit in host
 * memory can be checked).  Each value is still its full triple sum of Eq. 11;
 * only the partial sums over n2 and n1 are shared between coefficients that
 * have the same (k1,k2) / k2.
 *
 * acc: |S0|*|S1|*|S2| complex doubles, row-major over (i0,i1,i2); the caller
 * zeroes it before the first slab and reads it after the last.  The slab holds
 * planes n0 = plane_begin .. plane_begin+planes-1 as float32 complex.
 */
int oracle_subset_accumulate_f32(const float* slab, int64_t plane_begin, int64_t planes,
                                 int64_t n0, int64_t n1, int64_t n2, int sign,
                                 int scaled_inverse, const double* nodes0, const double* nodes1,
                                 const double* nodes2, int nodes_on_output, const int64_t* S0,
                                 int64_t s0, const int64_t* S1, int64_t s1, const int64_t* S2,
                                 int64_t s2, double* acc) {
  double c0 = scaled_inverse ? 1.0 / (double)n0 : 1.0;
  double c1 = scaled_inverse ? 1.0 / (double)n1 : 1.0;
  double c2 = scaled_inverse ? 1.0 / (double)n2 : 1.0;
  /* rows of the axis matrices for the wanted output indices only */
  double* R2 = (double*)malloc(sizeof(double) * 2 * (size_t)s2 * (size_t)n2);
  double* R1 = (double*)malloc(sizeof(double) * 2 * (size_t)s1 * (size_t)n1);
  double* T = (double*)malloc(sizeof(double) * 2 * (size_t)planes * (size_t)s1 * (size_t)s2);
  if (!R2 || !R1 || !T) { free(R2); free(R1); free(T); return -1; }
  for (int64_t i = 0; i < s2; ++i)
    for (int64_t j = 0; j < n2; ++j) {
      double re, im;
      matrix_entry(n2, S2[i], j, sign, nodes2, nodes_on_output, &re, &im);
      R2[2 * (i * n2 + j)] = c2 * re;
      R2[2 * (i * n2 + j) + 1] = c2 * im;
    }
  for (int64_t i = 0; i < s1; ++i)
    for (int64_t j = 0; j < n1; ++j) {
      double re, im;
      matrix_entry(n1, S1[i], j, sign, nodes1, nodes_on_output, &re, &im);
      R1[2 * (i * n1 + j)] = c1 * re;
      R1[2 * (i * n1 + j) + 1] = c1 * im;
    }
#pragma omp parallel
  {
    double* U = (double*)malloc(sizeof(double) * 2 * (size_t)n1 * (size_t)s2);
#pragma omp for schedule(dynamic, 1)
    for (int64_t p = 0; p < planes; ++p) {
      /* U[b, i2] = sum_c x[p,b,c] M_2[S2[i2], c] */
      for (int64_t b = 0; b < n1; ++b) {
        const float* x = slab + 2 * ((p * n1 + b) * n2);
        for (int64_t i2 = 0; i2 < s2; ++i2) {
          const double* m = R2 + 2 * i2 * n2;
          double sr = 0.0, si = 0.0;
          for (int64_t c = 0; c < n2; ++c) {
            double xr = (double)x[2 * c], xi = (double)x[2 * c + 1];
            sr += m[2 * c] * xr - m[2 * c + 1] * xi;
            si += m[2 * c] * xi + m[2 * c + 1] * xr;
          }
          U[2 * (b * s2 + i2)] = sr;
          U[2 * (b * s2 + i2) + 1] = si;
        }
      }
      /* T[p, i1, i2] = sum_b M_1[S1[i1], b] U[b, i2] */
      for (int64_t i1 = 0; i1 < s1; ++i1)
        for (int64_t i2 = 0; i2 < s2; ++i2) {
          double sr = 0.0, si = 0.0;
          for (int64_t b = 0; b < n1; ++b) {
            double mr = R1[2 * (i1 * n1 + b)], mi = R1[2 * (i1 * n1 + b) + 1];
            double ur = U[2 * (b * s2 + i2)], ui = U[2 * (b * s2 + i2) + 1];
            sr += mr * ur - mi * ui;
            si += mr * ui + mi * ur;
          }
          T[2 * ((p * s1 + i1) * s2 + i2)] = sr;
          T[2 * ((p * s1 + i1) * s2 + i2) + 1] = si;
        }
    }
    free(U);
  }
  /* acc[i0, i1, i2] += sum_p M_0[S0[i0], plane_begin+p] T[p, i1, i2] */
  for (int64_t i0 = 0; i0 < s0; ++i0)
    for (int64_t p = 0; p < planes; ++p) {
      double mr, mi;
      matrix_entry(n0, S0[i0], plane_begin + p, sign, nodes0, nodes_on_output, &mr, &mi);
      mr *= c0;
      mi *= c0;
      const double* t = T + 2 * (p * s1 * s2);
      double* a = acc + 2 * (i0 * s1 * s2);
      for (int64_t q = 0; q < s1 * s2; ++q) {
        a[2 * q] += mr * t[2 * q] - mi * t[2 * q + 1];
        a[2 * q + 1] += mr * t[2 * q + 1] + mi * t[2 * q];
      }
    }
  free(R2);
  free(R1);
  free(T);
  return 0;
}
