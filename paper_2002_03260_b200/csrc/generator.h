// Host-side table generator: DFT / Vandermonde matrices and twiddles evaluated in float64 with
// exactly reduced phases, then rounded once to the float32 pieces the kernels consume.
#pragma once
#include <cstdint>
#include <vector>

namespace dft3d {
namespace gen {

// exp(sign*2*pi*i*num/den) for integers 0 <= num < den, exact at multiples of an eighth turn
void root_of_unity(int64_t num, int64_t den, int sign, double* re, double* im);

// M[k][j] (interleaved complex, n*n entries) of one axis, times `scale`.
//   nodes == nullptr : exp(sign*2*pi*i*k*j/n)                       (Eq. 14)
//   nodes, default   : exp(sign*2*pi*i*k*nodes[j])                  (Eq. 3, unit-circle points, nonuniform input)
//   nodes, on output : exp(sign*2*pi*i*nodes[k]*j)                  (Eq. 1 read literally)
void axis_matrix(int64_t n, int sign, double scale, const double* nodes, bool nodes_on_output, double* M);

// In-place inverse of a complex n x n matrix (interleaved, row-major) by Gauss-Jordan elimination with partial
// pivoting in float64, rows shared among up to 16 host threads.  This is the inverse nonuniform transform of
// Section III-A: for sample points that are not the roots of unity the matrix of Eq. 3 is not unitary and the inverse
// "amounts to solving the linear system"; with the inverse as a table the solve is one more matrix product per axis.
// Returns false if a pivot vanishes (the nodes are not distinct modulo 1); *growth receives max|inverse entry| *
// max|matrix entry|, a cheap indication of how much accuracy the solve costs.
bool invert_matrix(int64_t n, double* M, double* growth);

// T[k1][beta] = exp(sign*2*pi*i*k1*beta/(N1*N2))  (phase adjustment of Eq. 17), N1*N2 complex entries
void twiddle(int64_t N1, int64_t N2, int sign, double* T);

// nearest value with an 11-bit significand (TF32), returned as float (low 13 mantissa bits zero)
float round_to_tf32(double v);

// nearest fp16 value (11-bit significand down to 2^-14, multiples of 2^-24 below; no overflow handling: |v| < 65504)
double round_to_fp16(double v);

// v ~= hi + lo with both pieces TF32-exact
inline void split_tf32(double v, float* hi, float* lo) {
  *hi = round_to_tf32(v);
  *lo = round_to_tf32(v - static_cast<double>(*hi));
}

// Real 2n x 2n form of a complex n x n matrix M (interleaved), split in two TF32 pieces:
//   W[2k][2j] = Re, W[2k][2j+1] = -Im, W[2k+1][2j] = Im, W[2k+1][2j+1] = Re.
void real_table_from_matrix(int64_t n, const double* M, float* hi, float* lo);

}  // namespace gen
}  // namespace dft3d
