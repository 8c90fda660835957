// The second launch of an 8192-point axis in the FFT formulation (paper Eq. 17 with N = 8192, N1 = 1024, N2 = 8).
//
// With n = 8*l + beta and k = k1 + 1024*k2:
//     X[k1 + 1024*k2] = sum_{beta<8} W8^(beta*k2) * T[k1, beta] * B[k1, beta],   T[k1, beta] = exp(s*2*pi*i*k1*beta/8192),
//     B[k1, beta]     = sum_{l<1024} W1024^(l*k1) * x[8*l + beta].
// B is what the fused 1024-point kernel (itself 32 x 32: GEMM, twiddle, GEMM) leaves when it runs over the view
// [lines][l = 1024][columns = 8 * C] of the data, the eight interleaved sub-sequences being eight times as many
// neighbouring columns; it arrives here in the natural order [line][k1][beta][c].  This kernel applies the phase
// adjustment T and the 8-point DFT over beta on the CUDA cores (fp32: three levels of additions and four multiplications
// by sqrt(1/2), like the radix-2 and radix-4 steps of the fused kernel) and stores X in natural order, i.e. transposed
// in (k1, k2): out[line][k2][k1][c].  16 bytes of HBM traffic per point.
//
// A thread owns one (line, k1, c): it reads its eight B values (C complex apart; for the last axis, C = 1, they are 64
// contiguous bytes) and its row of T (64 bytes), and writes eight values 1024*C complex apart; neighbouring threads
// are neighbouring c (or k1 when C = 1), so both sides are coalesced.
#pragma once
#include <cuda_runtime.h>

namespace dft3d {

constexpr int kRadix8Threads = 256;

struct Radix8Params {
  const float2* in;       // [lines][1024][8][C]
  float2* out;            // [lines][8][1024][C]
  const float2* tw;       // [1024][8] complex64: T[k1][beta], times 1/8 for a scaled inverse
  long long lines;        // product of the dimensions before the axis
  long long C;            // columns behind the axis (1 for the last axis)
  float sign;             // s of the exponent: -1 forward, +1 inverse
};

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
  return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x);
}
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
// a * (s*i)
__device__ __forceinline__ float2 cmul_si(float2 a, float s) { return make_float2(-s * a.y, s * a.x); }

__global__ void __launch_bounds__(kRadix8Threads)
fft_radix8_kernel(const Radix8Params p) {
  const long long total = p.lines * 1024 * p.C;
  const float s = p.sign;
  const float h = 0.70710678118654752440f;
  for (long long idx = blockIdx.x * (long long)kRadix8Threads + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * kRadix8Threads) {
    const long long c = idx % p.C;
    const long long k1 = (idx / p.C) % 1024;
    const long long line = idx / (p.C * 1024);
    float2 z[8];
    const float2* src = p.in + ((line * 1024 + k1) * 8) * p.C + c;
    const float4* trow = reinterpret_cast<const float4*>(p.tw + k1 * 8);
    float2 t[8];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const float4 v = __ldg(trow + b);
      t[2 * b] = make_float2(v.x, v.y);
      t[2 * b + 1] = make_float2(v.z, v.w);
    }
    if (p.C == 1) {
      const float4* s4 = reinterpret_cast<const float4*>(src);     // 64 contiguous, 64-byte aligned bytes
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const float4 v = __ldcs(s4 + b);
        z[2 * b] = make_float2(v.x, v.y);
        z[2 * b + 1] = make_float2(v.z, v.w);
      }
    } else {
#pragma unroll
      for (int b = 0; b < 8; ++b) z[b] = __ldcs(src + b * p.C);
    }
#pragma unroll
    for (int b = 0; b < 8; ++b) z[b] = cmul(z[b], t[b]);
    // 8-point DFT with w = exp(s*2*pi*i/8): X[k2] = sum_beta z[beta] * w^(beta*k2), decimation in time
    const float2 e0 = cadd(z[0], z[4]), e1 = csub(z[0], z[4]);          // even part: z0, z2, z4, z6
    const float2 e2 = cadd(z[2], z[6]), e3 = cmul_si(csub(z[2], z[6]), s);
    const float2 E0 = cadd(e0, e2), E2 = csub(e0, e2), E1 = cadd(e1, e3), E3 = csub(e1, e3);
    const float2 o0 = cadd(z[1], z[5]), o1 = csub(z[1], z[5]);          // odd part: z1, z3, z5, z7
    const float2 o2 = cadd(z[3], z[7]), o3 = cmul_si(csub(z[3], z[7]), s);
    const float2 O0 = cadd(o0, o2), O2 = csub(o0, o2), O1 = cadd(o1, o3), O3 = csub(o1, o3);
    // w^k2 * O[k2]: w = (1 + s*i)/sqrt(2), w^2 = s*i, w^3 = (-1 + s*i)/sqrt(2)
    const float2 w1 = make_float2(h * (O1.x - s * O1.y), h * (O1.y + s * O1.x));
    const float2 w2 = cmul_si(O2, s);
    const float2 w3 = make_float2(h * (-O3.x - s * O3.y), h * (-O3.y + s * O3.x));
    float2 X[8];
    X[0] = cadd(E0, O0); X[4] = csub(E0, O0);
    X[1] = cadd(E1, w1); X[5] = csub(E1, w1);
    X[2] = cadd(E2, w2); X[6] = csub(E2, w2);
    X[3] = cadd(E3, w3); X[7] = csub(E3, w3);
    float2* dst = p.out + ((line * 8) * 1024 + k1) * p.C + c;
#pragma unroll
    for (int k2 = 0; k2 < 8; ++k2) __stcs(dst + (long long)k2 * 1024 * p.C, X[k2]);
  }
}

}  // namespace dft3d
