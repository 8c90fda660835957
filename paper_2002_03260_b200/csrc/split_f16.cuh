// Packed fp32 arithmetic and the fp16 two-piece split, shared by the KDFT and FFT kernels with fp16 pieces.
#pragma once

#include <cstdint>
#include <cuda_fp16.h>

namespace dft3d {

// Two fp32 values in one 64-bit register for the packed fp32 instructions of sm_100 (one issue slot for two results).
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

// (re, im) -> packed fp16 pairs: hi = the value rounded to fp16, lo = the exact remainder x - hi rounded to fp16.
__device__ __forceinline__ void split_half2(uint64_t x, uint32_t& hi, uint32_t& lo) {
  float re, im, lr, li;
  unpack2(x, re, im);
  const __half2 h = __floats2half2_rn(re, im);
  const float2 hf = __half22float2(h);
  unpack2(sub2(x, pack2(hf.x, hf.y)), lr, li);
  const __half2 l = __floats2half2_rn(lr, li);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// the same from two registers that hold float bit patterns (data as it comes out of shared memory)
__device__ __forceinline__ uint64_t pack2_bits(uint32_t a, uint32_t b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(a), "r"(b));
  return r;
}

}  // namespace dft3d
