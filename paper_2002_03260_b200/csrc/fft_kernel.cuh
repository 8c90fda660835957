// FFT formulation (paper Section III-B, Eq. 14-18): placeholder interface; the fused kernel follows.
#pragma once
#include <cstdio>
#include <cuda_runtime.h>

namespace dft3d {

struct FftAxis {
  long long n = 0;
  int N1 = 0, N2 = 0;
};

inline int fft_set_kernel_attributes() { return 0; }

inline int fft_build_axis(FftAxis*, long long, int, bool, int, int, char* err, size_t errlen) {
  snprintf(err, errlen, "the FFT formulation is not built yet");
  return 2;  // DFT3D_ERR_UNSUPPORTED
}

inline int fft_axis_pass(const FftAxis*, int, const long long*, const float*, float*, unsigned int*, int, cudaStream_t,
                         char* err, size_t errlen) {
  snprintf(err, errlen, "the FFT formulation is not built yet");
  return 2;
}

inline void fft_free_axis(FftAxis*) {}

}  // namespace dft3d
