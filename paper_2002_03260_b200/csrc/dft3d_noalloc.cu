// dft3d_kdft_execute_static: the KDFT transform for callers that must not allocate.
//
// Some callers cannot call cudaMalloc at the point where they need a transform: code running inside a
// memory-pool or real-time section where the allocator is off limits, a plugin whose host owns all device
// memory and forbids side allocations, or a process that has already handed every free byte to its own arena
// (an allocation there would fail or, worse, synchronise the whole device).  dft3d_plan_create allocates tables,
// a workspace and a status word; this entry point allocates nothing.  The caller passes the input, the output
// and the three per-axis tables (which it generated with dft3d_generate_real_table and copied into memory it
// owns); the one thing the transform still needs, the scratch cube between the axis passes, lives in a
// file-scope device array of fixed size.
#include <cstdarg>
#include <cstdio>
#include <cstring>

#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/dft3d.h"
#include "kdft_kernel.cuh"

namespace {

constexpr long long kStaticMaxPoints = 1ll << 21;                       // 2,097,152 complex points = 16 MiB
constexpr size_t kStaticHeaderBytes = 256;                              // status word, padded
constexpr size_t kStaticScratchBytes = kStaticHeaderBytes + size_t(kStaticMaxPoints) * 8;
constexpr int kMaxDevices = 64;

// Every GPU that loads the library holds these 16 MiB (+256 B) until the process exits.  In host code this
// name is only a handle: the device address is fetched with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_static_scratch on this device
  int sm_count = 0;
};
DeviceSetup g_setup[kMaxDevices];

thread_local char g_error[384] = "";

int fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof(g_error), fmt, ap);
  va_end(ap);
  return status;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int encode(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
           const cuuint32_t* box, bool swizzle128) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess || !fn)
      return fail(DFT3D_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    enc = reinterpret_cast<EncodeTiledFn>(fn);
  }
  const cuuint32_t es[3] = {1, 1, 1};
  CUresult cr = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, rank, const_cast<void*>(base), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return cr == CUDA_SUCCESS ? DFT3D_OK : fail(DFT3D_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", int(cr));
}

// once per device, with that device current: resolve the scratch array's device address
int setup_device(int dev, DeviceSetup** out) {
  if (dev < 0 || dev >= kMaxDevices) return fail(DFT3D_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
  DeviceSetup& s = g_setup[dev];
  if (!s.ready) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr)
      return fail(DFT3D_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10)
      return fail(DFT3D_ERR_UNSUPPORTED, "device %d is not sm_100", dev);
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return fail(DFT3D_ERR_CUDA, "cannot query the SM count");
    e = cudaFuncSetAttribute(dft3d::kdft_axis_kernel<dft3d::KDFT_CONTIG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             int(dft3d::kKdftSmemBytes));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(dft3d::kdft_axis_kernel<dft3d::KDFT_STRIDED>,
                               cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::kKdftSmemBytes));
    if (e != cudaSuccess) return fail(DFT3D_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    s.scratch = static_cast<unsigned char*>(ptr);
    s.ready = true;
  }
  *out = &s;
  return DFT3D_OK;
}

int launch_axis(const DeviceSetup& s, int axis, long long n0, long long n1, long long n2, const float* w,
                const float* in, float* out, unsigned int* status, cudaStream_t stream) {
  const long long nn[3] = {n0, n1, n2};
  const long long J = nn[axis];
  dft3d::KdftParams kp;
  memset(&kp, 0, sizeof(kp));
  kp.k2 = int(2 * J);
  kp.bn = int(2 * J < 256 ? 2 * J : 256);
  kp.n_tiles = (kp.k2 + kp.bn - 1) / kp.bn;
  kp.chunk_kb = 4;
  kp.out = out;
  kp.status = status;
  kp.profile = nullptr;
  CUtensorMap map_w, map_data;
  const cuuint64_t wd[3] = {cuuint64_t(2 * J), cuuint64_t(2 * J), 2};
  const cuuint64_t ws[2] = {cuuint64_t(2 * J * 4), cuuint64_t(4 * J * J * 4)};
  const cuuint32_t wb[3] = {cuuint32_t(dft3d::kBlockK), cuuint32_t(kp.bn), 2};
  int rc = encode(&map_w, w, 3, wd, ws, wb, true);
  if (rc != DFT3D_OK) return rc;
  if (axis == 2) {
    kp.rows = n0 * n1;
    kp.m_tiles = (kp.rows + dft3d::kTileM - 1) / dft3d::kTileM;
    kp.lpb = 128; kp.bpt = 1; kp.c_tiles = 1;
    const cuuint64_t dd[2] = {cuuint64_t(2 * J), cuuint64_t(kp.rows)};
    const cuuint64_t ds[1] = {cuuint64_t(J * 8)};
    const cuuint32_t db[2] = {cuuint32_t(dft3d::kBlockK), cuuint32_t(dft3d::kTileM)};
    if ((rc = encode(&map_data, in, 2, dd, ds, db, true)) != DFT3D_OK) return rc;
  } else {
    const long long batches = axis == 0 ? 1 : n0;
    const long long C = axis == 0 ? n1 * n2 : n2;
    kp.batches = batches;
    kp.C = C;
    kp.lpb = int(C < 128 ? C : 128);
    kp.bpt = 128 / kp.lpb;
    kp.c_tiles = (C + kp.lpb - 1) / kp.lpb;
    kp.m_tiles = kp.c_tiles * ((batches + kp.bpt - 1) / kp.bpt);
    const cuuint64_t dd[3] = {cuuint64_t(2 * C), cuuint64_t(J), cuuint64_t(batches)};
    const cuuint64_t ds[2] = {cuuint64_t(C * 8), cuuint64_t(J * C * 8)};
    const cuuint32_t db[3] = {cuuint32_t(2 * kp.lpb), cuuint32_t(dft3d::kBlockK / 2), cuuint32_t(kp.bpt)};
    if ((rc = encode(&map_data, in, 3, dd, ds, db, false)) != DFT3D_OK) return rc;
  }
  const long long total = kp.m_tiles * kp.n_tiles;
  const int grid = int(total < s.sm_count ? total : s.sm_count);
  if (axis == 2)
    dft3d::kdft_axis_kernel<dft3d::KDFT_CONTIG><<<grid, dft3d::kKdftThreads, dft3d::kKdftSmemBytes, stream>>>(map_data, map_w, kp);
  else
    dft3d::kdft_axis_kernel<dft3d::KDFT_STRIDED><<<grid, dft3d::kKdftThreads, dft3d::kKdftSmemBytes, stream>>>(map_data, map_w, kp);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DFT3D_OK : fail(DFT3D_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
}

}  // namespace

extern "C" int dft3d_kdft_execute_static(long long n0, long long n1, long long n2, const float* w0, const float* w1,
                                          const float* w2, const void* in, void* out, void* cuda_stream,
                                          char* error_message, size_t error_message_size) {
  int rc = DFT3D_OK;
  g_error[0] = 0;
  do {
    if (n0 < 1 || n1 < 1 || n2 < 1) { rc = fail(DFT3D_ERR_INVALID_ARG, "sizes must be >= 1"); break; }
    if (!w0 || !w1 || !w2 || !in || !out) { rc = fail(DFT3D_ERR_INVALID_ARG, "NULL pointer argument"); break; }
    if ((n0 % 64) || (n1 % 64) || (n2 % 64)) { rc = fail(DFT3D_ERR_UNSUPPORTED, "every size must be a multiple of 64"); break; }
    // bound every factor before forming the product (which could otherwise wrap around)
    if (n0 > kStaticMaxPoints || n1 > kStaticMaxPoints || n2 > kStaticMaxPoints) {
      rc = fail(DFT3D_ERR_UNSUPPORTED, "%lld x %lld x %lld points exceed the static scratch of %lld points (16 MiB); use "
                "dft3d_plan_create for larger transforms", n0, n1, n2, kStaticMaxPoints);
      break;
    }
    const long long P = n0 * n1 * n2;
    if (P > kStaticMaxPoints) {
      rc = fail(DFT3D_ERR_UNSUPPORTED, "%lld x %lld x %lld = %lld points exceed the static scratch of %lld points "
                "(16 MiB); use dft3d_plan_create for larger transforms", n0, n1, n2, P, kStaticMaxPoints);
      break;
    }
    const uintptr_t a = reinterpret_cast<uintptr_t>(in), b = reinterpret_cast<uintptr_t>(out);
    if ((a & 15) || (b & 15) || ((reinterpret_cast<uintptr_t>(w0) | reinterpret_cast<uintptr_t>(w1) |
                                  reinterpret_cast<uintptr_t>(w2)) & 15)) {
      rc = fail(DFT3D_ERR_INVALID_ARG, "pointers must be 16-byte aligned"); break;
    }
    if (a < b + size_t(P) * 8 && b < a + size_t(P) * 8) { rc = fail(DFT3D_ERR_INVALID_ARG, "in and out overlap"); break; }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { rc = fail(DFT3D_ERR_CUDA, "no current CUDA device"); break; }
    DeviceSetup* s = nullptr;
    if ((rc = setup_device(dev, &s)) != DFT3D_OK) break;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned int* status = reinterpret_cast<unsigned int*>(s->scratch);
    float* scratch = reinterpret_cast<float*>(s->scratch + kStaticHeaderBytes);
    // the array keeps whatever the last call left: the status word must start at zero
    if (cudaMemsetAsync(status, 0, sizeof(unsigned int), stream) != cudaSuccess) { rc = fail(DFT3D_ERR_CUDA, "cudaMemsetAsync"); break; }
    const float* fin = static_cast<const float*>(in);
    float* fout = static_cast<float*>(out);
    if ((rc = launch_axis(*s, 0, n0, n1, n2, w0, fin, fout, status, stream)) != DFT3D_OK) break;
    if ((rc = launch_axis(*s, 1, n0, n1, n2, w1, fout, scratch, status, stream)) != DFT3D_OK) break;
    if ((rc = launch_axis(*s, 2, n0, n1, n2, w2, scratch, fout, status, stream)) != DFT3D_OK) break;
    unsigned int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, status, sizeof(word), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) { rc = fail(DFT3D_ERR_CUDA, "waiting for the transform: %s", cudaGetErrorString(e)); break; }
    if (word != 0) rc = fail(DFT3D_ERR_DEVICE_TIMEOUT, "a kernel abandoned a bounded wait (code 0x%x)", word);
  } while (0);
  if (error_message && error_message_size) {
    strncpy(error_message, g_error, error_message_size - 1);
    error_message[error_message_size - 1] = 0;
  }
  return rc;
}
