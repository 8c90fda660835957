// C-ABI of the dft3d library: plans, the float64 table generator entry points, and the launch
// logic for the per-axis tensor-core kernels.  See include/dft3d.h for the contract of each call.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <tuple>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/dft3d.h"
#include "generator.h"
#include "kdft_kernel.cuh"
#include "kdft_f16_kernel.cuh"
#include "fft_f16_kernel.cuh"
#include "kdft_f16x2_kernel.cuh"
#include "fft_kernel.cuh"
#include "radix8_kernel.cuh"

namespace {

thread_local char g_last_error[512] = "";

int fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
  va_end(ap);
  return status;
}

#define DFT3D_CUDA(call)                                                                          \
  do {                                                                                            \
    cudaError_t e_ = (call);                                                                      \
    if (e_ != cudaSuccess)                                                                        \
      return fail(e_ == cudaErrorMemoryAllocation ? DFT3D_ERR_ALLOC : DFT3D_ERR_CUDA, "%s: %s", #call, \
                  cudaGetErrorString(e_));                                                        \
  } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is fetched through the runtime so that the library has no link-time
// dependency on libcuda and can be loaded (for its host-only entry points) on a machine without a GPU.
int get_encoder(EncodeTiledFn* fn) {
  static std::once_flag once;
  static EncodeTiledFn cached = nullptr;
  static cudaError_t err = cudaSuccess;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr);
    if (err == cudaSuccess && p && qr == cudaDriverEntryPointSuccess) cached = reinterpret_cast<EncodeTiledFn>(p);
  });
  if (!cached) return fail(DFT3D_ERR_CUDA, "cuTensorMapEncodeTiled is not available: %s", cudaGetErrorString(err));
  *fn = cached;
  return DFT3D_OK;
}

// Tuning knobs.  Environment variables are read ONCE, when a plan is created, and the values live in the plan:
// nothing a later dft3d_execute does depends on the environment.  -1 = not set (the measured default applies).
struct Knobs {
  int promo_narrow = -1, promo_pair = -1, promo_blocked = -1;   // L2 promotion of tensor maps (0/64/128/256 bytes)
  int fft_cols[2] = {-1, -1};                                   // lines per strided FFT stage, axis 0 / axis 1
  int fft_no_pair = 0, fft_pair = -1;                           // blocked order: rows per 128-byte line
  int fft_stage_out = -1, fft_stage_out_blocked = -1;           // results leave through the raw stage + TMA stores
  int fft_l2_prefetch = -1, fft_nb2 = -1;
  int fft_inplace = 0, fft_no_half = 0, fft_slices = 0;
  int fft_fuse = -1;                                            // axes 1 and 2 in one launch through an L2-resident ring
  int fft_fuse_ring = -1, fft_fuse_writers = -1, fft_fuse_hints = -1;   // its ring length (planes), writer CTAs, L2 hints
  int kdft_pair = -1, chunk_kb = -1, kdft_ngroup = -1;
  long long wait_limit = 0;                                     // clock budget of the kernels' bounded waits (0 = default)
  int test_silent_producer = 0;                                 // test of the give-up path: TMA producers issue nothing
};

int env_int(const char* name, int unset) {
  const char* v = getenv(name);
  return v ? atoi(v) : unset;
}

Knobs read_knobs() {
  Knobs k;
  k.promo_narrow = env_int("DFT3D_TMA_PROMO_NARROW", -1);
  k.promo_pair = env_int("DFT3D_TMA_PROMO_PAIR", -1);
  k.promo_blocked = env_int("DFT3D_TMA_PROMO_BLOCKED", -1);
  const int cols = env_int("DFT3D_FFT_COLS", -1);
  k.fft_cols[0] = env_int("DFT3D_FFT_COLS0", cols);
  k.fft_cols[1] = env_int("DFT3D_FFT_COLS1", cols);
  k.fft_no_pair = getenv("DFT3D_FFT_NO_PAIR") ? 1 : 0;
  k.fft_pair = env_int("DFT3D_FFT_PAIR", -1);
  k.fft_stage_out = env_int("DFT3D_FFT_STAGE_OUT", -1);
  k.fft_stage_out_blocked = env_int("DFT3D_FFT_STAGE_OUT_BLOCKED", -1);
  k.fft_l2_prefetch = env_int("DFT3D_FFT_L2_PREFETCH", -1);
  k.fft_nb2 = env_int("DFT3D_FFT_NB2", -1);
  k.fft_inplace = getenv("DFT3D_FFT_INPLACE") ? 1 : 0;
  k.fft_no_half = getenv("DFT3D_FFT_NO_HALF") ? 1 : 0;
  k.fft_slices = env_int("DFT3D_FFT_SLICES", 0);
  k.fft_fuse = env_int("DFT3D_FFT_FUSE", -1);
  k.fft_fuse_ring = env_int("DFT3D_FFT_FUSE_RING", -1);
  k.fft_fuse_writers = env_int("DFT3D_FFT_FUSE_WRITERS", -1);
  k.fft_fuse_hints = env_int("DFT3D_FFT_FUSE_HINTS", -1);
  k.kdft_pair = env_int("DFT3D_KDFT_PAIR", -1);
  k.chunk_kb = env_int("DFT3D_CHUNK_KB", -1);
  k.kdft_ngroup = env_int("DFT3D_KDFT_NGROUP", -1);
  if (const char* v = getenv("DFT3D_WAIT_LIMIT_CLOCKS")) k.wait_limit = atoll(v);
  k.test_silent_producer = env_int("DFT3D_TEST_SILENT_PRODUCER", 0);
  return k;
}

// float32 tensor map with up to 4 dimensions; dims/box innermost first; strides in bytes for dims 1..rank-1
// promotion_bytes >= 0 fixes the L2 promotion; otherwise 256 bytes, or `narrow_promo` (if >= 0) for rows under 128 bytes
int encode_map(CUtensorMap* map, CUtensorMapDataType dtype, const void* base, int rank,
               const unsigned long long* dims, const unsigned long long* strides_bytes, const unsigned* box,
               int swizzle_bytes, int promotion_bytes = -1, int narrow_promo = -1);

int encode_f32(CUtensorMap* map, const void* base, int rank, const unsigned long long* dims,
               const unsigned long long* strides_bytes, const unsigned* box, int swizzle_bytes, int promotion_bytes = -1,
               int narrow_promo = -1) {
  return encode_map(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, base, rank, dims, strides_bytes, box, swizzle_bytes,
                    promotion_bytes, narrow_promo);
}

int encode_map(CUtensorMap* map, CUtensorMapDataType dtype, const void* base, int rank,
               const unsigned long long* dims, const unsigned long long* strides_bytes, const unsigned* box,
               int swizzle_bytes, int promotion_bytes, int narrow_promo) {
  EncodeTiledFn enc = nullptr;
  int rc = get_encoder(&enc);
  if (rc != DFT3D_OK) return rc;
  cuuint64_t d[5], s[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) s[i] = strides_bytes[i];
  // L2 promotion: what a miss fetches around the requested bytes.  Rows of 128 bytes and more: 256 bytes (the
  // neighbouring line belongs to the neighbouring stage, which runs at the same time).  Narrower rows: see below.
  const unsigned inner_bytes = box[0] * (dtype == CU_TENSOR_MAP_DATA_TYPE_FLOAT32 ? 4u : 2u);
  CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
  if (inner_bytes < 128 || promotion_bytes >= 0) {
    int v = narrow_promo >= 0 ? narrow_promo : 256;
    if (promotion_bytes >= 0) v = promotion_bytes;
    promo = v == 0 ? CU_TENSOR_MAP_L2_PROMOTION_NONE
                   : (v == 64 ? CU_TENSOR_MAP_L2_PROMOTION_L2_64B
                              : (v == 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B));
  }
  CUresult cr = enc(map, dtype, rank, const_cast<void*>(base), d, s, b, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                         : (swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE),
                    promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS)
    return fail(DFT3D_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d (rank %d, dims %llu %llu %llu, box %u %u %u)",
                int(cr), rank, dims[0], rank > 1 ? dims[1] : 0ull, rank > 2 ? dims[2] : 0ull, box[0],
                rank > 1 ? box[1] : 0u, rank > 2 ? box[2] : 0u);
  return DFT3D_OK;
}

struct KdftAxis {
  long long n = 0;
  float* d_w = nullptr;   // [2 pieces][2n][2n] floats (TF32 pieces), or halves holding 1024*W (fp16 pieces)
  CUtensorMap map_w;
  CUtensorMap map_w_pair; // fp16 pieces, paired CTAs: boxes of 128 table rows (half an N-tile)
  bool pair = false;      // the paired-CTA kernel applies (fp16 pieces, 2n >= 256)
  int bn = 0;
  float out_mul = 1.0f;   // fp16 pieces: 2^-10, times 1/n for a scaled inverse
};

struct FftAxis {
  long long n = 0;
  int R = 0, RX = 1;       // n = RX*R*R, RX = 1 or 2
  int cols = 16;           // lines per STRIDED stage
  float* d_w = nullptr;    // real form of F_R: [piece hi|lo][2R/32 panels][2R rows][32 floats]
  float2* d_tw = nullptr;  // T[k1][beta], R*R complex64
  float2* d_tw2 = nullptr; // RX == 2: exp(s*2*pi*i*m/n), m < R*R
  float out_mul = 1.0f;    // fp16 pieces: the factor the store applies (powers of two, 1/n for a scaled inverse)
  CUtensorMap map_w;
  // 8192-point axis = 1024 x 8 (Eq. 17 once more): the fused kernel transforms the eight stride-8 sub-sequences (n = 1024
  // above), a second launch applies the phase adjustment and the 8-point DFT (radix8_kernel.cuh)
  bool r8 = false;
  float2* d_tw8 = nullptr; // [1024][8] complex64, exp(s*2*pi*i*k1*beta/8192), times 1/8 for a scaled inverse
};

}  // namespace

struct dft3d_plan_s {
  long long n[3] = {0, 0, 0};
  int mode = 0, sign = 0;
  unsigned flags = 0;
  bool f16 = false;       // fp16 pieces (else TF32 pieces)
  bool in_is_ws = false;  // DFT3D_DESTROY_INPUT: the caller's input buffer serves as the workspace
  int ws_slices = 0;      // FFT, fp16 pieces: the workspace holds 1/ws_slices of a cube (2, 4 or 8); the strided passes run
                          // once per slice of axis 2; 0 = not this schedule
  int amode[3] = {0, 0, 0};  // DFT3D_AUTO with both formulations in one plan: the formulation of each axis
  unsigned axes = 7;            // bit a: axis a is transformed
  int device = 0;
  int sm_count = 0;
  KdftAxis kax[3];
  FftAxis fax[3];
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  long long group_planes = 0;   // n0-planes per workspace group (KDFT)
  int chunk_kb = 4;             // 32-real stages per tensor-core accumulation chain (KDFT)
  // FFT, axes 1 and 2 in one launch: a ring of n0-planes between them (meant to stay in L2) and per-plane counters
  bool fuse12 = false;
  int ring_planes = 0, fuse_writers = 0;
  void* ring = nullptr;
  unsigned int* d_fuse_counters = nullptr;   // [2][n0]: written, consumed
  unsigned int* d_status = nullptr;
  unsigned int* d_amax = nullptr;   // fp16 pieces: float bits of the largest magnitude before pass 0, 1, 2, (3)
  long long* d_profile = nullptr;   // wait-cycle counters, only allocated in DFT3D_PROFILE_WAITS builds
  void* host_in_dev = nullptr;  // device staging for dft3d_execute_host
  void* host_out_dev = nullptr;
  // dft3d_execute_host_batch: a second pair of staging buffers, two copy streams and the events that order them
  void* host_in_dev2 = nullptr;
  void* host_out_dev2 = nullptr;
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t ev_in_ready[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out_free[2] = {nullptr, nullptr};
  bool attrs_set = false;
  Knobs knobs;                  // environment knobs as they were when the plan was created
  // Tensor maps of the data operands, encoded once per (pass, base pointer, slice) and reused by later executes on the
  // same buffers (a plan serves one execute at a time, so no lock)
  typedef std::tuple<int, const void*, long long, long long> MapKey;
  std::map<MapKey, CUtensorMap> map_cache;
};

namespace {

long long points(const dft3d_plan_s* p) { return p->n[0] * p->n[1] * p->n[2]; }

// Looks up the tensor map of (tag, base, x0, x1) in the plan's cache; `make` encodes it on a miss.
template <class Make>
int cached_map(dft3d_plan_s* p, CUtensorMap* map, int tag, const void* base, long long x0, long long x1, Make&& make) {
  const dft3d_plan_s::MapKey key(tag, base, x0, x1);
  auto it = p->map_cache.find(key);
  if (it != p->map_cache.end()) { *map = it->second; return DFT3D_OK; }
  const int rc = make(map);
  if (rc != DFT3D_OK) return rc;
  if (p->map_cache.size() >= 8192) p->map_cache.clear();   // a caller that keeps changing buffers: start over
  try { p->map_cache.emplace(key, *map); } catch (const std::bad_alloc&) { /* uncached is still correct */ }
  return DFT3D_OK;
}

dft3d::WaitControl wait_control(const dft3d_plan_s* p) {
  dft3d::WaitControl wc;
  wc.limit_clocks = p->knobs.wait_limit;
  wc.silent_producer = p->knobs.test_silent_producer;
  return wc;
}

// the opt-in to large dynamic shared memory is a per-device property of each kernel
int set_kernel_attributes(int device) {
  static std::mutex mu;
  static bool done_on[64] = {false};
  std::lock_guard<std::mutex> lock(mu);
  bool& done = done_on[device & 63];
  if (done) return DFT3D_OK;
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::kdft_axis_kernel<dft3d::KDFT_CONTIG>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::kKdftSmemBytes)));
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::kdft_axis_kernel<dft3d::KDFT_STRIDED>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::kKdftSmemBytes)));
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::kdft_f16_axis_kernel<dft3d::KDFT_CONTIG>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::kKdftF16SmemBytes)));
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::kdft_f16_axis_kernel<dft3d::KDFT_STRIDED>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::kKdftF16SmemBytes)));
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::kdft_f16x2_axis_kernel<dft3d::KDFT_CONTIG>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::kKdftX2SmemBytes)));
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::kdft_f16x2_axis_kernel<dft3d::KDFT_STRIDED>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::kKdftX2SmemBytes)));
#define DFT3D_FFT_ATTR(MODE, R, RX, COLS, NB2, SO)                                                            \
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::fft_axis_kernel<MODE, R, RX, COLS, NB2, SO>,                          \
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::fft_smem_bytes(R, NB2))))
  DFT3D_FFT_ATTR(dft3d::FFT_CONTIG, 32, 1, 16, 2, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_CONTIG, 16, 1, 16, 2, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_CONTIG, 32, 2, 16, 2, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_CONTIG, 16, 2, 16, 2, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 1, 16, 1, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 1, 8, 2, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 16, 1, 16, 2, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 2, 8, 1, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 16, 2, 16, 2, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 1, 16, 1, 1);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 1, 8, 1, 0);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 1, 8, 1, 1);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 1, 8, 2, 1);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 16, 1, 16, 2, 1);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 32, 2, 8, 1, 1);
  DFT3D_FFT_ATTR(dft3d::FFT_STRIDED, 16, 2, 16, 2, 1);
#undef DFT3D_FFT_ATTR
#define DFT3D_FFT16_ATTR(MODE, R, RX, COLS, SO)                                                   \
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::fft_f16_axis_kernel<MODE, R, RX, COLS, SO>,              \
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, int(dft3d::fft16_smem_bytes(R, RX))))
  DFT3D_FFT16_ATTR(dft3d::FFT_CONTIG, 32, 1, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_CONTIG, 16, 1, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_CONTIG, 32, 2, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_CONTIG, 16, 2, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 1, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 1, 8, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 16, 1, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 2, 8, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 16, 2, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 1, 16, 1);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 1, 8, 1);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 16, 1, 16, 1);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 2, 8, 1);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 16, 2, 16, 1);
  DFT3D_FFT16_ATTR(dft3d::FFT_CONTIG, 32, 4, 16, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 4, 4, 0);
  DFT3D_FFT16_ATTR(dft3d::FFT_STRIDED, 32, 4, 4, 1);
#undef DFT3D_FFT16_ATTR
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::fft_f16_fused_kernel<32, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  int(dft3d::fft16_smem_bytes(32, 1))));
  DFT3D_CUDA(cudaFuncSetAttribute(dft3d::fft_f16_fused_kernel<16, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  int(dft3d::fft16_smem_bytes(16, 1))));
  done = true;
  return DFT3D_OK;
}

int build_kdft_axis(dft3d_plan_s* p, int a, const double* nodes) {
  KdftAxis& ax = p->kax[a];
  const long long n = p->n[a];
  ax.n = n;
  ax.bn = int(2 * n < 256 ? (2 * n + 15) / 16 * 16 : 256);   // MMA N: a multiple of 16, rows beyond 2n are zero-filled
  const bool scaled = (p->sign > 0) && !(p->flags & DFT3D_UNSCALED_INVERSE);
  const double scale = scaled ? 1.0 / double(n) : 1.0;
  std::vector<double> M;
  std::vector<float> W;
  try {
    M.resize(size_t(2) * n * n);
    if (!p->f16) W.resize(size_t(2) * 4 * n * n);
  } catch (const std::bad_alloc&) {
    return fail(DFT3D_ERR_ALLOC, "host allocation of the axis-%d table failed", a);
  }
  // DFT3D_INVERSE_SOLVE on an axis with nodes: the table is the inverse of the forward matrix of those nodes
  const bool solve = (p->flags & DFT3D_INVERSE_SOLVE) && nodes;
  if (solve) {
    dft3d::gen::axis_matrix(n, DFT3D_FORWARD, 1.0, nodes, (p->flags & DFT3D_NODES_ON_OUTPUT) != 0, M.data());
    double growth = 0.0;
    if (!dft3d::gen::invert_matrix(n, M.data(), &growth))
      return fail(DFT3D_ERR_INVALID_ARG, "axis %d: the matrix of these nodes is singular (nodes must be distinct modulo 1)", a);
    if (growth > 1e6)
      return fail(DFT3D_ERR_UNSUPPORTED, "axis %d: the nodes make the system too ill-conditioned for fp32 data "
                  "(|V| |V^-1| = %.3g)", a, growth);
  }
  if (p->f16) {
    // fp16 pieces of 2^s*W (s = 10 for entries of modulus one); the 1/n of a scaled inverse goes into the epilogue
    // multiplier instead of the table
    if (!solve) dft3d::gen::axis_matrix(n, p->sign, 1.0, nodes, (p->flags & DFT3D_NODES_ON_OUTPUT) != 0, M.data());
    int s2 = 10;
    if (solve) {
      double mx = 0.0;
      for (size_t i = 0; i < M.size(); ++i) mx = std::fmax(mx, std::fabs(M[i]));
      s2 = 9 - std::ilogb(mx);           // largest table entry in [512, 1024)
    }
    const double tscale = std::ldexp(1.0, s2);
    std::vector<__half> H;
    try {
      H.resize(size_t(2) * 4 * n * n);
    } catch (const std::bad_alloc&) {
      return fail(DFT3D_ERR_ALLOC, "host allocation of the axis-%d table failed", a);
    }
    const size_t piece = size_t(4) * n * n, ld = size_t(2) * n;
    for (long long k = 0; k < n; ++k)
      for (long long j = 0; j < n; ++j) {
        const double re = tscale * M[2 * (k * n + j)], im = tscale * M[2 * (k * n + j) + 1];
        const double vals[4] = {re, -im, im, re};                  // W[2k][2j], W[2k][2j+1], W[2k+1][2j], W[2k+1][2j+1]
        const size_t idx[4] = {(2 * k) * ld + 2 * j, (2 * k) * ld + 2 * j + 1, (2 * k + 1) * ld + 2 * j,
                               (2 * k + 1) * ld + 2 * j + 1};
        for (int q = 0; q < 4; ++q) {
          const double hi = dft3d::gen::round_to_fp16(vals[q]);
          const double lo = dft3d::gen::round_to_fp16(vals[q] - hi);
          H[idx[q]] = __float2half_rn(float(hi));                  // exact: already on the fp16 grid
          H[piece + idx[q]] = __float2half_rn(float(lo));
        }
      }
    ax.out_mul = float((solve ? 1.0 : scale) / tscale);
    DFT3D_CUDA(cudaMalloc(&ax.d_w, H.size() * sizeof(__half)));
    DFT3D_CUDA(cudaMemcpy(ax.d_w, H.data(), H.size() * sizeof(__half), cudaMemcpyHostToDevice));
    const unsigned long long hdims[3] = {(unsigned long long)(2 * n), (unsigned long long)(2 * n), 2ull};
    const unsigned long long hstrides[2] = {(unsigned long long)(2 * n * 2), (unsigned long long)(4 * n * n * 2)};
    const unsigned hbox[3] = {unsigned(dft3d::kF16BlockK), unsigned(ax.bn), 2u};
    {
      // pairs of CTAs (cta_group::2) share a 256-column table tile, each loading 128 of its rows
      const int env = p->knobs.kdft_pair;
      // Same bits as the one-CTA kernel.  Its MMAs run at full rate but every chain end waits for a cross-CTA round
      // trip, which cancels out at n = 1024 (77.6 vs 78.5 ms); at n = 2048, where the 64 MiB table no longer sits in
      // L2 beside the data and the part runs at its 1 kW cap, fetching every table tile once per CTA pair wins
      // (1365 -> 1235 ms, 1305 -> 1522 MHz).  Default: pairs from n = 2048 on.
      ax.pair = ax.bn == 256 && (p->sm_count % 2 == 0) && (env >= 0 ? env != 0 : n >= 2048);
      if (ax.pair) {
        const unsigned pbox[3] = {unsigned(dft3d::kF16BlockK), 128u, 2u};
        int rc = encode_map(&ax.map_w_pair, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, ax.d_w, 3, hdims, hstrides, pbox, 128);
        if (rc != DFT3D_OK) return rc;
      }
    }
    return encode_map(&ax.map_w, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, ax.d_w, 3, hdims, hstrides, hbox, 128);
  }
  if (!solve) dft3d::gen::axis_matrix(n, p->sign, scale, nodes, (p->flags & DFT3D_NODES_ON_OUTPUT) != 0, M.data());
  dft3d::gen::real_table_from_matrix(n, M.data(), W.data(), W.data() + size_t(4) * n * n);
  // TMA wants every row of the table to start on a 16-byte boundary: rows of 2n floats do when n is even; for odd n the
  // TABLE gets two columns of padding per row (never read: the tensor map's extent stays 2n), the data is left alone
  const long long ld = 2 * n + (n % 2 ? 2 : 0);
  if (ld != 2 * n) {
    std::vector<float> padded;
    try {
      padded.assign(size_t(2) * 2 * n * ld, 0.0f);
    } catch (const std::bad_alloc&) {
      return fail(DFT3D_ERR_ALLOC, "host allocation of the axis-%d table failed", a);
    }
    for (int pc = 0; pc < 2; ++pc)
      for (long long r = 0; r < 2 * n; ++r)
        memcpy(&padded[(size_t(pc) * 2 * n + r) * ld], &W[(size_t(pc) * 2 * n + r) * 2 * n], sizeof(float) * 2 * n);
    W.swap(padded);
  }
  DFT3D_CUDA(cudaMalloc(&ax.d_w, W.size() * sizeof(float)));
  DFT3D_CUDA(cudaMemcpy(ax.d_w, W.data(), W.size() * sizeof(float), cudaMemcpyHostToDevice));
  const unsigned long long dims[3] = {(unsigned long long)(2 * n), (unsigned long long)(2 * n), 2ull};
  const unsigned long long strides[2] = {(unsigned long long)(ld * 4), (unsigned long long)(2 * n * ld * 4)};
  const unsigned box[3] = {unsigned(dft3d::kBlockK), unsigned(ax.bn), 2u};
  return encode_f32(&ax.map_w, ax.d_w, 3, dims, strides, box, 128);
}

// One KDFT axis pass over a [batches][J][C] complex view (STRIDED) or rows x J (CONTIG).
template <class Params>
void fill_f16_params(Params& fp, const dft3d::KdftParams& kp, const KdftAxis& ax, dft3d_plan_s* p, int chain_pos) {
  fp.k2 = kp.k2; fp.bn = kp.bn; fp.n_tiles = kp.n_tiles; fp.chunk_kb = kp.chunk_kb;
  fp.m_tiles = kp.m_tiles; fp.rows = kp.rows; fp.batches = kp.batches; fp.C = kp.C;
  fp.lpb = kp.lpb; fp.bpt = kp.bpt; fp.c_tiles = kp.c_tiles;
  fp.out = kp.out; fp.status = kp.status; fp.profile = kp.profile;
  fp.out_mul = ax.out_mul;
  fp.amax_in = p->d_amax + chain_pos;
  fp.amax_out = p->d_amax + chain_pos + 1;
  fp.wc = kp.wc;
  // paired-CTA kernel: eight table panels live at a time once there are sixteen or more (measured: 8192 x 8192 26.9 -> 24.5 ms,
  // 64 x 4096 x 4096 214 -> 202 ms, 2048^3 unchanged; groups of 1, 2, 4, 16, 32 panels are slower)
  fp.n_group = p->knobs.kdft_ngroup >= 0 ? p->knobs.kdft_ngroup : ((kp.n_tiles >= 16 && ax.pair) ? 8 : 0);
}

// chain_pos: position of this pass in the sequence of passes of one execute (fp16 pieces: which amax word to read)
int launch_kdft_strided(dft3d_plan_s* p, int a, const float* in, float* out, long long batches, long long C,
                        cudaStream_t stream, int chain_pos) {
  const KdftAxis& ax = p->kax[a];
  const long long J = ax.n;
  dft3d::KdftParams kp;
  memset(&kp, 0, sizeof(kp));
  kp.k2 = int(2 * J);
  kp.bn = ax.bn;
  kp.n_tiles = int((2 * J + ax.bn - 1) / ax.bn);
  kp.chunk_kb = p->chunk_kb;
  kp.batches = batches;
  kp.C = C;
  kp.lpb = C <= 64 ? 64 : 128;   // lanes of one batch in a tile; columns beyond C are zero-filled and masked
  kp.bpt = 128 / kp.lpb;
  kp.c_tiles = (C + kp.lpb - 1) / kp.lpb;
  kp.m_tiles = kp.c_tiles * ((batches + kp.bpt - 1) / kp.bpt);
  kp.rows = 0;
  kp.out = out;
  kp.status = p->d_status;
  kp.profile = p->d_profile;
  kp.wc = wait_control(p);
  CUtensorMap map_data;
  const bool f16 = p->f16;
  int rc = cached_map(p, &map_data, 0x100 + a, in, batches, C, [&](CUtensorMap* m) {
    const unsigned long long dims[3] = {(unsigned long long)(2 * C), (unsigned long long)J, (unsigned long long)batches};
    const unsigned long long strides[2] = {(unsigned long long)(C * 8), (unsigned long long)(J * C * 8)};
    // rows j per box: a whole stage for the paired-CTA kernel (32), half a stage for the one-CTA fp16 kernel, a TF32 stage (16)
    const unsigned box[3] = {unsigned(2 * kp.lpb), unsigned((f16 && ax.pair) ? dft3d::kF16BlockK / 2 : 16), unsigned(kp.bpt)};
    return encode_f32(m, in, 3, dims, strides, box, 0, -1, p->knobs.promo_narrow);
  });
  if (rc != DFT3D_OK) return rc;
  const long long total = kp.m_tiles * kp.n_tiles;
  const int grid = int(total < p->sm_count ? total : p->sm_count);
  if (f16 && ax.pair) {
    dft3d::KdftF16Params fp;
    fill_f16_params(fp, kp, ax, p, chain_pos);
    const long long pairs = ((kp.m_tiles + 1) / 2) * kp.n_tiles;
    const int pgrid = 2 * int(pairs < p->sm_count / 2 ? pairs : p->sm_count / 2);
    dft3d::kdft_f16x2_axis_kernel<dft3d::KDFT_STRIDED>
        <<<pgrid, dft3d::kKdftThreads, dft3d::kKdftX2SmemBytes, stream>>>(map_data, ax.map_w_pair, fp);
  } else if (f16) {
    dft3d::KdftF16Params fp;
    fill_f16_params(fp, kp, ax, p, chain_pos);
    dft3d::kdft_f16_axis_kernel<dft3d::KDFT_STRIDED>
        <<<grid, dft3d::kKdftThreads, dft3d::kKdftF16SmemBytes, stream>>>(map_data, ax.map_w, fp);
  } else
  dft3d::kdft_axis_kernel<dft3d::KDFT_STRIDED>
      <<<grid, dft3d::kKdftThreads, dft3d::kKdftSmemBytes, stream>>>(map_data, ax.map_w, kp);
  DFT3D_CUDA(cudaGetLastError());
  return DFT3D_OK;
}

int launch_kdft_contig(dft3d_plan_s* p, int a, const float* in, float* out, long long rows, cudaStream_t stream,
                       int chain_pos) {
  const KdftAxis& ax = p->kax[a];
  const long long J = ax.n;
  dft3d::KdftParams kp;
  memset(&kp, 0, sizeof(kp));
  kp.k2 = int(2 * J);
  kp.bn = ax.bn;
  kp.n_tiles = int((2 * J + ax.bn - 1) / ax.bn);
  kp.chunk_kb = p->chunk_kb;
  kp.rows = rows;
  kp.m_tiles = (rows + dft3d::kTileM - 1) / dft3d::kTileM;
  kp.lpb = 128;
  kp.bpt = 1;
  kp.c_tiles = 1;
  kp.out = out;
  kp.status = p->d_status;
  kp.profile = p->d_profile;
  kp.wc = wait_control(p);
  CUtensorMap map_data;
  int rc = cached_map(p, &map_data, 0x110 + a, in, rows, 0, [&](CUtensorMap* m) {
    const unsigned long long dims[2] = {(unsigned long long)(2 * J), (unsigned long long)rows};
    const unsigned long long strides[1] = {(unsigned long long)(J * 8)};
    const unsigned box[2] = {unsigned(dft3d::kBlockK), unsigned(dft3d::kTileM)};
    return encode_f32(m, in, 2, dims, strides, box, 128);
  });
  if (rc != DFT3D_OK) return rc;
  const long long total = kp.m_tiles * kp.n_tiles;
  const int grid = int(total < p->sm_count ? total : p->sm_count);
  if (p->f16 && ax.pair) {
    dft3d::KdftF16Params fp;
    fill_f16_params(fp, kp, ax, p, chain_pos);
    const long long pairs = ((kp.m_tiles + 1) / 2) * kp.n_tiles;
    const int pgrid = 2 * int(pairs < p->sm_count / 2 ? pairs : p->sm_count / 2);
    dft3d::kdft_f16x2_axis_kernel<dft3d::KDFT_CONTIG>
        <<<pgrid, dft3d::kKdftThreads, dft3d::kKdftX2SmemBytes, stream>>>(map_data, ax.map_w_pair, fp);
  } else if (p->f16) {
    dft3d::KdftF16Params fp;
    fill_f16_params(fp, kp, ax, p, chain_pos);
    dft3d::kdft_f16_axis_kernel<dft3d::KDFT_CONTIG>
        <<<grid, dft3d::kKdftThreads, dft3d::kKdftF16SmemBytes, stream>>>(map_data, ax.map_w, fp);
  } else
  dft3d::kdft_axis_kernel<dft3d::KDFT_CONTIG>
      <<<grid, dft3d::kKdftThreads, dft3d::kKdftSmemBytes, stream>>>(map_data, ax.map_w, kp);
  DFT3D_CUDA(cudaGetLastError());
  return DFT3D_OK;
}

int kdft_axis_pass(dft3d_plan_s* p, int axis, const float* in, float* out, long long planes, cudaStream_t stream,
                   int chain_pos) {
  // `planes` n0-planes starting at in/out (axis 0 always takes the whole cube)
  const long long n1 = p->n[1], n2 = p->n[2];
  if (axis == 0) return launch_kdft_strided(p, 0, in, out, 1, n1 * n2, stream, chain_pos);
  if (axis == 1) return launch_kdft_strided(p, 1, in, out, planes, n2, stream, chain_pos);
  return launch_kdft_contig(p, 2, in, out, planes * n1, stream, chain_pos);
}

// fp16 pieces: before the first pass of an execute, clear the chain of amax words and measure the input
int prepare_scales(dft3d_plan_s* p, const float* in, cudaStream_t stream) {
  if (!p->f16) return DFT3D_OK;
  DFT3D_CUDA(cudaMemsetAsync(p->d_amax, 0, 4 * sizeof(unsigned int), stream));
  const long long n4 = points(p) / 2;      // float4 = two complex points; the point count is even
  dft3d::amax_kernel<<<p->sm_count * 8, 256, 0, stream>>>(reinterpret_cast<const float4*>(in), n4, p->d_amax);
  DFT3D_CUDA(cudaGetLastError());
  return DFT3D_OK;
}

// FFT formulation, one axis: n = RX*R*R with R = 16 or 32 and RX = 1 or 2 (Eq. 17 with P = R, preceded for
// RX = 2 by one more application with P = n/2, a radix-2 butterfly).  Tables: the real form of F_R split in TF32
// pieces and stacked [hi; lo], in the panel layout the kernel's TMA loads expect, and the twiddle factors rounded
// once to complex64.  The 1/n of a scaled inverse is 1/R in each stage's matrix and 1/RX in the twiddles.
int build_fft_axis(dft3d_plan_s* p, int a, const int split[2]) {
  FftAxis& ax = p->fax[a];
  long long n = p->n[a];
  const bool scaled = (p->sign > 0) && !(p->flags & DFT3D_UNSCALED_INVERSE);
  if (n == 8192 && p->f16) {
    // 8192 = 1024 * 8: tables of the 1024-point kernel, and the phase adjustment between the two steps
    if ((split[0] || split[1]) && (split[0] != 1024 || split[1] != 8))
      return fail(DFT3D_ERR_UNSUPPORTED, "FFT split %dx%d for n%d = 8192 is not supported (only 1024x8)", split[0], split[1], a);
    ax.r8 = true;
    n = 1024;
    std::vector<double> T(size_t(2) * 1024 * 8);
    std::vector<float> t8(T.size());
    dft3d::gen::twiddle(1024, 8, p->sign, T.data());
    for (size_t i = 0; i < T.size(); ++i) t8[i] = float(T[i] * (scaled ? 0.125 : 1.0));
    DFT3D_CUDA(cudaMalloc(&ax.d_tw8, t8.size() * sizeof(float)));
    DFT3D_CUDA(cudaMemcpy(ax.d_tw8, t8.data(), t8.size() * sizeof(float), cudaMemcpyHostToDevice));
  }
  int R = 0, RX = 1;
  if (n == 256) { R = 16; }
  if (n == 512) { R = 16; RX = 2; }
  if (n == 1024) { R = 32; }
  if (n == 2048) { R = 32; RX = 2; }
  if (n == 4096 && p->f16) { R = 32; RX = 4; }   // three factors: 4 * 32 * 32 (fp16-piece kernel only)
  if (!R)
    return fail(DFT3D_ERR_UNSUPPORTED, "FFT mode supports axis lengths 256, 512, 1024, 2048 and (fp16 pieces) 4096 and 8192; "
                "n%d = %lld", a, n);
  if (!ax.r8 && (split[0] || split[1]) && (split[0] != RX * R || split[1] != R))
    return fail(DFT3D_ERR_UNSUPPORTED, "FFT split %dx%d for n%d = %lld is not supported (only %dx%d)", split[0],
                split[1], a, n, RX * R, R);
  ax.n = n;
  ax.R = R;
  ax.RX = RX;
  ax.cols = (R == 32 && RX == 4) ? 4 : ((R == 32 && RX == 2) ? 8 : 16);   // a 128 KB stage holds all n rows of `cols` lines
                                                                           // (fft_axis_pass may pick 8 for R = 32, RX = 1)
  const int K = 2 * R, NB = 2 * R, panels = K / 32;
  if (p->f16) {
    // fp16 pieces: 1024 * F_R (real form), rows of 64 halves (zero-padded for R = 16), [hi piece; lo piece]; the twiddle
    // factors carry 2^-(10 + log2(R) - 1); everything else (1/n of a scaled inverse included) is one factor at the store
    const int sh = (R == 32 ? 5 : 4) - 1;
    std::vector<double> M(size_t(2) * R * R), T(size_t(2) * R * R);
    std::vector<__half> W(size_t(2) * NB * 64, __float2half(0.0f));
    std::vector<float> tw(size_t(2) * R * R);
    dft3d::gen::axis_matrix(R, p->sign, 1024.0, nullptr, false, M.data());
    for (int k = 0; k < R; ++k)
      for (int j = 0; j < R; ++j) {
        const double re = M[2 * (size_t(k) * R + j)], im = M[2 * (size_t(k) * R + j) + 1];
        const double v[2][2] = {{re, -im}, {im, re}};
        for (int pp = 0; pp < 2; ++pp)
          for (int q = 0; q < 2; ++q) {
            const double hi = dft3d::gen::round_to_fp16(v[pp][q]);
            const double lo = dft3d::gen::round_to_fp16(v[pp][q] - hi);
            const size_t at = size_t(2 * k + pp) * 64 + (2 * j + q);
            W[at] = __float2half(float(hi));
            W[size_t(NB) * 64 + at] = __float2half(float(lo));
          }
      }
    dft3d::gen::twiddle(R, R, p->sign, T.data());
    const double tscale = std::ldexp(1.0, -(10 + sh));
    for (size_t i = 0; i < T.size(); ++i) tw[i] = float(T[i] * tscale);
    ax.out_mul = float(std::ldexp(1.0, sh - 10) * (scaled ? 1.0 / double(n) : 1.0));
    DFT3D_CUDA(cudaMalloc(&ax.d_w, W.size() * sizeof(__half)));
    DFT3D_CUDA(cudaMemcpy(ax.d_w, W.data(), W.size() * sizeof(__half), cudaMemcpyHostToDevice));
    DFT3D_CUDA(cudaMalloc(&ax.d_tw, tw.size() * sizeof(float)));
    DFT3D_CUDA(cudaMemcpy(ax.d_tw, tw.data(), tw.size() * sizeof(float), cudaMemcpyHostToDevice));
    if (RX >= 2) {
      // exp(s*2*pi*i*b*m/n) for b = 1 .. RX-1, m < R*R: the twiddles between the radix-RX step and the R*R-point parts
      std::vector<float> tw2(size_t(2) * (RX - 1) * R * R);
      for (int b = 1; b < RX; ++b)
        for (long long m = 0; m < (long long)R * R; ++m) {
          double re, im;
          dft3d::gen::root_of_unity((b * m) % n, n, p->sign, &re, &im);
          tw2[2 * ((b - 1) * (size_t)R * R + m)] = float(re);
          tw2[2 * ((b - 1) * (size_t)R * R + m) + 1] = float(im);
        }
      DFT3D_CUDA(cudaMalloc(&ax.d_tw2, tw2.size() * sizeof(float)));
      DFT3D_CUDA(cudaMemcpy(ax.d_tw2, tw2.size() ? tw2.data() : nullptr, tw2.size() * sizeof(float), cudaMemcpyHostToDevice));
    }
    const unsigned long long dims[2] = {64ull, (unsigned long long)(2 * NB)};
    const unsigned long long strides[1] = {128ull};
    const unsigned box[2] = {64u, unsigned(NB)};
    return encode_map(&ax.map_w, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, ax.d_w, 2, dims, strides, box, 128);
  }
  std::vector<double> M(size_t(2) * R * R), T(size_t(2) * R * R);
  std::vector<float> hi(size_t(K) * K), lo(size_t(K) * K), W(size_t(2) * panels * NB * 32), tw(size_t(2) * R * R);
  dft3d::gen::axis_matrix(R, p->sign, scaled ? 1.0 / R : 1.0, nullptr, false, M.data());
  dft3d::gen::real_table_from_matrix(R, M.data(), hi.data(), lo.data());
  for (int pc = 0; pc < 2; ++pc)            // layout [piece][panel][2R rows][32 floats]
    for (int pn = 0; pn < panels; ++pn)
      for (int r = 0; r < NB; ++r)
        for (int c = 0; c < 32; ++c)
          W[((size_t(pc) * panels + pn) * NB + r) * 32 + c] = (pc ? lo : hi)[size_t(r) * K + pn * 32 + c];
  dft3d::gen::twiddle(R, R, p->sign, T.data());
  const double tscale = scaled ? 1.0 / RX : 1.0;
  for (size_t i = 0; i < T.size(); ++i) tw[i] = float(T[i] * tscale);
  DFT3D_CUDA(cudaMalloc(&ax.d_w, W.size() * sizeof(float)));
  DFT3D_CUDA(cudaMemcpy(ax.d_w, W.data(), W.size() * sizeof(float), cudaMemcpyHostToDevice));
  DFT3D_CUDA(cudaMalloc(&ax.d_tw, tw.size() * sizeof(float)));
  DFT3D_CUDA(cudaMemcpy(ax.d_tw, tw.data(), tw.size() * sizeof(float), cudaMemcpyHostToDevice));
  if (RX == 2) {
    // exp(s*2*pi*i*m/n) for m < R*R: the first column block of the (R*R) x 2 twiddle array
    std::vector<float> tw2(size_t(2) * R * R);
    for (long long m = 0; m < (long long)R * R; ++m) {
      double re, im;
      dft3d::gen::root_of_unity(m, n, p->sign, &re, &im);
      tw2[2 * m] = float(re);
      tw2[2 * m + 1] = float(im);
    }
    DFT3D_CUDA(cudaMalloc(&ax.d_tw2, tw2.size() * sizeof(float)));
    DFT3D_CUDA(cudaMemcpy(ax.d_tw2, tw2.data(), tw2.size() * sizeof(float), cudaMemcpyHostToDevice));
  }
  const unsigned long long dims[2] = {32ull, (unsigned long long)(2 * panels * NB)};
  const unsigned long long strides[1] = {128ull};
  const unsigned box[2] = {32u, unsigned(NB)};
  return encode_f32(&ax.map_w, ax.d_w, 2, dims, strides, box, 128);
}

// layout: 0 = `in` and `out` in the natural [n0][n1][n2] order.
//         1 = axis 0 only: `out` receives the blocked order T[column tile][k0][cols] (one contiguous block per stage)
//         2 = axis 1 only: `in` is in that blocked order (written by a layout-1 pass), `out` natural
// The blocked order exists because a pass along axis 0 touches rows that are n1*n2*8 bytes apart: reading them
// piecewise is cheap, writing them piecewise is not (1024^3: 3.7 ms without the stores, 9-11 ms with them).
enum { FFT_NATURAL = 0, FFT_OUT_BLOCKED = 1, FFT_IN_BLOCKED = 2 };

int fft_cols_for(const dft3d_plan_s* p, int axis, int layout) {
  const FftAxis& ax = p->fax[axis];
  int cols = ax.cols;
  if (axis != 2 && ax.R == 32 && ax.RX == 1) {
    // 1024-point strided axes: 16 lines per stage (128-byte rows) leave room for one stage-2 operand buffer only;
    // 8 lines per stage (64-byte rows) allow two.  Rows far apart (large strides) favour the wider rows.
    const long long C = (axis == 0) ? p->n[1] * p->n[2] : p->n[2];
    const int env = p->knobs.fft_cols[axis];
    // measured at 1024^3: natural layout, rows >= 1 MiB apart: 16; otherwise (close rows, or the blocked layout
    // where every stage is one contiguous block) 8-line stages, which leave room to load the next stage early
    cols = env >= 0 ? env : ((layout == FFT_NATURAL && C * 8 >= (1ll << 20)) ? 16 : 8);
    // fp16 kernel: always 16 (its raw stage is free again as soon as it has been split, so the second stage matters
    // less than the 128-byte pieces).  Measured at 1024^3: axis 1 in natural order 3.47 ms against 4.1 ms with 8;
    // from the blocked intermediate the same speed within 1 %, but 11 % less DRAM read traffic (no 64-byte halves
    // of lines), and the pass no longer has the slower second equilibrium that small timing changes tipped the
    // two-stage form into (3.6 -> 5.9 ms).
    if (env < 0 && p->f16) cols = 16;
    if (cols != 8 && cols != 16) cols = 16;
  }
  return cols;
}

// Blocked intermediate, fp16-piece kernel with direct stores: how many neighbouring rows i1 share the 128-byte lines
// of a block (see FftParams::blk_pair).  1 when the stages are 128 bytes wide anyway, or where the two passes differ.
int fft_blk_pair(const dft3d_plan_s* p) {
  if (!p->f16 || p->knobs.fft_no_pair) return 1;
  if (p->knobs.fft_stage_out_blocked > 0) return 1;
  const int colsA = fft_cols_for(p, 0, FFT_OUT_BLOCKED), cols1 = fft_cols_for(p, 1, FFT_IN_BLOCKED);
  if (cols1 != colsA) return 1;
  int P = 16 / colsA;
  if (p->knobs.fft_pair >= 0) P = p->knobs.fft_pair;
  if (P <= 1) return 1;
  return (p->n[1] % P == 0 && 256 % P == 0) ? P : 1;
}

// n2_sub != 0 (fp16-piece kernel, strided axes, blocked layouts only): the pass covers the slice
// [n2_off, n2_off + n2_sub) of the last axis.  FFT_OUT_BLOCKED: `in` is the full array, `out` receives the blocked
// order of the slice alone; FFT_IN_BLOCKED: `in` holds that, `out` is the full array (natural order).
// What fft_axis_pass prepares for one launch of the fp16-piece kernel; with `capture` it hands this back instead of
// launching (the two-axes launch combines two of them).
struct FftCapture {
  CUtensorMap map_data;
  dft3d::FftF16Params hp;
};

// A strided pass over an explicit view [batches][N][C] (natural layout) with the tables of `axis`: the first step of an
// 8192-point axis, whose eight stride-8 sub-sequences are eight times as many columns of 1024-point lines.
struct FftView {
  long long batches, C;
  int cols;              // lines per stage: 16, or 8 when the view has only eight columns
};

// map_rows != 0 (axis 2 only): the input is a ring of that many lines (the tensor map covers just them).
int fft_axis_pass(dft3d_plan_s* p, int axis, const float* in, float* out, cudaStream_t stream,
                  int layout = FFT_NATURAL, long long n2_off = 0, long long n2_sub = 0, long long map_rows = 0,
                  FftCapture* capture = nullptr, const FftView* view = nullptr) {
  const FftAxis& ax = p->fax[axis];
  const int R = ax.R, RX = ax.RX, N = int(ax.n), Lg = 128 / (R * RX);
  const int cols = view ? view->cols : fft_cols_for(p, axis, layout);
  dft3d::FftParams fp;
  memset(&fp, 0, sizeof(fp));
  fp.N = N;
  fp.twiddle = ax.d_tw;
  fp.twiddle2 = ax.d_tw2;
  fp.profile = p->d_profile;
  fp.out = out;
  fp.status = p->d_status;
  fp.blk_pair = 1;
  fp.wc = wait_control(p);
  CUtensorMap map_data, map_out;
  int rc;
  int stage_out = 0;
  const Knobs& kn = p->knobs;
  const int tag_in = 0x200 + axis * 8 + layout + (view ? 0x40 : 0), tag_out = 0x300 + axis * 8 + layout + (view ? 0x40 : 0);
  if (axis == 2 && !view) {
    const long long rows = p->n[0] * p->n[1];
    fp.rows = rows;
    fp.mtiles_per_stage = 1;
    fp.stage_bytes = Lg * N * 8;
    fp.num_stages = rows / Lg;
    rc = cached_map(p, &map_data, tag_in, in, map_rows, 0, [&](CUtensorMap* m) {
      const unsigned long long dims[3] = {256ull, (unsigned long long)(N / 128), (unsigned long long)(map_rows ? map_rows : rows)};
      const unsigned long long strides[2] = {1024ull, (unsigned long long)N * 8ull};
      const unsigned box[3] = {256u, unsigned(N / 128), unsigned(Lg)};
      return encode_f32(m, in, 3, dims, strides, box, 0);
    });
    map_out = map_data;   // unused on this axis
  } else {
    const long long batches = view ? view->batches : ((axis == 0) ? 1 : p->n[0]);
    const long long n2v = n2_sub ? n2_sub : p->n[2];                            // columns of the last axis this pass covers
    const long long C = view ? view->C : ((axis == 0) ? p->n[1] * n2v : n2v);   // columns per batch of this pass
    const long long Cmap = view ? view->C : ((axis == 0) ? p->n[1] * p->n[2] : p->n[2]);   // columns per batch of the full array
    if (n2_sub && (!p->f16 || layout == FFT_NATURAL)) return fail(DFT3D_ERR_UNSUPPORTED, "internal: sliced pass");
    fp.C = C;
    fp.out_pitch = (n2_sub && layout == FFT_IN_BLOCKED) ? Cmap : C;
    fp.out_off = (n2_sub && layout == FFT_IN_BLOCKED) ? n2_off : 0;
    if (n2_sub && layout == FFT_OUT_BLOCKED) {
      fp.col_tiles_row = int(n2_sub / cols);
      fp.col_pitch = p->n[2];
      fp.col_off = n2_off;
    }
    fp.c_tiles = C / cols;
    {
      // prefetching helps while rows are close (axis 1); with rows MiBs apart (axis 0) the pass is bound by the
      // rate of address translations and every extra request costs more than it hides (measured: 10.0 -> 12.2 ms)
      fp.l2_prefetch = kn.fft_l2_prefetch >= 0 ? kn.fft_l2_prefetch : (C * 8 < (1ll << 20) ? 1 : 0);
      if (n2_sub) fp.l2_prefetch = 0;
    }
    fp.mtiles_per_stage = cols / Lg;
    fp.stage_bytes = N * cols * 8;
    fp.num_stages = batches * fp.c_tiles;
    const unsigned long long dims[3] = {(unsigned long long)(2 * Cmap), (unsigned long long)N, (unsigned long long)batches};
    const unsigned long long strides[2] = {(unsigned long long)(Cmap * 8), (unsigned long long)N * Cmap * 8ull};
    const unsigned box[3] = {unsigned(2 * cols), 256u, 1u};
    if (layout == FFT_IN_BLOCKED) {
      // `in` = T[n2 tile][i1][k0][colsA] written by the axis-0 pass; this stage is (k0 = batch, n2 tile) and its rows are i1
      const int colsA = fft_cols_for(p, 0, FFT_OUT_BLOCKED);
      const long long n0 = p->n[0], n1 = p->n[1], n2 = n2v;
      const unsigned long long bdims[4] = {(unsigned long long)(2 * colsA), (unsigned long long)n0,
                                           (unsigned long long)n1, (unsigned long long)(n2 / colsA)};
      const unsigned long long bstr[3] = {(unsigned long long)(colsA * 8), (unsigned long long)(n0 * colsA * 8),
                                          (unsigned long long)(n1 * n0 * colsA * 8)};
      const unsigned bbox[4] = {unsigned(2 * cols), 1u, 256u, 1u};
      const int P = fft_blk_pair(p);
      if (P > 1) {
        // T[n2 tile][i1 / P][k0][i1 % P][cols]: a box takes the P neighbouring rows of one k0 (one 128-byte line) at a time
        const unsigned long long line = (unsigned long long)(P * colsA * 8);
        const unsigned long long pdims[5] = {(unsigned long long)(2 * colsA), (unsigned long long)P, (unsigned long long)n0,
                                             (unsigned long long)(n1 / P), (unsigned long long)(n2 / colsA)};
        const unsigned long long pstr[4] = {(unsigned long long)(colsA * 8), line, (unsigned long long)n0 * line,
                                            (unsigned long long)(n1 / P) * n0 * line};
        const unsigned pbox[5] = {unsigned(2 * cols), unsigned(P), 1u, unsigned(256 / P), 1u};
        rc = cached_map(p, &map_data, tag_in, in, n2_off, n2_sub, [&](CUtensorMap* m) {
          return encode_f32(m, in, 5, pdims, pstr, pbox, cols * 8, kn.promo_pair >= 0 ? kn.promo_pair : 128);
        });
        fp.blk_pair = P;
      } else {
        // rows of whole lines: fetch just them (the line after a row belongs to the next k0, a much later stage;
        // measured at 1024^3: 13 % less DRAM read traffic, same speed)
        rc = cached_map(p, &map_data, tag_in, in, n2_off, n2_sub, [&](CUtensorMap* m) {
          return encode_f32(m, in, 4, bdims, bstr, bbox, cols * 8,
                            kn.promo_blocked >= 0 ? kn.promo_blocked : (cols * 8 >= 128 ? 128 : -1), kn.promo_narrow);
        });
      }
      fp.in_blocked = 1;
      fp.blk_ratio = colsA / cols;
      fp.l2_prefetch = 0;
    } else {
      rc = cached_map(p, &map_data, tag_in, in, n2_off, n2_sub, [&](CUtensorMap* m) {
        return encode_f32(m, in, 3, dims, strides, box, cols * 8, -1, kn.promo_narrow);
      });
    }
    if (layout == FFT_OUT_BLOCKED) {
      const unsigned long long bdims[3] = {(unsigned long long)(2 * cols), (unsigned long long)N, (unsigned long long)(C / cols)};
      const unsigned long long bstr[2] = {(unsigned long long)(cols * 8), (unsigned long long)N * cols * 8ull};
      if (rc == DFT3D_OK)
        rc = cached_map(p, &map_out, tag_out, out, n2_off, n2_sub, [&](CUtensorMap* m) {
          return encode_f32(m, out, 3, bdims, bstr, box, cols * 8, -1, kn.promo_narrow);
        });
      fp.out_blocked = 1;
      fp.blk_pair = fft_blk_pair(p);
      fp.blk_tiles = int(n2v / cols);
      fp.blk_rows = int(p->n[1]);
      // TF32 kernel: the stage returns through shared memory and leaves as TMA stores; fp16 kernel: plain stores
      // from registers (a block is one contiguous region), which frees the raw stage right after the split
      stage_out = kn.fft_stage_out_blocked >= 0 ? kn.fft_stage_out_blocked : (p->f16 ? 0 : 1);
    } else {
      if (capture) map_out = map_data;   // the two-axes launch stores straight from registers
      else if (rc == DFT3D_OK)
        rc = cached_map(p, &map_out, tag_out, out, n2_off, n2_sub, [&](CUtensorMap* m) {
          return encode_f32(m, out, 3, dims, strides, box, cols * 8, -1, kn.promo_narrow);
        });
      // rows MiBs apart: send the results out as full rows through TMA stores instead of 32-byte pieces
      stage_out = kn.fft_stage_out >= 0 ? kn.fft_stage_out : (Cmap * 8 >= (1ll << 20) ? 1 : 0);
      if (capture) stage_out = 0;
    }
    if (n2_sub && stage_out) return fail(DFT3D_ERR_UNSUPPORTED, "internal: sliced pass with staged output");
  }
  if (rc != DFT3D_OK) return rc;
  if (p->f16) {
    // fp16 pieces: two stage-2 operand buffers and a 128 KB raw ring at every size
    dft3d::FftF16Params hp;
    hp.base = fp;
    hp.out_mul = ax.out_mul;
    hp.quarter_turn = float(p->sign);
    hp.base.raw_stages = dft3d::kFft16RawBytes / fp.stage_bytes;
    if (hp.base.raw_stages > 4) hp.base.raw_stages = 4;
    // a worker group takes every fourth M-tile, i.e. every (4 / tiles per stage)-th stage: that step must divide the
    // ring length so that the group meets each ring slot in consecutive phases
    if (fp.mtiles_per_stage == 1 && hp.base.raw_stages != 4) return fail(DFT3D_ERR_UNSUPPORTED, "internal: raw ring of %d stages", hp.base.raw_stages);
    if (fp.mtiles_per_stage == 2 && hp.base.raw_stages == 3) hp.base.raw_stages = 2;
    if (fp.mtiles_per_stage != 1 && fp.mtiles_per_stage != 2 && fp.mtiles_per_stage != 4)
      return fail(DFT3D_ERR_UNSUPPORTED, "internal: %d tiles per stage", fp.mtiles_per_stage);
    if (capture) {
      capture->map_data = map_data;
      capture->hp = hp;
      return DFT3D_OK;
    }
    const int grid = int(fp.num_stages < p->sm_count ? fp.num_stages : p->sm_count);
    const size_t smem = dft3d::fft16_smem_bytes(R, RX);
#define DFT3D_FFT16_LAUNCH(MODE, R_, RX_, COLS_, SO_)                                         \
  dft3d::fft_f16_axis_kernel<MODE, R_, RX_, COLS_, SO_>                                        \
      <<<grid, dft3d::kFftThreads, smem, stream>>>(map_data, ax.map_w, map_out, hp)
    if (axis == 2 && !view) {
      if (R == 32 && RX == 1) DFT3D_FFT16_LAUNCH(dft3d::FFT_CONTIG, 32, 1, 16, 0);
      else if (R == 16 && RX == 1) DFT3D_FFT16_LAUNCH(dft3d::FFT_CONTIG, 16, 1, 16, 0);
      else if (R == 32 && RX == 4) DFT3D_FFT16_LAUNCH(dft3d::FFT_CONTIG, 32, 4, 16, 0);
      else if (R == 32) DFT3D_FFT16_LAUNCH(dft3d::FFT_CONTIG, 32, 2, 16, 0);
      else DFT3D_FFT16_LAUNCH(dft3d::FFT_CONTIG, 16, 2, 16, 0);
    } else if (!stage_out) {
      if (R == 32 && RX == 1 && cols == 16) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 16, 0);
      else if (R == 32 && RX == 1) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 8, 0);
      else if (R == 16 && RX == 1) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 16, 1, 16, 0);
      else if (R == 32 && RX == 4) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 4, 4, 0);
      else if (R == 32) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 2, 8, 0);
      else DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 16, 2, 16, 0);
    } else {
      if (R == 32 && RX == 1 && cols == 16) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 16, 1);
      else if (R == 32 && RX == 1) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 8, 1);
      else if (R == 16 && RX == 1) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 16, 1, 16, 1);
      else if (R == 32 && RX == 4) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 4, 4, 1);
      else if (R == 32) DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 32, 2, 8, 1);
      else DFT3D_FFT16_LAUNCH(dft3d::FFT_STRIDED, 16, 2, 16, 1);
    }
#undef DFT3D_FFT16_LAUNCH
    DFT3D_CUDA(cudaGetLastError());
    return DFT3D_OK;
  }
  int nb2 = (axis == 2 || R == 16 || (R == 32 && RX == 1 && cols == 8)) ? 2 : 1;
  if (axis != 2 && R == 32 && RX == 1 && cols == 8) {
    // 8-line stages: two stage-2 operand buffers and one raw stage (best with direct stores), or one operand
    // buffer and two raw stages (best when the results return through the raw stage, which then stays busy longer)
    nb2 = kn.fft_nb2 >= 0 ? kn.fft_nb2 : (layout != FFT_NATURAL ? 1 : 2);
    if (nb2 != 1 && nb2 != 2) nb2 = 2;
  }
  fp.raw_stages = dft3d::fft_raw_bytes(R, nb2) / fp.stage_bytes;
  if (fp.raw_stages > 4) fp.raw_stages = 4;
  const int grid = int(fp.num_stages < p->sm_count ? fp.num_stages : p->sm_count);
  const size_t smem = dft3d::fft_smem_bytes(R, nb2);
#define DFT3D_FFT_LAUNCH(MODE, R_, RX_, COLS_, NB2_, SO_)                                                     \
  dft3d::fft_axis_kernel<MODE, R_, RX_, COLS_, NB2_, SO_>                                                      \
      <<<grid, dft3d::kFftThreads, smem, stream>>>(map_data, ax.map_w, map_out, fp)
  if (axis == 2) {
    if (R == 32 && RX == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_CONTIG, 32, 1, 16, 2, 0);
    else if (R == 16 && RX == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_CONTIG, 16, 1, 16, 2, 0);
    else if (R == 32) DFT3D_FFT_LAUNCH(dft3d::FFT_CONTIG, 32, 2, 16, 2, 0);
    else DFT3D_FFT_LAUNCH(dft3d::FFT_CONTIG, 16, 2, 16, 2, 0);
  } else if (!stage_out) {
    if (R == 32 && RX == 1 && cols == 16) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 16, 1, 0);
    else if (R == 32 && RX == 1 && nb2 == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 8, 1, 0);
    else if (R == 32 && RX == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 8, 2, 0);
    else if (R == 16 && RX == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 16, 1, 16, 2, 0);
    else if (R == 32) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 2, 8, 1, 0);
    else DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 16, 2, 16, 2, 0);
  } else {
    if (R == 32 && RX == 1 && cols == 16) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 16, 1, 1);
    else if (R == 32 && RX == 1 && nb2 == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 8, 1, 1);
    else if (R == 32 && RX == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 1, 8, 2, 1);
    else if (R == 16 && RX == 1) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 16, 1, 16, 2, 1);
    else if (R == 32) DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 32, 2, 8, 1, 1);
    else DFT3D_FFT_LAUNCH(dft3d::FFT_STRIDED, 16, 2, 16, 2, 1);
  }
#undef DFT3D_FFT_LAUNCH
  DFT3D_CUDA(cudaGetLastError());
  return DFT3D_OK;
}

// The two launches of an 8192-point axis (see FftAxis::r8), natural layout: src -> mid -> dst (three distinct cubes, or
// mid == the caller's scratch).  lines = product of the dimensions before the axis, C = columns behind it.
void r8_geometry(const dft3d_plan_s* p, int axis, long long* lines, long long* C) {
  *lines = axis == 0 ? 1 : (axis == 1 ? p->n[0] : p->n[0] * p->n[1]);
  *C = axis == 0 ? p->n[1] * p->n[2] : (axis == 1 ? p->n[2] : 1);
}

int fft_r8_first(dft3d_plan_s* p, int axis, const float* src, float* mid, cudaStream_t stream) {
  long long lines, C;
  r8_geometry(p, axis, &lines, &C);
  FftView v;
  v.batches = lines;
  v.C = 8 * C;                       // sub-sequence beta of column c is column beta*C + c of the 1024-point lines
  v.cols = (8 * C) % 16 == 0 ? 16 : 8;
  return fft_axis_pass(p, axis, src, mid, stream, FFT_NATURAL, 0, 0, 0, nullptr, &v);
}

int fft_r8_second(dft3d_plan_s* p, int axis, const float* mid, float* dst, cudaStream_t stream) {
  dft3d::Radix8Params rp;
  rp.in = reinterpret_cast<const float2*>(mid);
  rp.out = reinterpret_cast<float2*>(dst);
  rp.tw = p->fax[axis].d_tw8;
  r8_geometry(p, axis, &rp.lines, &rp.C);
  rp.sign = float(p->sign);
  const long long total = rp.lines * 1024 * rp.C;
  long long blocks = (total + dft3d::kRadix8Threads - 1) / dft3d::kRadix8Threads;
  const long long cap = (long long)p->sm_count * 32;
  if (blocks > cap) blocks = cap;
  dft3d::fft_radix8_kernel<<<int(blocks), dft3d::kRadix8Threads, 0, stream>>>(rp);
  DFT3D_CUDA(cudaGetLastError());
  return DFT3D_OK;
}

// Axes 1 and 2 of a 3D FFT plan in one launch: `blocked` holds the axis-0 pass's result in the blocked order, the
// result goes to `out`; the intermediate lives in the plan's ring of n0-planes.
int fft_fused12_pass(dft3d_plan_s* p, const float* blocked, float* out, cudaStream_t stream) {
  FftCapture w, r;
  int rc = fft_axis_pass(p, 1, blocked, static_cast<float*>(p->ring), stream, FFT_IN_BLOCKED, 0, 0, 0, &w);
  if (rc != DFT3D_OK) return rc;
  const long long ring_rows = (long long)p->ring_planes * p->n[1];
  rc = fft_axis_pass(p, 2, static_cast<const float*>(p->ring), out, stream, FFT_NATURAL, 0, 0, ring_rows, &r);
  if (rc != DFT3D_OK) return rc;
  const long long n0 = p->n[0];
  DFT3D_CUDA(cudaMemsetAsync(p->d_fuse_counters, 0, sizeof(unsigned int) * 2 * size_t(n0), stream));
  dft3d::FftFuse fz;
  memset(&fz, 0, sizeof(fz));
  fz.written = p->d_fuse_counters;
  fz.consumed = p->d_fuse_counters + n0;
  fz.ring = p->ring_planes;
  fz.ring_rows = ring_rows;
  fz.ctas_writer = p->fuse_writers;
  fz.evict_hints = p->knobs.fft_fuse_hints >= 0 ? p->knobs.fft_fuse_hints : 0;
  // every worker warp (4 per tile) counts itself in once per tile
  fz.written_target = unsigned(w.hp.base.c_tiles * w.hp.base.mtiles_per_stage * 4);
  const long long reader_spp = p->n[1] / (128 / (p->fax[2].R * p->fax[2].RX));
  fz.consumed_target = unsigned(reader_spp * r.hp.base.mtiles_per_stage * 4);
  // each side counts planes in its own stages
  w.hp.base.fuse_stages_per_plane = w.hp.base.c_tiles;
  r.hp.base.fuse_stages_per_plane = reader_spp;
  const int grid = p->sm_count;
  if (p->fax[1].R == 32)
    dft3d::fft_f16_fused_kernel<32, 16><<<grid, dft3d::kFftThreads, dft3d::fft16_smem_bytes(32, 1), stream>>>(
        w.map_data, p->fax[1].map_w, r.map_data, w.hp, r.hp, fz);
  else
    dft3d::fft_f16_fused_kernel<16, 16><<<grid, dft3d::kFftThreads, dft3d::fft16_smem_bytes(16, 1), stream>>>(
        w.map_data, p->fax[1].map_w, r.map_data, w.hp, r.hp, fz);
  DFT3D_CUDA(cudaGetLastError());
  return DFT3D_OK;
}

int check_io(const dft3d_plan_s* p, const void* in, const void* out) {
  if (!p) return fail(DFT3D_ERR_INVALID_ARG, "plan is NULL");
  if (!in || !out) return fail(DFT3D_ERR_INVALID_ARG, "in/out must not be NULL");
  if ((reinterpret_cast<uintptr_t>(in) & 15) || (reinterpret_cast<uintptr_t>(out) & 15))
    return fail(DFT3D_ERR_INVALID_ARG, "in/out must be 16-byte aligned");
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != p->device)
    return fail(DFT3D_ERR_INVALID_ARG, "the plan was created on device %d but device %d is current", p->device, dev);
  const size_t bytes = size_t(points(p)) * 8;
  const char* a = static_cast<const char*>(in);
  const char* b = static_cast<const char*>(out);
  if (a < b + bytes && b < a + bytes) return fail(DFT3D_ERR_INVALID_ARG, "in and out overlap");
  return DFT3D_OK;
}

}  // namespace

extern "C" {

const char* dft3d_status_string(int status) {
  switch (status) {
    case DFT3D_OK: return "ok";
    case DFT3D_ERR_INVALID_ARG: return "invalid argument";
    case DFT3D_ERR_UNSUPPORTED: return "unsupported size or option";
    case DFT3D_ERR_ALLOC: return "allocation failed";
    case DFT3D_ERR_CUDA: return "CUDA call failed";
    case DFT3D_ERR_DEVICE_TIMEOUT: return "a kernel abandoned a bounded wait";
    default: return "unknown status";
  }
}

const char* dft3d_last_error(void) { return g_last_error; }

#ifdef DFT3D_PROFILE_WAITS
// diagnostic builds only: copies the MMA issuer's cycle counters [grid][4] = {total, wait acc, wait W, wait data}
int dft3d_debug_read_profile(dft3d_plan_t p, long long* host, int ctas) {
  if (cudaMemcpy(host, p->d_profile, sizeof(long long) * ctas, cudaMemcpyDeviceToHost) != cudaSuccess) return 4;
  return cudaMemset(p->d_profile, 0, sizeof(long long) * ctas) == cudaSuccess ? 0 : 4;   // counters restart after a read
}
#endif

int dft3d_generate_axis_matrix(long long n, int sign, double scale, const double* nodes, int nodes_on_output,
                               double* matrix) {
  if (n < 1 || !matrix || (sign != -1 && sign != 1)) return fail(DFT3D_ERR_INVALID_ARG, "bad argument");
  if (nodes)
    for (long long i = 0; i < n; ++i)
      if (!std::isfinite(nodes[i])) return fail(DFT3D_ERR_INVALID_ARG, "node %lld is not finite", i);
  dft3d::gen::axis_matrix(n, sign, scale, nodes, nodes_on_output != 0, matrix);
  return DFT3D_OK;
}

int dft3d_generate_inverse_matrix(long long n, const double* nodes, int nodes_on_output, double* matrix, double* growth) {
  if (n < 1 || !matrix || !nodes) return fail(DFT3D_ERR_INVALID_ARG, "bad argument");
  for (long long i = 0; i < n; ++i)
    if (!std::isfinite(nodes[i])) return fail(DFT3D_ERR_INVALID_ARG, "node %lld is not finite", i);
  dft3d::gen::axis_matrix(n, DFT3D_FORWARD, 1.0, nodes, nodes_on_output != 0, matrix);
  if (!dft3d::gen::invert_matrix(n, matrix, growth))
    return fail(DFT3D_ERR_INVALID_ARG, "the matrix of these nodes is singular (nodes must be distinct modulo 1)");
  return DFT3D_OK;
}

int dft3d_generate_twiddle(long long N1, long long N2, int sign, double* twiddle) {
  if (N1 < 1 || N2 < 1 || !twiddle || (sign != -1 && sign != 1)) return fail(DFT3D_ERR_INVALID_ARG, "bad argument");
  dft3d::gen::twiddle(N1, N2, sign, twiddle);
  return DFT3D_OK;
}

int dft3d_generate_real_table(long long n, int sign, double scale, const double* nodes, int nodes_on_output,
                              float* hi, float* lo) {
  if (n < 1 || !hi || !lo || (sign != -1 && sign != 1)) return fail(DFT3D_ERR_INVALID_ARG, "bad argument");
  std::vector<double> M;
  try {
    M.resize(size_t(2) * n * n);
  } catch (const std::bad_alloc&) {
    return fail(DFT3D_ERR_ALLOC, "host allocation failed");
  }
  int rc = dft3d_generate_axis_matrix(n, sign, scale, nodes, nodes_on_output, M.data());
  if (rc != DFT3D_OK) return rc;
  dft3d::gen::real_table_from_matrix(n, M.data(), hi, lo);
  return DFT3D_OK;
}

int dft3d_plan_create_ex(dft3d_plan_t* out, long long n0, long long n1, long long n2, int mode, int sign,
                         const double* nodes0, const double* nodes1, const double* nodes2,
                         const dft3d_options_t* options) {
  if (!out) return fail(DFT3D_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (n0 < 1 || n1 < 1 || n2 < 1) return fail(DFT3D_ERR_INVALID_ARG, "sizes must be >= 1");
  if (mode != DFT3D_KDFT && mode != DFT3D_FFT && mode != DFT3D_AUTO)
    return fail(DFT3D_ERR_INVALID_ARG, "mode must be DFT3D_KDFT, DFT3D_FFT or DFT3D_AUTO");
  if (sign != DFT3D_FORWARD && sign != DFT3D_INVERSE) return fail(DFT3D_ERR_INVALID_ARG, "sign must be -1 or +1");
  const long long nn[3] = {n0, n1, n2};
  const double* nodes[3] = {nodes0, nodes1, nodes2};
  for (int a = 0; a < 3; ++a)
    if (nodes[a])
      for (long long i = 0; i < nn[a]; ++i)
        if (!std::isfinite(nodes[a][i])) return fail(DFT3D_ERR_INVALID_ARG, "node %lld of axis %d is not finite", i, a);
  dft3d_options_t opt;
  memset(&opt, 0, sizeof(opt));
  if (options) {
    if (options->struct_size < sizeof(size_t) + sizeof(unsigned) || options->struct_size > sizeof(opt))
      return fail(DFT3D_ERR_INVALID_ARG, "options->struct_size is not a known size");
    memcpy(&opt, options, options->struct_size);
  }
  if (opt.flags & ~(DFT3D_NODES_ON_OUTPUT | DFT3D_UNSCALED_INVERSE | DFT3D_SPLIT_FP16 | DFT3D_SPLIT_TF32 | DFT3D_DESTROY_INPUT |
                    DFT3D_INVERSE_SOLVE))
    return fail(DFT3D_ERR_INVALID_ARG, "unknown flag");
  if (opt.flags & DFT3D_INVERSE_SOLVE) {
    if (mode == DFT3D_FFT || sign != DFT3D_INVERSE || (opt.flags & DFT3D_UNSCALED_INVERSE))
      return fail(DFT3D_ERR_INVALID_ARG, "DFT3D_INVERSE_SOLVE needs mode KDFT (or AUTO), sign +1 and the scaled inverse");
    for (int a = 0; a < 3; ++a)
      if (nodes[a] && nn[a] > 2048)
        return fail(DFT3D_ERR_UNSUPPORTED, "DFT3D_INVERSE_SOLVE inverts the n x n matrix on the host: n%d = %lld exceeds 2048", a, nn[a]);
  }
  if ((opt.flags & DFT3D_SPLIT_FP16) && (opt.flags & DFT3D_SPLIT_TF32))
    return fail(DFT3D_ERR_INVALID_ARG, "DFT3D_SPLIT_FP16 and DFT3D_SPLIT_TF32 exclude each other");
  // default: fp16 pieces (KDFT: where the sizes allow it, see below)
  bool f16 = !(opt.flags & DFT3D_SPLIT_TF32);
  if (opt.axes > 7) return fail(DFT3D_ERR_INVALID_ARG, "axes must be a mask of bits 0..2");
  const unsigned axes = opt.axes ? opt.axes : 7u;
  for (int a = 0; a < 3; ++a) {
    const bool transformed = (axes >> a) & 1u;
    if (a == 0 && !transformed) continue;   // a pure batch index
    // KDFT: rows of the data must start on 16-byte boundaries (TMA): the last axis must be even, the others may have
    // any length (odd lengths pad the table, not the data).  FFT: the untransformed axes are split into groups of 16 lines
    const long long quantum = (mode == DFT3D_FFT) ? 64 : (a == 2 ? 2 : 1);
    if (nn[a] % quantum != 0)
      return fail(DFT3D_ERR_UNSUPPORTED, "n%d = %lld is not a multiple of %lld%s", a, nn[a], quantum,
                  (mode != DFT3D_FFT && a == 2) ? " (rows of the data, 8*n2 bytes each, must start on 16-byte boundaries)" : "");
    if (transformed && nn[a] > 8192) return fail(DFT3D_ERR_UNSUPPORTED, "n%d = %lld exceeds 8192", a, nn[a]);
    if (transformed && nn[a] % 4 != 0) {
      if (opt.flags & DFT3D_SPLIT_FP16)
        return fail(DFT3D_ERR_UNSUPPORTED, "DFT3D_SPLIT_FP16 needs n%d = %lld to be a multiple of 4", a, nn[a]);
      f16 = false;
    }
  }
  if (mode == DFT3D_FFT && (nodes0 || nodes1 || nodes2))
    return fail(DFT3D_ERR_UNSUPPORTED, "the FFT formulation needs a uniform grid (no nodes)");
  // DFT3D_AUTO: the FFT formulation on every axis where it applies (uniform grid, a supported length, and enough
  // neighbouring lines for its stages), the KDFT formulation on the others
  int amode[3] = {mode, mode, mode};
  if (mode == DFT3D_AUTO) {
    const long long inner[3] = {n1 * n2, n2, n0 * n1};   // columns beside a line (axes 0, 1) / number of lines (axis 2)
    bool all_fft = true, all_kdft = true, fft_sizes_ok = true;
    for (int a = 0; a < 3; ++a) {
      if (!((axes >> a) & 1u)) { if (a != 0 && nn[a] % 64 != 0) fft_sizes_ok = false; continue; }
      const long long n = nn[a];
      const bool length_ok = n == 256 || n == 512 || n == 1024 || n == 2048 || (n == 4096 && f16);
      // (8192 points: the first launch sees eight times as many columns, so an even count, or the last axis, will do)
      const bool fft_ok = !nodes[a] && ((length_ok && inner[a] % 16 == 0) ||
                                        (n == 8192 && f16 && (a == 2 || inner[a] % 2 == 0)));
      amode[a] = fft_ok ? DFT3D_FFT : DFT3D_KDFT;
      (fft_ok ? all_kdft : all_fft) = false;
      if (nn[a] % 64 != 0) fft_sizes_ok = false;
    }
    if (all_kdft) mode = DFT3D_KDFT;                       // one formulation only: its own schedules apply
    else if (all_fft && fft_sizes_ok) mode = DFT3D_FFT;
    if (mode != DFT3D_AUTO)
      for (int a = 0; a < 3; ++a) amode[a] = mode;
  }
  // An 8192-point FFT axis takes two launches (FftAxis::r8); plans that have one run the axes one after the other in
  // the natural layout, like plans that mix the formulations
  if (mode == DFT3D_FFT)
    for (int a = 0; a < 3; ++a)
      if (((axes >> a) & 1u) && nn[a] == 8192) mode = DFT3D_AUTO;

  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return fail(DFT3D_ERR_CUDA, "no CUDA device available");
  dft3d_plan_s* p = new (std::nothrow) dft3d_plan_s();
  if (!p) return fail(DFT3D_ERR_ALLOC, "host allocation of the plan failed");
  int rc = DFT3D_OK;
  do {
    for (int a = 0; a < 3; ++a) p->n[a] = nn[a];
    p->mode = mode;
    for (int a = 0; a < 3; ++a) p->amode[a] = amode[a];
    p->sign = sign;
    p->flags = opt.flags;
    p->f16 = f16;
    p->axes = axes;
    cudaDeviceProp prop;
    if (cudaGetDevice(&p->device) != cudaSuccess || cudaGetDeviceProperties(&prop, p->device) != cudaSuccess) {
      rc = fail(DFT3D_ERR_CUDA, "cannot query the current device");
      break;
    }
    if (prop.major != 10) {
      rc = fail(DFT3D_ERR_UNSUPPORTED, "device %s is sm_%d%d; this library is built for sm_100a only", prop.name,
                prop.major, prop.minor);
      break;
    }
    p->sm_count = prop.multiProcessorCount;
    p->knobs = read_knobs();
    if (p->knobs.chunk_kb >= 1) p->chunk_kb = p->knobs.chunk_kb;   // tuning knob: stages per accumulation chain
    if ((rc = set_kernel_attributes(p->device)) != DFT3D_OK) break;
    cudaError_t e = cudaMalloc(&p->d_status, sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(p->d_status, 0, sizeof(unsigned int));
    if (e != cudaSuccess) { rc = fail(DFT3D_ERR_ALLOC, "cudaMalloc(status): %s", cudaGetErrorString(e)); break; }
#ifdef DFT3D_PROFILE_WAITS
    e = cudaMalloc(&p->d_profile, sizeof(long long) * 128 * 256);
    if (e == cudaSuccess) e = cudaMemset(p->d_profile, 0, sizeof(long long) * 128 * 256);
    if (e != cudaSuccess) { rc = fail(DFT3D_ERR_ALLOC, "cudaMalloc(profile)"); break; }
#endif
    e = cudaMalloc(&p->d_amax, 4 * sizeof(unsigned int));
    if (e != cudaSuccess) { rc = fail(DFT3D_ERR_ALLOC, "cudaMalloc(amax): %s", cudaGetErrorString(e)); break; }
    if (mode == DFT3D_AUTO) {
      // both formulations in one plan: every pass goes from one cube to another in the natural layout
      int count = 0;   // passes: one per axis, two for an 8192-point FFT axis
      for (int a = 0; a < 3 && rc == DFT3D_OK; ++a)
        if ((axes >> a) & 1u) {
          rc = amode[a] == DFT3D_FFT ? build_fft_axis(p, a, opt.fft_split[a]) : build_kdft_axis(p, a, nodes[a]);
          count += (amode[a] == DFT3D_FFT && p->fax[a].r8) ? 2 : 1;
        }
      if (rc != DFT3D_OK) break;
      p->group_planes = n0;
      const size_t cube_bytes = size_t(n0) * n1 * n2 * 8;
      const size_t limit = opt.workspace_limit ? opt.workspace_limit : (size_t(16) << 30);
      if (count >= 2) {
        // Three passes go in -> out -> workspace -> out, so the input may serve as the workspace once the first pass
        // has read it.  Two passes go in -> workspace -> out: the first would run in place on the input, which a KDFT
        // pass cannot (every output tile re-reads whole lines), so two-axis plans allocate their workspace.
        if ((opt.flags & DFT3D_DESTROY_INPUT) && count >= 3 && count % 2 == 1) {
          p->in_is_ws = true;
        } else if (cube_bytes > limit) {
          rc = fail(DFT3D_ERR_UNSUPPORTED, "a plan that mixes the formulations needs a workspace as large as the cube "
                    "(%zu bytes): raise workspace_limit or pass DFT3D_DESTROY_INPUT", cube_bytes);
          break;
        } else {
          e = cudaMalloc(&p->workspace, cube_bytes);
          if (e != cudaSuccess) { rc = fail(DFT3D_ERR_ALLOC, "cudaMalloc(workspace %zu bytes): %s", cube_bytes, cudaGetErrorString(e)); break; }
          p->workspace_bytes = cube_bytes;
        }
      }
    } else if (mode == DFT3D_KDFT) {
      for (int a = 0; a < 3 && rc == DFT3D_OK; ++a)
        if ((axes >> a) & 1u) rc = build_kdft_axis(p, a, nodes[a]);
      if (rc != DFT3D_OK) break;
      // workspace: whole cube when it fits the limit, else a group of n0-planes with at least ~8 waves of tiles
      const size_t plane_bytes = size_t(n1) * n2 * 8;
      size_t limit = opt.workspace_limit ? opt.workspace_limit : (size_t(16) << 30);
      long long g = n0;
      // with DFT3D_DESTROY_INPUT the input cube is the workspace once the first pass has read it
      p->in_is_ws = (opt.flags & DFT3D_DESTROY_INPUT) && axes == 7u;
      if (p->in_is_ws) limit = ~size_t(0);
      if (size_t(g) * plane_bytes > limit) {
        g = (long long)(limit / plane_bytes);
        if (g < 1) g = 1;
        while (n0 % g) --g;   // groups of equal size
      }
      if (g != n0 && (axes == 3u || axes == 5u)) {
        rc = fail(DFT3D_ERR_UNSUPPORTED, "transforming axis 0 and one other axis needs a workspace as large as the cube "
                  "(%zu bytes); raise workspace_limit", size_t(n0) * plane_bytes);
        break;
      }
      if (axes == 1u || axes == 2u || axes == 4u) g = 0;   // a single axis goes straight from in to out
      p->group_planes = g ? g : n0;
      p->workspace_bytes = p->in_is_ws ? 0 : size_t(g) * plane_bytes;
      if (g != 0 && !p->in_is_ws) {
        e = cudaMalloc(&p->workspace, p->workspace_bytes);
        if (e != cudaSuccess) { rc = fail(DFT3D_ERR_ALLOC, "cudaMalloc(workspace %zu bytes): %s", p->workspace_bytes, cudaGetErrorString(e)); break; }
      }
    } else {
      for (int a = 0; a < 3 && rc == DFT3D_OK; ++a)
        if ((axes >> a) & 1u) rc = build_fft_axis(p, a, opt.fft_split[a]);
      if (rc != DFT3D_OK) break;
      // a cube of workspace, if it fits the limit, lets the axis-0 pass avoid piecewise writes to far-apart rows;
      // without it the three passes run in place on `out`
      const size_t cube_bytes = size_t(n0) * n1 * n2 * 8;
      const size_t limit = opt.workspace_limit ? opt.workspace_limit : (size_t(16) << 30);
      const bool nests = fft_cols_for(p, 0, FFT_OUT_BLOCKED) % fft_cols_for(p, 1, FFT_IN_BLOCKED) == 0;
      if (axes == 7u && nests && (opt.flags & DFT3D_DESTROY_INPUT)) {
        p->in_is_ws = true;   // in -> out (blocked) -> in (natural) -> out
      } else if (axes == 7u && cube_bytes <= limit && nests) {
        e = cudaMalloc(&p->workspace, cube_bytes);
        if (e == cudaSuccess) p->workspace_bytes = cube_bytes;
        else { p->workspace = nullptr; (void)cudaGetLastError(); }   // fall back to the in-place schedule
        // On request (DFT3D_FFT_FUSE=1): axes 1 and 2 in one launch through a ring of n0-planes that stays in L2 (fp16
        // pieces, both axes R*R points with the same R, 16-line stages on both strided passes); the axis-0 pass then
        // writes the blocked order into the workspace.  Not the default: measured at 1024^3 the launch moves 33 instead
        // of 48 bytes per point through HBM (every ring read hits L2) but takes as long as the two launches it replaces,
        // because each SM's tile rate, not the HBM stream, bounds these passes (12.1 against 11.6 ms per transform).
        const FftAxis& a1 = p->fax[1];
        const FftAxis& a2 = p->fax[2];
        const int ring = p->knobs.fft_fuse_ring > 0 ? p->knobs.fft_fuse_ring : 4;
        if (p->workspace && p->f16 && p->knobs.fft_fuse > 0 && a1.R == a2.R && a1.RX == 1 && a2.RX == 1 &&
            fft_cols_for(p, 0, FFT_OUT_BLOCKED) == 16 && fft_cols_for(p, 1, FFT_IN_BLOCKED) == 16 && n0 >= 2 * ring &&
            p->sm_count >= 8 && p->knobs.fft_stage_out_blocked <= 0) {
          const size_t ring_bytes = size_t(ring) * n1 * n2 * 8;
          e = cudaMalloc(&p->ring, ring_bytes);
          if (e == cudaSuccess) e = cudaMalloc(&p->d_fuse_counters, sizeof(unsigned int) * 2 * size_t(n0));
          if (e == cudaSuccess) {
            p->fuse12 = true;
            p->ring_planes = ring;
            p->workspace_bytes += ring_bytes;
            // CTAs of the axis-1 side; the rest run the axis-2 side.  The strided side needs a little more time per
            // point than the contiguous one (3.5 against 2.9 ms per pass of 1024^3), so it gets the larger share.
            int wr = p->knobs.fft_fuse_writers > 0 ? p->knobs.fft_fuse_writers : (p->sm_count * 80 + 74) / 148;
            if (wr >= p->sm_count) wr = p->sm_count - 1;
            p->fuse_writers = wr;
          } else {
            if (p->ring) { cudaFree(p->ring); p->ring = nullptr; }
            (void)cudaGetLastError();
          }
        }
      } else if (axes == 7u && nests && p->f16 && !p->knobs.fft_no_half) {
        // Too large for a whole cube of workspace: a half, a quarter or an eighth of a cube, whichever fits first.
        // The two strided passes then run once per slice of the last axis through the blocked order in the workspace,
        // each writing its slice of `out` in natural order, and the contiguous pass runs in place on `out`.
        const int c0 = fft_cols_for(p, 0, FFT_OUT_BLOCKED), c1 = fft_cols_for(p, 1, FFT_IN_BLOCKED);
        const int forced = p->knobs.fft_slices;
        for (int k = 2; k <= 8 && !p->ws_slices; k *= 2) {
          const long long sub = n2 / k;
          if (forced && k != forced) continue;
          if (n2 % k != 0 || sub % c0 != 0 || sub % c1 != 0 || n2 * 8 >= (1ll << 20)) break;
          if (cube_bytes / k > limit && !forced) continue;
          e = cudaMalloc(&p->workspace, cube_bytes / k);
          if (e == cudaSuccess) { p->workspace_bytes = cube_bytes / k; p->ws_slices = k; }
          else { p->workspace = nullptr; (void)cudaGetLastError(); break; }
        }
      }
    }
  } while (0);
  if (rc != DFT3D_OK) {
    char keep[sizeof(g_last_error)];
    memcpy(keep, g_last_error, sizeof(keep));
    dft3d_plan_destroy(p);
    memcpy(g_last_error, keep, sizeof(keep));
    return rc;
  }
  *out = p;
  return DFT3D_OK;
}

int dft3d_plan_create(dft3d_plan_t* out, long long n0, long long n1, long long n2, int mode, int sign,
                      const double* nodes0, const double* nodes1, const double* nodes2) {
  return dft3d_plan_create_ex(out, n0, n1, n2, mode, sign, nodes0, nodes1, nodes2, nullptr);
}

int dft3d_execute_axis(dft3d_plan_t p, int axis, const void* in, void* out, void* cuda_stream) {
  int rc = check_io(p, in, out);
  if (rc != DFT3D_OK) return rc;
  if (axis < 0 || axis > 2) return fail(DFT3D_ERR_INVALID_ARG, "axis must be 0, 1 or 2");
  if (!((p->axes >> axis) & 1u)) return fail(DFT3D_ERR_INVALID_ARG, "axis %d is not among the plan's axes", axis);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (p->amode[axis] == DFT3D_KDFT) {
    if ((rc = prepare_scales(p, static_cast<const float*>(in), stream)) != DFT3D_OK) return rc;
    return kdft_axis_pass(p, axis, static_cast<const float*>(in), static_cast<float*>(out), p->n[0], stream, 0);
  }
  if (p->fax[axis].r8) {
    if (!p->workspace) return fail(DFT3D_ERR_UNSUPPORTED, "an 8192-point FFT axis alone needs the plan's workspace, which this plan does not own");
    if ((rc = fft_r8_first(p, axis, static_cast<const float*>(in), static_cast<float*>(p->workspace), stream)) != DFT3D_OK) return rc;
    return fft_r8_second(p, axis, static_cast<const float*>(p->workspace), static_cast<float*>(out), stream);
  }
  return fft_axis_pass(p, axis, static_cast<const float*>(in), static_cast<float*>(out), stream);
}

int dft3d_execute(dft3d_plan_t p, const void* in, void* out, void* cuda_stream) {
  int rc = check_io(p, in, out);
  if (rc != DFT3D_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const float* fin = static_cast<const float*>(in);
  float* fout = static_cast<float*>(out);
  const unsigned axes = p->axes;
  if (p->mode == DFT3D_AUTO) {
    // mixed formulations: axis 0, 1, 2 in turn, natural layout throughout, alternating between the cubes so that the
    // last pass writes `out` (three passes: in -> out -> workspace -> out; two: in -> workspace -> out)
    float* ws = p->in_is_ws ? const_cast<float*>(fin) : static_cast<float*>(p->workspace);
    // the passes: one per axis, two for an 8192-point FFT axis
    int remaining = 0;
    for (int a = 0; a < 3; ++a)
      if ((axes >> a) & 1u) remaining += (p->amode[a] == DFT3D_FFT && p->fax[a].r8) ? 2 : 1;
    if (p->f16) DFT3D_CUDA(cudaMemsetAsync(p->d_amax, 0, 4 * sizeof(unsigned int), stream));
    const float* src = fin;
    int pos = 0;
    bool have_amax = false;     // whether the word d_amax[pos] holds the largest magnitude of `src`
    for (int a = 0; a < 3; ++a) {
      if (!((axes >> a) & 1u)) continue;
      float* dst = (remaining % 2 == 1) ? fout : ws;
      if (p->amode[a] == DFT3D_FFT && p->fax[a].r8) {
        float* dst2 = (remaining % 2 == 1) ? ws : fout;   // the second launch's target: the other cube
        if ((rc = fft_r8_first(p, a, src, dst, stream)) != DFT3D_OK) return rc;
        if ((rc = fft_r8_second(p, a, dst, dst2, stream)) != DFT3D_OK) return rc;
        src = dst2;
        remaining -= 2;
        ++pos;
        have_amax = false;
        continue;
      }
      if (p->amode[a] == DFT3D_FFT) {
        if ((rc = fft_axis_pass(p, a, src, dst, stream)) != DFT3D_OK) return rc;
        have_amax = false;
      } else {
        if (p->f16 && !have_amax) {
          // a KDFT pass with fp16 pieces scales by the largest magnitude of its input, which only a KDFT
          // predecessor records: measure it
          dft3d::amax_kernel<<<p->sm_count * 8, 256, 0, stream>>>(reinterpret_cast<const float4*>(src), points(p) / 2,
                                                                 p->d_amax + pos);
          DFT3D_CUDA(cudaGetLastError());
        }
        if ((rc = kdft_axis_pass(p, a, src, dst, p->n[0], stream, pos)) != DFT3D_OK) return rc;
        have_amax = true;
      }
      src = dst;
      ++pos;
      --remaining;
    }
    return DFT3D_OK;
  }
  if (p->mode == DFT3D_KDFT) {
    const long long g = p->group_planes;
    const long long plane_floats = p->n[1] * p->n[2] * 2;
    float* ws = p->in_is_ws ? const_cast<float*>(fin) : static_cast<float*>(p->workspace);
    if ((rc = prepare_scales(p, fin, stream)) != DFT3D_OK) return rc;
    // the last argument is the pass's position in the chain (fp16 pieces: every pass reads the largest magnitude its
    // predecessor recorded; a later group of planes may read a value that earlier groups already raised, which is
    // still an upper bound for its own data)
    if (axes == 7u) {
      // axis 0: in -> out; then per group of n0-planes: axis 1 out -> workspace, axis 2 workspace -> out
      if ((rc = kdft_axis_pass(p, 0, fin, fout, p->n[0], stream, 0)) != DFT3D_OK) return rc;
      for (long long a = 0; a < p->n[0]; a += g) {
        float* slab = fout + a * plane_floats;
        if ((rc = kdft_axis_pass(p, 1, slab, ws, g, stream, 1)) != DFT3D_OK) return rc;
        if ((rc = kdft_axis_pass(p, 2, ws, slab, g, stream, 2)) != DFT3D_OK) return rc;
      }
    } else if (axes == 6u) {
      // batch of 2D transforms: per group axis 1 in -> workspace, axis 2 workspace -> out
      for (long long a = 0; a < p->n[0]; a += g) {
        if ((rc = kdft_axis_pass(p, 1, fin + a * plane_floats, ws, g, stream, 0)) != DFT3D_OK) return rc;
        if ((rc = kdft_axis_pass(p, 2, ws, fout + a * plane_floats, g, stream, 1)) != DFT3D_OK) return rc;
      }
    } else if (axes == 3u || axes == 5u) {
      // axis 0 and one more: the other axis in -> workspace (whole cube), then axis 0 workspace -> out
      if ((rc = kdft_axis_pass(p, axes == 3u ? 1 : 2, fin, ws, p->n[0], stream, 0)) != DFT3D_OK) return rc;
      if ((rc = kdft_axis_pass(p, 0, ws, fout, p->n[0], stream, 1)) != DFT3D_OK) return rc;
    } else {
      const int a = axes == 1u ? 0 : (axes == 2u ? 1 : 2);
      if ((rc = kdft_axis_pass(p, a, fin, fout, p->n[0], stream, 0)) != DFT3D_OK) return rc;
    }
    return DFT3D_OK;
  }
  // FFT: the first transformed axis (last axis first) in -> out, the others in place on out (a CTA loads a group of
  // lines completely into shared memory before it stores any of their results, and groups are disjoint)
  if (axes == 7u && p->ws_slices && !p->knobs.fft_inplace) {
    float* ws = static_cast<float*>(p->workspace);
    const long long sub = p->n[2] / p->ws_slices;
    for (int h = 0; h < p->ws_slices; ++h) {
      if ((rc = fft_axis_pass(p, 0, fin, ws, stream, FFT_OUT_BLOCKED, h * sub, sub)) != DFT3D_OK) return rc;
      if ((rc = fft_axis_pass(p, 1, ws, fout, stream, FFT_IN_BLOCKED, h * sub, sub)) != DFT3D_OK) return rc;
    }
    return fft_axis_pass(p, 2, fout, fout, stream);   // in place: a CTA has its lines in shared memory before it stores them
  }
  if (axes == 7u && ((p->workspace && !p->ws_slices) || p->in_is_ws) && !p->knobs.fft_inplace) {
    // with a cube of workspace: axis 0 in -> out (blocked order: its far-apart rows are only read, never written
    // piecewise), axis 1 out -> workspace (natural order), axis 2 workspace -> out
    float* ws = p->in_is_ws ? const_cast<float*>(fin) : static_cast<float*>(p->workspace);
#ifdef DFT3D_PROFILE_WAITS
    if (const char* only = getenv("DFT3D_DEBUG_ONLY_PASS")) {   // diagnostic builds: one pass of the schedule alone
      const int k = atoi(only);
      if (k == 0) return fft_axis_pass(p, 0, fin, fout, stream, FFT_OUT_BLOCKED);
      if (k == 1) return fft_axis_pass(p, 1, fout, ws, stream, FFT_IN_BLOCKED);
      return fft_axis_pass(p, 2, ws, fout, stream);
    }
#endif
    if (p->fuse12) {
      // axis 0 in -> workspace (blocked order), then axes 1 and 2 in one launch: workspace -> ring (L2) -> out
      if ((rc = fft_axis_pass(p, 0, fin, ws, stream, FFT_OUT_BLOCKED)) != DFT3D_OK) return rc;
      return fft_fused12_pass(p, ws, fout, stream);
    }
    if ((rc = fft_axis_pass(p, 0, fin, fout, stream, FFT_OUT_BLOCKED)) != DFT3D_OK) return rc;
    if ((rc = fft_axis_pass(p, 1, fout, ws, stream, FFT_IN_BLOCKED)) != DFT3D_OK) return rc;
    return fft_axis_pass(p, 2, ws, fout, stream);
  }
  const float* src = fin;
  for (int a = 2; a >= 0; --a) {
    if (!((axes >> a) & 1u)) continue;
    if ((rc = fft_axis_pass(p, a, src, fout, stream)) != DFT3D_OK) return rc;
    src = fout;
  }
  return DFT3D_OK;
}

int dft3d_execute_host(dft3d_plan_t p, const void* host_in, void* host_out, void* cuda_stream) {
  if (!p) return fail(DFT3D_ERR_INVALID_ARG, "plan is NULL");
  if (!host_in || !host_out) return fail(DFT3D_ERR_INVALID_ARG, "host_in/host_out must not be NULL");
  const size_t bytes = size_t(points(p)) * 8;
  if (!p->host_in_dev) DFT3D_CUDA(cudaMalloc(&p->host_in_dev, bytes));
  if (!p->host_out_dev) DFT3D_CUDA(cudaMalloc(&p->host_out_dev, bytes));
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  DFT3D_CUDA(cudaMemcpyAsync(p->host_in_dev, host_in, bytes, cudaMemcpyHostToDevice, stream));
  int rc = dft3d_execute(p, p->host_in_dev, p->host_out_dev, cuda_stream);
  if (rc != DFT3D_OK) return rc;
  DFT3D_CUDA(cudaMemcpyAsync(host_out, p->host_out_dev, bytes, cudaMemcpyDeviceToHost, stream));
  DFT3D_CUDA(cudaStreamSynchronize(stream));
  return dft3d_plan_status(p);
}

int dft3d_execute_host_batch(dft3d_plan_t p, const void* const* host_in, void* const* host_out, int count,
                             void* cuda_stream) {
  if (!p) return fail(DFT3D_ERR_INVALID_ARG, "plan is NULL");
  if (count < 0 || (count > 0 && (!host_in || !host_out))) return fail(DFT3D_ERR_INVALID_ARG, "host_in/host_out/count");
  for (int i = 0; i < count; ++i)
    if (!host_in[i] || !host_out[i]) return fail(DFT3D_ERR_INVALID_ARG, "host_in[%d]/host_out[%d] must not be NULL", i, i);
  if (count == 0) return DFT3D_OK;
  const size_t bytes = size_t(points(p)) * 8;
  if (!p->host_in_dev) DFT3D_CUDA(cudaMalloc(&p->host_in_dev, bytes));
  if (!p->host_out_dev) DFT3D_CUDA(cudaMalloc(&p->host_out_dev, bytes));
  if (count > 1) {
    if (!p->host_in_dev2) DFT3D_CUDA(cudaMalloc(&p->host_in_dev2, bytes));
    if (!p->host_out_dev2) DFT3D_CUDA(cudaMalloc(&p->host_out_dev2, bytes));
  }
  if (!p->copy_in) DFT3D_CUDA(cudaStreamCreateWithFlags(&p->copy_in, cudaStreamNonBlocking));
  if (!p->copy_out) DFT3D_CUDA(cudaStreamCreateWithFlags(&p->copy_out, cudaStreamNonBlocking));
  for (int b = 0; b < 2; ++b) {
    if (!p->ev_in_ready[b]) DFT3D_CUDA(cudaEventCreateWithFlags(&p->ev_in_ready[b], cudaEventDisableTiming));
    if (!p->ev_done[b]) DFT3D_CUDA(cudaEventCreateWithFlags(&p->ev_done[b], cudaEventDisableTiming));
    if (!p->ev_out_free[b]) DFT3D_CUDA(cudaEventCreateWithFlags(&p->ev_out_free[b], cudaEventDisableTiming));
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  void* din[2] = {p->host_in_dev, p->host_in_dev2};
  void* dout[2] = {p->host_out_dev, p->host_out_dev2};
  // the copy streams start after whatever the caller's stream holds so far
  DFT3D_CUDA(cudaEventRecord(p->ev_done[0], stream));
  DFT3D_CUDA(cudaStreamWaitEvent(p->copy_in, p->ev_done[0], 0));
  DFT3D_CUDA(cudaStreamWaitEvent(p->copy_out, p->ev_done[0], 0));
  int rc = DFT3D_OK;
  for (int i = 0; i < count; ++i) {
    const int b = i & 1;
    // item i uses buffer pair b; its upload may start once item i-2 has been transformed out of in[b] ...
    if (i >= 2) DFT3D_CUDA(cudaStreamWaitEvent(p->copy_in, p->ev_done[b], 0));
    DFT3D_CUDA(cudaMemcpyAsync(din[b], host_in[i], bytes, cudaMemcpyHostToDevice, p->copy_in));
    DFT3D_CUDA(cudaEventRecord(p->ev_in_ready[b], p->copy_in));
    // ... its transform once the upload is there and item i-2's result has left out[b] ...
    DFT3D_CUDA(cudaStreamWaitEvent(stream, p->ev_in_ready[b], 0));
    if (i >= 2) DFT3D_CUDA(cudaStreamWaitEvent(stream, p->ev_out_free[b], 0));
    rc = dft3d_execute(p, din[b], dout[b], cuda_stream);
    if (rc != DFT3D_OK) break;
    DFT3D_CUDA(cudaEventRecord(p->ev_done[b], stream));
    // ... and its download once the transform is done (downloads run in order on their own stream)
    DFT3D_CUDA(cudaStreamWaitEvent(p->copy_out, p->ev_done[b], 0));
    DFT3D_CUDA(cudaMemcpyAsync(host_out[i], dout[b], bytes, cudaMemcpyDeviceToHost, p->copy_out));
    DFT3D_CUDA(cudaEventRecord(p->ev_out_free[b], p->copy_out));
  }
  // everything is done when the last download is: hand that back to the caller's stream, then wait for it
  DFT3D_CUDA(cudaStreamSynchronize(p->copy_in));
  DFT3D_CUDA(cudaStreamSynchronize(p->copy_out));
  DFT3D_CUDA(cudaStreamSynchronize(stream));
  if (rc != DFT3D_OK) return rc;
  return dft3d_plan_status(p);
}

int dft3d_plan_status(dft3d_plan_t p) {
  if (!p) return fail(DFT3D_ERR_INVALID_ARG, "plan is NULL");
  unsigned int word = 0;
  DFT3D_CUDA(cudaMemcpy(&word, p->d_status, sizeof(word), cudaMemcpyDeviceToHost));
  if (word != 0) return fail(DFT3D_ERR_DEVICE_TIMEOUT, "a kernel abandoned a bounded wait (code 0x%x)", word);
  return DFT3D_OK;
}

size_t dft3d_plan_workspace_bytes(dft3d_plan_t p) { return p ? p->workspace_bytes : 0; }

int dft3d_plan_launches(dft3d_plan_t p) {
  if (!p) return 0;
  const int count = int((p->axes & 1u) + ((p->axes >> 1) & 1u) + ((p->axes >> 2) & 1u));
  if (p->mode == DFT3D_AUTO) {
    int launches = 0;
    bool have_amax = false;
    for (int a = 0; a < 3; ++a) {
      if (!((p->axes >> a) & 1u)) continue;
      if (p->amode[a] == DFT3D_FFT) { launches += p->fax[a].r8 ? 2 : 1; have_amax = false; }
      else { launches += (p->f16 && !have_amax) ? 2 : 1; have_amax = true; }
    }
    return launches;
  }
  const int pre = (p->f16 && p->mode == DFT3D_KDFT) ? 1 : 0;   // the reduction that finds the largest input magnitude
  if (p->mode == DFT3D_KDFT && p->axes == 7u) return pre + int(1 + 2 * (p->n[0] / p->group_planes));
  if (p->mode == DFT3D_KDFT && p->axes == 6u) return pre + int(2 * (p->n[0] / p->group_planes));
  if (p->mode == DFT3D_FFT && p->ws_slices && !p->knobs.fft_inplace)
    return 2 * p->ws_slices + 1;   // two strided passes per slice, one contiguous
  if (p->mode == DFT3D_FFT && p->fuse12 && !p->knobs.fft_inplace) return 2;   // axis 0, then axes 1 and 2 together
  return pre + count;
}

int dft3d_plan_split(dft3d_plan_t p) {
  if (!p) return 0;
  return p->f16 ? DFT3D_SPLIT_FP16 : DFT3D_SPLIT_TF32;
}

int dft3d_plan_fft_split(dft3d_plan_t p, int axis, int* n1, int* n2) {
  if (!p || !n1 || !n2) return fail(DFT3D_ERR_INVALID_ARG, "plan, n1 and n2 must not be NULL");
  if (axis < 0 || axis > 2 || !((p->axes >> axis) & 1u) || p->amode[axis] != DFT3D_FFT)
    return fail(DFT3D_ERR_INVALID_ARG, "axis %d is not transformed in the FFT formulation by this plan", axis);
  *n1 = p->fax[axis].r8 ? 1024 : p->fax[axis].RX * p->fax[axis].R;
  *n2 = p->fax[axis].r8 ? 8 : p->fax[axis].R;
  return DFT3D_OK;
}

int dft3d_plan_destroy(dft3d_plan_t p) {
  if (!p) return DFT3D_OK;
  for (int a = 0; a < 3; ++a) {
    if (p->kax[a].d_w) cudaFree(p->kax[a].d_w);
    if (p->fax[a].d_w) cudaFree(p->fax[a].d_w);
    if (p->fax[a].d_tw) cudaFree(p->fax[a].d_tw);
    if (p->fax[a].d_tw2) cudaFree(p->fax[a].d_tw2);
    if (p->fax[a].d_tw8) cudaFree(p->fax[a].d_tw8);
  }
  if (p->workspace) cudaFree(p->workspace);
  if (p->ring) cudaFree(p->ring);
  if (p->d_fuse_counters) cudaFree(p->d_fuse_counters);
  if (p->d_status) cudaFree(p->d_status);
  if (p->d_amax) cudaFree(p->d_amax);
  if (p->d_profile) cudaFree(p->d_profile);
  if (p->host_in_dev) cudaFree(p->host_in_dev);
  if (p->host_out_dev) cudaFree(p->host_out_dev);
  if (p->host_in_dev2) cudaFree(p->host_in_dev2);
  if (p->host_out_dev2) cudaFree(p->host_out_dev2);
  for (int b = 0; b < 2; ++b) {
    if (p->ev_in_ready[b]) cudaEventDestroy(p->ev_in_ready[b]);
    if (p->ev_done[b]) cudaEventDestroy(p->ev_done[b]);
    if (p->ev_out_free[b]) cudaEventDestroy(p->ev_out_free[b]);
  }
  if (p->copy_in) cudaStreamDestroy(p->copy_in);
  if (p->copy_out) cudaStreamDestroy(p->copy_out);
  delete p;
  return DFT3D_OK;
}

}  // extern "C"
