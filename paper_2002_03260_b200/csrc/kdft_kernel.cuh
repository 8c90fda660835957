// One axis of the KDFT formulation (paper Section III-A, Eq. 12): the mode-n product of the data
// cube with that axis' N x N Vandermonde / DFT matrix, as a real GEMM on the 5th-generation
// tensor cores.
//
// Complex-as-real mapping.  With the data kept interleaved (re, im), a lane of the tile is one
// "line" of the cube along the transformed axis, seen as 2N reals  a[2j+q] (q = 0 re, 1 im), and
//     y[2k+p] = sum_{j,q} a[2j+q] * W[2k+p][2j+q],
//     W[2k][2j] = Re M[k][j],  W[2k][2j+1] = -Im M[k][j],  W[2k+1][2j] = Im M[k][j],  W[2k+1][2j+1] = Re M[k][j]
// is the complex product y_k = sum_j M[k][j] x_j with y again interleaved.  So every axis is the
// same real GEMM  D[128 lanes, 2N] = A[128 lanes, 2N] * W^T ; only the way a tile's lines are
// fetched and stored differs:
//   CONTIG  (last axis)        : a lane is a row of the (n0*n1) x (2*n2) float matrix.
//   STRIDED (axes 0 and 1)     : a lane is one complex column c of a [batch][j][c] view; the TMA box
//                                brings rows j of 128 neighbouring columns and the split step below
//                                transposes while it copies (no standalone transpose pass).
//
// fp32-level accuracy from TF32 tensor cores (Section II-A describes float32 accuracy from several
// reduced-precision pieces whose products are accumulated; here the pieces are TF32): x = x_hi + x_lo, W = W_hi + W_lo, and
//     D += x_hi*W_hi + x_lo*W_hi + x_hi*W_lo      (the x_lo*W_lo term is below fp32 rounding).
// W_hi/W_lo come pre-split from the float64 generator.  x_hi is the raw fp32 word (the tensor core
// ignores the low 13 mantissa bits, i.e. truncates), x_lo = x - trunc(x) rounded to TF32.
//
// Pipeline per CTA (persistent over tiles, one CTA per SM):
//   warp 0      TMA producer: W tile (both pieces, K-major, 128B swizzle) and the raw data tile
//   warps 4-7   split: shared memory -> registers -> (x_hi, x_lo) -> tensor memory (A operand)
//   warp 1      one thread issues tcgen05.mma kind::tf32, A from tensor memory, B from shared memory,
//               fp32 accumulator 128 x 256 in tensor memory
//   warps 8-15  epilogue: tcgen05.ld every chunk -> fp32 running sum in registers -> global stores
// All waits are bounded; a wait that gives up sets the status word and the CTA unwinds.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>
#include "ptx_sm100.cuh"

// registers per thread of each warp group after the split of the register file (sum x 128 = 65536)
#ifndef DFT3D_REGS_WG0
#define DFT3D_REGS_WG0 40
#define DFT3D_REGS_SPLIT 120
#define DFT3D_REGS_EPI 176
#endif

namespace dft3d {

enum : int { KDFT_CONTIG = 0, KDFT_STRIDED = 1 };

constexpr int kTileM = 128;         // lanes (lines) per tile
constexpr int kMaxTileN = 256;      // output reals per tile (128 complex outputs)
constexpr int kBlockK = 32;         // reals of the contraction per pipeline stage (128 bytes)
constexpr int kStagesB = 3;         // W stages in shared memory
constexpr int kStagesA = 2;         // raw data stages in shared memory
constexpr int kStagesT = 4;         // split data stages in tensor memory
constexpr int kAccCols = 256;       // accumulator columns in tensor memory
constexpr int kTmemCols = 512;
constexpr int kBytesStageB = 2 * kMaxTileN * kBlockK * 4;   // hi + lo
constexpr int kBytesStageA = kTileM * kBlockK * 4;
constexpr int kKdftThreads = 512;      // 4 warp groups: {producer, MMA, 2 idle}, split, epilogue x 2
constexpr int kEpilogueWarps = 8;
constexpr size_t kKdftSmemBytes = size_t(kStagesB) * kBytesStageB + size_t(kStagesA) * kBytesStageA + 1024 + 512;

constexpr long long kDefaultWaitClocks = 4000000000LL;   // about two seconds

// what a launch may override for tests of the give-up path (0 / 0 = the defaults)
struct WaitControl {
  long long limit_clocks;   // clock budget of every bounded wait; 0 = kDefaultWaitClocks
  int silent_producer;      // test only: the TMA producer issues nothing, so every wait of the CTA runs out
};

struct KdftParams {
  int k2;              // 2*N: real contraction length = real output length per line
  int bn;              // output reals per tile: min(256, 2N)
  int n_tiles;         // ceil(2N / bn)
  int chunk_kb;        // pipeline stages (of 32 reals) per tensor-core accumulation chain
  long long m_tiles;   // tiles along the lines
  // CONTIG
  long long rows;      // number of lines
  // STRIDED: view [batches][J = N][C] complex
  long long batches;
  long long C;
  int lpb;             // lanes per batch in a tile: min(128, C)
  int bpt;             // batches per tile: 128 / lpb
  long long c_tiles;   // ceil(C / lpb)
  float* out;
  unsigned int* status;  // device word, set non-zero when a wait gives up
  long long* profile;    // optional [grid][4] cycle counters of the MMA issuer (builds with DFT3D_PROFILE_WAITS)
  WaitControl wc;
};

struct KdftShared {
  uint64_t b_full[kStagesB], b_empty[kStagesB];
  uint64_t a_full[kStagesA], a_empty[kStagesA];
  uint64_t t_full[kStagesT], t_empty[kStagesT];
  uint64_t acc_full, acc_empty;
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;
};

__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                             long long limit = kDefaultWaitClocks) {
  const long long t0 = clock64();
  const uint32_t addr = ptx::smem_u32(bar);
  for (uint32_t spin = 0;; ++spin) {
    uint32_t done;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t"
        "}\n"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    if (done) return true;
    if ((spin & 0xff) == 0xff) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) return false;
    }
  }
}

// single-thread wait (producer, MMA issuer)
#define DFT3D_WAIT(bar, parity, code)                               \
  if (!bounded_wait((bar), (parity), &sh.abort_flag, sh.wait_limit)) {             \
    sh.abort_flag = 1;                                              \
    atomicCAS(p.status, 0u, (unsigned)(code));                      \
    goto role_done;                                                 \
  }
// whole-warp wait: the warp leaves together, so the .sync.aligned tensor-memory
// instructions that follow are never executed by a partial warp
#define DFT3D_WAIT_WARP(bar, parity, code)                                              \
  if (!__all_sync(0xffffffffu, bounded_wait((bar), (parity), &sh.abort_flag, sh.wait_limit) ? 1 : 0)) { \
    sh.abort_flag = 1;                                                                  \
    atomicCAS(p.status, 0u, (unsigned)(code));                                          \
    goto role_done;                                                                     \
  }

template <int MODE>
__global__ void __launch_bounds__(kKdftThreads, 1)
kdft_axis_kernel(const __grid_constant__ CUtensorMap map_data, const __grid_constant__ CUtensorMap map_w,
                 const KdftParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_b = smem;
  uint8_t* smem_a = smem + size_t(kStagesB) * kBytesStageB;
  KdftShared& sh = *reinterpret_cast<KdftShared*>(smem_a + size_t(kStagesA) * kBytesStageA);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < kStagesB; ++i) { ptx::mbar_init(&sh.b_full[i], 1); ptx::mbar_init(&sh.b_empty[i], 1); }
    for (int i = 0; i < kStagesA; ++i) { ptx::mbar_init(&sh.a_full[i], 1); ptx::mbar_init(&sh.a_empty[i], 4); }
    for (int i = 0; i < kStagesT; ++i) { ptx::mbar_init(&sh.t_full[i], 4); ptx::mbar_init(&sh.t_empty[i], 1); }
    ptx::mbar_init(&sh.acc_full, 1);
    ptx::mbar_init(&sh.acc_empty, kEpilogueWarps);
    sh.abort_flag = 0;
    sh.wait_limit = p.wc.limit_clocks > 0 ? p.wc.limit_clocks : kDefaultWaitClocks;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&sh.tmem_base, kTmemCols);
    ptx::tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&map_data);
    ptx::prefetch_tensormap(&map_w);
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  const long long total_tiles = p.m_tiles * p.n_tiles;
  const int num_kb = (p.k2 + kBlockK - 1) / kBlockK;   // a ragged last stage is zero-filled by TMA on both operands
  const uint32_t bytes_b = 2u * uint32_t(p.bn) * kBlockK * 4u;

  if (warp < 4) {
    // warp group 0: producer and MMA issuer need few registers; hand the rest to the epilogue
    ptx::setmaxnreg_dec<DFT3D_REGS_WG0>();
    if (warp == 0) {
      // ------------------------------------------------------------ TMA producer
      if (lane == 0 && !p.wc.silent_producer) {
        uint32_t ib = 0, ia = 0;   // running stage counters
        for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
          const long long mt = t / p.n_tiles;
          const int nt = int(t % p.n_tiles);
          int ax = 0, ay = 0, az = 0;
          if (MODE == KDFT_CONTIG) {
            ay = int(mt * kTileM);
          } else {
            const long long ct = mt % p.c_tiles;
            const long long bt = mt / p.c_tiles;
            ax = int(ct * p.lpb * 2);
            az = int(bt * p.bpt);
          }
          for (int kb = 0; kb < num_kb; ++kb) {
            {
              const uint32_t s = ib % kStagesB, ph = (ib / kStagesB) & 1;
              DFT3D_WAIT(&sh.b_empty[s], ph ^ 1, 0x101);
              ptx::mbar_arrive_expect_tx(&sh.b_full[s], bytes_b);
              ptx::tma_load_3d(smem_b + size_t(s) * kBytesStageB, &map_w, &sh.b_full[s], kb * kBlockK, nt * p.bn, 0);
              ++ib;
            }
            {
              const uint32_t s = ia % kStagesA, ph = (ia / kStagesA) & 1;
              DFT3D_WAIT(&sh.a_empty[s], ph ^ 1, 0x102);
              ptx::mbar_arrive_expect_tx(&sh.a_full[s], kBytesStageA);
              if (MODE == KDFT_CONTIG)
                ptx::tma_load_2d(smem_a + size_t(s) * kBytesStageA, &map_data, &sh.a_full[s], kb * kBlockK, ay);
              else
                ptx::tma_load_3d(smem_a + size_t(s) * kBytesStageA, &map_data, &sh.a_full[s], ax, kb * (kBlockK / 2), az);
              ++ia;
            }
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------ MMA issuer
      if (lane == 0) {
        const uint32_t idesc = ptx::make_idesc_tf32(kTileM, p.bn);
        uint32_t ib = 0, it = 0, chunk_count = 0;
#ifdef DFT3D_PROFILE_WAITS
        long long w_acc = 0, w_b = 0, w_t = 0, t_begin = clock64(), tq;
#define PW_BEGIN tq = clock64();
#define PW_END(v) v += clock64() - tq;
#else
#define PW_BEGIN
#define PW_END(v)
#endif
        for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
          for (int kb = 0; kb < num_kb; ++kb) {
            const bool chunk_first = (kb % p.chunk_kb) == 0;
            if (chunk_first) {
              // the tensor-core accumulator restarts from zero every chunk (see the epilogue)
              PW_BEGIN
              DFT3D_WAIT(&sh.acc_empty, (chunk_count & 1) ^ 1, 0x201);
              PW_END(w_acc)
              ptx::tc_fence_after();
            }
            const uint32_t sb = ib % kStagesB, phb = (ib / kStagesB) & 1;
            const uint32_t st = it % kStagesT, pht = (it / kStagesT) & 1;
            PW_BEGIN
            DFT3D_WAIT(&sh.b_full[sb], phb, 0x202);
            PW_END(w_b)
            PW_BEGIN
            DFT3D_WAIT(&sh.t_full[st], pht, 0x203);
            PW_END(w_t)
            ptx::tc_fence_after();
            const uint32_t b_hi = ptx::smem_u32(smem_b + size_t(sb) * kBytesStageB);
            const uint32_t b_lo = b_hi + uint32_t(p.bn) * kBlockK * 4u;
            const uint32_t a_hi = tmem + kAccCols + st * 64;
            const uint32_t a_lo = a_hi + 32;
#pragma unroll
            for (int k = 0; k < kBlockK / 8; ++k) {
              const uint64_t dhi = ptx::make_kmajor_sw128_desc(b_hi + k * 32);
              const uint64_t dlo = ptx::make_kmajor_sw128_desc(b_lo + k * 32);
              ptx::mma_tf32_ts(tmem, a_hi + k * 8, dhi, idesc, (k != 0 || !chunk_first) ? 1u : 0u);
              ptx::mma_tf32_ts(tmem, a_lo + k * 8, dhi, idesc, 1);
              ptx::mma_tf32_ts(tmem, a_hi + k * 8, dlo, idesc, 1);
            }
            ptx::tc_commit(&sh.b_empty[sb]);
            ptx::tc_commit(&sh.t_empty[st]);
            ++ib;
            ++it;
            if ((kb + 1) % p.chunk_kb == 0 || kb + 1 == num_kb) {
              ptx::tc_commit(&sh.acc_full);
              ++chunk_count;
            }
          }
        }
#ifdef DFT3D_PROFILE_WAITS
        if (p.profile) {
          p.profile[blockIdx.x * 4 + 0] = clock64() - t_begin;
          p.profile[blockIdx.x * 4 + 1] = w_acc;
          p.profile[blockIdx.x * 4 + 2] = w_b;
          p.profile[blockIdx.x * 4 + 3] = w_t;
        }
#endif
      }
    }
  } else if (warp < 8) {
    // ------------------------------------------------------------ split: smem -> (hi, lo) -> tensor memory
    ptx::setmaxnreg_dec<DFT3D_REGS_SPLIT>();
    const int q = warp & 3;                 // lane quarter this warp may touch in tensor memory
    const int m = q * 32 + lane;            // lane of the tile
    const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16);
    int strided_off = 0;                    // float2 index of (j = 0) for this lane in a STRIDED stage
    if (MODE == KDFT_STRIDED) strided_off = (m / p.lpb) * (kBlockK / 2) * p.lpb + (m % p.lpb);
    uint32_t ia = 0, it = 0;
    for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const uint32_t sa = ia % kStagesA, pha = (ia / kStagesA) & 1;
        const uint32_t st = it % kStagesT, pht = (it / kStagesT) & 1;
        DFT3D_WAIT_WARP(&sh.a_full[sa], pha, 0x301);
        uint32_t x[32];
        const uint8_t* stage = smem_a + size_t(sa) * kBytesStageA;
        if (MODE == KDFT_CONTIG) {
          const uint4* rowp = reinterpret_cast<const uint4*>(stage + m * 128);
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 v = rowp[c ^ (m & 7)];
            x[4 * c] = v.x; x[4 * c + 1] = v.y; x[4 * c + 2] = v.z; x[4 * c + 3] = v.w;
          }
        } else {
          const uint2* colp = reinterpret_cast<const uint2*>(stage) + strided_off;
#pragma unroll
          for (int j = 0; j < kBlockK / 2; ++j) {
            const uint2 v = colp[j * p.lpb];
            x[2 * j] = v.x; x[2 * j + 1] = v.y;
          }
        }
        // the stage is refilled by TMA (async proxy): order this thread's reads before that write
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.a_empty[sa]);
        uint32_t lo[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float xf = __uint_as_float(x[i]);
          const float hi = __uint_as_float(x[i] & 0xffffe000u);
          const float r = xf - hi;                               // exact
          lo[i] = (__float_as_uint(r) + 0x1000u) & 0xffffe000u;  // round to TF32
        }
        DFT3D_WAIT_WARP(&sh.t_empty[st], pht ^ 1, 0x302);
        ptx::tc_fence_after();
        ptx::tmem_st_32x32(lane_addr + kAccCols + st * 64, x);
        ptx::tmem_st_32x32(lane_addr + kAccCols + st * 64 + 32, lo);
        ptx::tc_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.t_full[st]);
        ++ia;
        ++it;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (8 warps)
    // The tensor core adds into its fp32 accumulator with truncation, a bias that grows with the
    // number of MMAs chained on one accumulator.  So the chain is cut every `chunk_kb` stages: the
    // partial sum is pulled into registers and summed there in round-to-nearest fp32, and the tensor
    // core restarts from zero.
    ptx::setmaxnreg_inc<DFT3D_REGS_EPI>();
    const int q = warp & 3;
    const int half = (warp - 8) >> 2;        // which 128 columns of the 256-wide accumulator
    const int m = q * 32 + lane;
    const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16) + half * 128;
    const bool cols_active = half * 128 < p.bn;
    const int chunks_per_tile = (num_kb + p.chunk_kb - 1) / p.chunk_kb;
    uint32_t chunk_count = 0;
    for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      const long long mt = t / p.n_tiles;
      const int nt = int(t % p.n_tiles);
      float acc[128];
#pragma unroll
      for (int i = 0; i < 128; ++i) acc[i] = 0.0f;
      for (int c = 0; c < chunks_per_tile; ++c, ++chunk_count) {
        DFT3D_WAIT_WARP(&sh.acc_full, chunk_count & 1, 0x401);
        ptx::tc_fence_after();
        if (cols_active) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint32_t v[32];
            ptx::tmem_ld_32x32(lane_addr + g * 32, v);
            ptx::tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[g * 32 + i] += __uint_as_float(v[i]);
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.acc_empty);
      }
      // ---- store this lane's 128 reals
      const int c0 = nt * p.bn + half * 128;   // first real output column held by this thread
      if (cols_active && c0 < p.k2) {
        if (MODE == KDFT_CONTIG) {
          const long long row = mt * kTileM + m;
          if (row < p.rows) {
            float4* dst = reinterpret_cast<float4*>(p.out + row * (long long)p.k2 + c0);
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + 4 * i < p.k2) dst[i] = make_float4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
          }
        } else {
          const long long ct = mt % p.c_tiles;
          const long long bt = mt / p.c_tiles;
          const long long batch = bt * p.bpt + m / p.lpb;
          const long long cc = ct * p.lpb + (m % p.lpb);
          if (batch < p.batches && cc < p.C) {
            const long long J = p.k2 / 2;
            const long long k_stride = 2 * p.C;
            float* dst = p.out + 2 * ((batch * J + c0 / 2) * p.C + cc);
#pragma unroll
            for (int i = 0; i < 64; ++i)
              if (c0 / 2 + i < J) *reinterpret_cast<float2*>(dst + i * k_stride) = make_float2(acc[2 * i], acc[2 * i + 1]);
          }
        }
      }
    }
  }

role_done:
  if (warp == 0 && lane == 0 && sh.abort_flag) {
    // give loads that were already issued a bounded chance to land before the CTA goes away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) { }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, kTmemCols);
}

#undef DFT3D_WAIT
#undef DFT3D_WAIT_WARP

}  // namespace dft3d
