// One axis of the FFT formulation (paper Section III-B, Eq. 14-18) as ONE fused kernel: with the line
// index split as n = R*l + beta and the output index as k = k1 + R*k2 (N = R*R),
//
//   stage 1   B[k1][beta] = sum_l  F_R[k1][l] * x[R*l + beta]          (the "local transform" of Eq. 18, as a GEMM)
//   twiddle   C[k1][beta] = B[k1][beta] * exp(s*2*pi*i*k1*beta/N)      (the phase adjustment, outer factor of Eq. 17)
//   stage 2   X[k1 + R*k2] = sum_beta F_R[k2][beta] * C[k1][beta]      (second GEMM; stored in natural order)
//
// The intermediate never leaves the SM: stage 1 accumulates in tensor memory, the twiddle is applied
// in the registers of the warps that drain that accumulator, and the result is written to shared memory
// directly in the operand layout stage 2's MMA reads.  HBM traffic is one read and one write of the data.
//
// Both stages use the same complex-as-real mapping as the KDFT kernel (interleaved re/im, real 2R x 2R
// matrix W).  fp32 accuracy from TF32 as in the KDFT kernel: x = hi + lo, W = W_hi + W_lo and three MMAs per
// K step (hi*hi, lo*hi, hi*lo) into one 2R-column accumulator.  A chain is at most 24 MMAs long, so the
// truncation bias of the tensor-core accumulator stays far below fp32 rounding.
//
// Tile geometry.  An "M-tile" is 128 accumulator lanes.
//   stage 1 lanes = (line g, beta)  : 128/R lines of the tile, all beta
//   stage 2 lanes = (line g, k1)    : the same lines, all k1
//   CONTIG  (last axis): a shared-memory stage holds 128/R whole lines (one M-tile), loaded as contiguous rows.
//   STRIDED (axes 0, 1): a stage holds all N rows of 16 neighbouring lines (128-byte rows, 128B swizzle), i.e.
//                        R/8 M-tiles; loads and stores touch 128-byte / 32-byte contiguous pieces.
//
// Lengths N = 2*R*R (512, 2048) take one more application of Eq. 17 with P = N/2: the split warps first form
//   a[m] = x[m] + x[m + N/2],   b[m] = (x[m] - x[m + N/2]) * exp(s*2*pi*i*m/N),   m < R*R
// (a radix-2 butterfly on the CUDA cores), treat a and b as two lines of length R*R, and the final store
// interleaves them: X[2k] from a, X[2k+1] from b.
//
// Warp roles (512 threads): warp 0 TMA producer, warps 1 and 2 MMA issuers (stage 1, stage 2), warps 4-7 split (smem -> hi/lo -> tensor
// memory), warps 8-15 drain stage 1 (+twiddle, write stage-2 operand; two groups, 16 values of k1 each),
// warps 16-19 drain stage 2 (+store).
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>
#include "ptx_sm100.cuh"
#include "kdft_kernel.cuh"   // bounded_wait

namespace dft3d {

enum : int { FFT_CONTIG = 0, FFT_STRIDED = 1 };

constexpr int kFftThreads = 640;      // 5 warp groups: {producer, 2 MMA issuers}, split, drain 1 (x2), drain 2
// STRIDED stages hold COLS neighbouring lines: 16 (128-byte rows, 128B swizzle) or 8 (64-byte rows, 64B swizzle)
// STAGE_OUT (STRIDED only): results go back into the raw stage they came from (each M-tile owns its columns there) and
//   leave as full rows through TMA stores, instead of 32-byte pieces from registers; pays off when the rows are so far
//   apart that every piece costs an address translation (1024^3 axis 0: 11.0 ms with direct stores, 3.7 ms without
//   any stores)
// NB2 = buffers of the stage-2 operand (2 lets drain 1 write the next M-tile while stage 2 still reads this one)
constexpr int kFftTmemD1 = 0, kFftTmemD2 = 128, kFftTmemA1 = 256;   // tensor-memory column map (A1: two buffers of 128)

struct FftParams {
  int N;                 // RX*R*R
  int raw_stages;        // stages in the raw ring
  int stage_bytes;       // bytes of one raw stage
  int mtiles_per_stage;  // CONTIG 1, STRIDED 16/(128/R)
  long long num_stages;  // work items (stages) in the whole pass
  // CONTIG
  long long rows;        // number of lines
  // STRIDED: view [batches][N][C] complex
  long long C;
  long long c_tiles;     // C / COLS
  int l2_prefetch;       // STRIDED: prefetch the next stage's rows into L2
  // Blocked intermediate layout T[n2 tile][i1][k0][COLS] (one contiguous block [k0][COLS] per axis-0 stage), used
  // between the axis-0 and the axis-1 pass of a 3D transform so that the far-apart rows of axis 0 are only ever READ
  // piecewise, and so that the n1 rows an axis-1 stage gathers lie close together (one block apart, not a plane apart):
  int out_blocked;       // the stage of column tile ct = i1*blk_tiles + n2tile goes to block n2tile*blk_rows + i1 of T
  int blk_tiles;         // out_blocked: n2 / COLS
  int blk_rows;          // out_blocked: n1
  int blk_ratio;         // in_blocked: columns of a block of T / COLS of this pass
  int in_blocked;        // load rows from T through a 4D map {COLS, k0, i1, n2 tile}; batch = k0
  // fp16-piece kernel: a pass over a slice [n2_off, n2_off + n2_sub) of the last axis (the cube in halves through a
  // half-cube workspace).  Column tile ct of the slice is tile ct % col_tiles_row of row ct / col_tiles_row:
  int col_tiles_row;     // 0: the columns of a batch are contiguous (no slice); else n2_sub / COLS
  long long col_pitch;   // natural input, sliced: columns per row of the full array (n2)
  long long col_off;     // natural input, sliced: first column of the slice (n2_off)
  long long out_pitch;   // natural output: columns per output row (C, or n2 when the pass writes a slice of the full array)
  long long out_off;     // natural output: first column (0, or n2_off)
  int blk_pair;          // fp16-piece kernel, stages narrower than 128 bytes: P = 128 / (8*COLS) rows i1 share the lines of
                         // T, T[n2 tile][i1 / P][k0][i1 % P][COLS], so that the axis-1 pass reads whole 128-byte lines
                         // (5D map {COLS, i1 % P, k0, i1 / P, n2 tile}); 1 otherwise
  const float2* twiddle; // [R][R] complex64, T[k1][beta] (times 1/RX for a scaled inverse)
  const float2* twiddle2;// RX == 2: [R*R] complex64, exp(s*2*pi*i*m/N)
  float* out;
  unsigned int* status;
  long long* profile;    // optional cycle counters (builds with DFT3D_PROFILE_WAITS): [grid][16][8]
  WaitControl wc;
  long long fuse_stages_per_plane;   // two-axes launch (fp16-piece kernel): stages of this pass per n0-plane
};

struct FftShared {
  uint64_t raw_full[4], raw_empty[4];
  uint64_t a1_full[2], a1_empty[2];
  uint64_t d1_full, d1_empty;
  uint64_t a2_full[2], a2_empty[2];
  uint64_t d2_full, d2_empty;
  uint64_t w_full;
  uint64_t out_ready;      // STAGE_OUT: the four drain-2 warps have written the stage's last M-tile
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;
};

// shared memory: [W: 2 pieces x 2R/32 panels of 2R rows x 128 B] [A2: hi panels, lo panels] [raw ring] [barriers]
__host__ __device__ constexpr int fft_w_bytes(int R) { return (2 * R / 32) * 4 * R * 128; }
__host__ __device__ constexpr int fft_a2_piece_bytes(int R) { return (2 * R / 32) * 128 * 128; }
// the stage-2 operand has NB2 = 1 or 2 buffers; with two of them for R = 32 the raw ring shrinks to 64 KB
__host__ __device__ constexpr int fft_raw_bytes(int R, int NB2) { return (R == 32 && NB2 == 2) ? 64 * 1024 : 128 * 1024; }
__host__ __device__ constexpr size_t fft_smem_bytes(int R, int NB2) {
  return size_t(fft_w_bytes(R)) + size_t(2 * NB2) * fft_a2_piece_bytes(R) + fft_raw_bytes(R, NB2) + 1024 + 512;
}

#ifdef DFT3D_PROFILE_WAITS
#define FFT_PROF_BEGIN const long long prof_t0_ = clock64();
#define FFT_PROF_END(code) prof_wait[(code) >> 8] [(code) & 7] += clock64() - prof_t0_;
#else
#define FFT_PROF_BEGIN
#define FFT_PROF_END(code)
#endif
#define FFT_WAIT(bar, parity, code)                                 \
  {                                                                 \
    FFT_PROF_BEGIN                                                  \
    if (!bounded_wait((bar), (parity), &sh.abort_flag, sh.wait_limit)) {           \
      sh.abort_flag = 1;                                            \
      atomicCAS(p.status, 0u, (unsigned)(code));                    \
      goto role_done;                                               \
    }                                                               \
    FFT_PROF_END(code)                                              \
  }
#define FFT_WAIT_WARP(bar, parity, code)                                                  \
  {                                                                                       \
    FFT_PROF_BEGIN                                                                        \
    if (!__all_sync(0xffffffffu, bounded_wait((bar), (parity), &sh.abort_flag, sh.wait_limit) ? 1 : 0)) { \
      sh.abort_flag = 1;                                                                  \
      atomicCAS(p.status, 0u, (unsigned)(code));                                          \
      goto role_done;                                                                     \
    }                                                                                     \
    FFT_PROF_END(code)                                                                    \
  }

template <int MODE, int R, int RX, int COLS, int NB2, int STAGE_OUT>
__global__ void __launch_bounds__(kFftThreads, 1)
fft_axis_kernel(const __grid_constant__ CUtensorMap map_data, const __grid_constant__ CUtensorMap map_w,
                const __grid_constant__ CUtensorMap map_out, const FftParams p) {
  extern __shared__ uint8_t smem_raw_[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_) + 1023) & ~uintptr_t(1023));
  constexpr int K = 2 * R;             // reals per contraction
  constexpr int NB = 2 * R;            // MMA N: the 2R output reals (k, re/im) of one stage
  constexpr int kWPiece = (K / 32) * NB * 128;   // bytes of one table piece in shared memory
  constexpr int panels = K / 32;
  uint8_t* smem_w = smem;
  uint8_t* smem_a2 = smem_w + fft_w_bytes(R);
  constexpr int a2_piece = fft_a2_piece_bytes(R);
  uint8_t* smem_rawring = smem_a2 + 2 * NB2 * a2_piece;     // A2 buffer i = [hi piece][lo piece] at i * 2 * a2_piece
  FftShared& sh = *reinterpret_cast<FftShared*>(smem_rawring + fft_raw_bytes(R, NB2));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef DFT3D_PROFILE_WAITS
  long long prof_wait[16][8];
  for (int i = 0; i < 16; ++i) for (int j = 0; j < 8; ++j) prof_wait[i][j] = 0;
  const long long prof_start = clock64();
#endif
  constexpr int SL = 128 / R;          // lines of length R*R per M-tile (sub-lines when RX == 2)
  constexpr int Lg = SL / RX;          // lines of the cube per M-tile
  constexpr int NL = R * R;            // length of a (sub-)line
  constexpr int kRowBytes = COLS * 8;  // STRIDED: bytes of one row of a raw stage

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) {
      ptx::mbar_init(&sh.raw_full[i], 1);
      ptx::mbar_init(&sh.raw_empty[i], 4 * p.mtiles_per_stage + (STAGE_OUT ? 1 : 0));
    }
    ptx::mbar_init(&sh.out_ready, 4);
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&sh.a1_full[i], 4); ptx::mbar_init(&sh.a1_empty[i], 1); }
    ptx::mbar_init(&sh.d1_full, 1); ptx::mbar_init(&sh.d1_empty, 4 * (K / 32));
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&sh.a2_full[i], 4 * (K / 32)); ptx::mbar_init(&sh.a2_empty[i], 1); }
    ptx::mbar_init(&sh.d2_full, 1); ptx::mbar_init(&sh.d2_empty, 4);
    ptx::mbar_init(&sh.w_full, 1);
    sh.abort_flag = 0;
    sh.wait_limit = p.wc.limit_clocks > 0 ? p.wc.limit_clocks : kDefaultWaitClocks;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&sh.tmem_base, 512);
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

  // this CTA's share of the stages, and the M-tiles in them
  long long my_stages = 0;
  if ((long long)blockIdx.x < p.num_stages) my_stages = (p.num_stages - 1 - blockIdx.x) / gridDim.x + 1;
  const long long my_mtiles = my_stages * p.mtiles_per_stage;

  // 640 threads x 96 registers: every role fits its share, so the register file is not re-split here

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      ptx::mbar_arrive_expect_tx(&sh.w_full, uint32_t(fft_w_bytes(R)));
      for (int pn = 0; pn < 2 * panels; ++pn)       // [piece][panel][2R rows][32 floats]
        ptx::tma_load_2d(smem_w + pn * NB * 128, &map_w, &sh.w_full, 0, pn * NB);
      long long i = 0;
      for (long long sidx = blockIdx.x; sidx < p.num_stages; sidx += gridDim.x, ++i) {
        const uint32_t s = uint32_t(i % p.raw_stages), ph = uint32_t(i / p.raw_stages) & 1;
        FFT_WAIT(&sh.raw_empty[s], ph ^ 1, 0x501);
        ptx::mbar_arrive_expect_tx(&sh.raw_full[s], uint32_t(p.stage_bytes));
        uint8_t* dst = smem_rawring + size_t(s) * p.stage_bytes;
        if (MODE == FFT_CONTIG) {
          ptx::tma_load_3d(dst, &map_data, &sh.raw_full[s], 0, 0, int(sidx * Lg));
        } else {
          const long long ct = sidx % p.c_tiles, bt = sidx / p.c_tiles;
          for (int r0 = 0; r0 < p.N; r0 += 256) {
            if (p.in_blocked)
              ptx::tma_load_4d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s],
                               int(ct % p.blk_ratio) * 2 * COLS, int(bt), r0, int(ct / p.blk_ratio));
            else
              ptx::tma_load_3d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s], int(ct * 2 * COLS), r0, int(bt));
          }
          // the ring is short on the strided axes (one or two stages), so the loads of the next stage cannot be
          // issued yet; pull its rows into L2 meanwhile (rows are far apart: this also absorbs the TLB misses)
          const long long nidx = sidx + gridDim.x;
          if (p.l2_prefetch && nidx < p.num_stages) {
            const long long nct = nidx % p.c_tiles, nbt = nidx / p.c_tiles;
            for (int r0 = 0; r0 < p.N; r0 += 256)
              ptx::tma_prefetch_l2_3d(&map_data, int(nct * 2 * COLS), r0, int(nbt));
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer, stage 1 (A from tensor memory)
    // Two issuing threads (this one and warp 2 for stage 2) keep the tensor pipe fed: every operand of the
    // unrolled MMAs below is loop-invariant (the two A1 buffers alternate, hence the unroll by two), so the
    // issue loop is a handful of instructions per MMA.
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_tf32(128, NB);
      const uint32_t w_addr = ptx::smem_u32(smem_w);
      uint64_t wh[K / 8], wl[K / 8];                 // loop-invariant operand descriptors, kept in registers
#pragma unroll
      for (int k8 = 0; k8 < K / 8; ++k8) {
        wh[k8] = ptx::make_kmajor_sw128_desc(w_addr + (k8 >> 2) * NB * 128 + (k8 & 3) * 32);
        wl[k8] = ptx::make_kmajor_sw128_desc(w_addr + kWPiece + (k8 >> 2) * NB * 128 + (k8 & 3) * 32);
      }
      FFT_WAIT(&sh.w_full, 0, 0x601);
      for (long long t = 0; t < my_mtiles; t += 2) {
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          if (t + b < my_mtiles) {
            const uint32_t phb = uint32_t(t >> 1) & 1;
            FFT_WAIT(&sh.a1_full[b], phb, 0x602);
            FFT_WAIT(&sh.d1_empty, uint32_t(b) ^ 1, 0x603);
            ptx::tc_fence_after();
            const uint32_t a_hi = tmem + kFftTmemA1 + b * 128, a_lo = a_hi + K;
#pragma unroll
            for (int k8 = 0; k8 < K / 8; ++k8) {   // small products first: each addition into the accumulator
              ptx::mma_tf32_ts(tmem + kFftTmemD1, a_lo + k8 * 8, wh[k8], idesc, k8 != 0);   // truncates to its ulp
              ptx::mma_tf32_ts(tmem + kFftTmemD1, a_hi + k8 * 8, wl[k8], idesc, 1);
            }
#pragma unroll
            for (int k8 = 0; k8 < K / 8; ++k8) ptx::mma_tf32_ts(tmem + kFftTmemD1, a_hi + k8 * 8, wh[k8], idesc, 1);
            ptx::tc_commit(&sh.a1_empty[b]);
            ptx::tc_commit(&sh.d1_full);
          }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ MMA issuer, stage 2 (A from shared memory)
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_tf32(128, NB);
      const uint32_t w_addr = ptx::smem_u32(smem_w);
      const uint32_t a2_addr = ptx::smem_u32(smem_a2);
      uint64_t wh[K / 8], wl[K / 8], ah[K / 8], al[K / 8];
#pragma unroll
      for (int k8 = 0; k8 < K / 8; ++k8) {
        const uint32_t off = (k8 >> 2) * 128 * 128 + (k8 & 3) * 32;
        wh[k8] = ptx::make_kmajor_sw128_desc(w_addr + (k8 >> 2) * NB * 128 + (k8 & 3) * 32);
        wl[k8] = ptx::make_kmajor_sw128_desc(w_addr + kWPiece + (k8 >> 2) * NB * 128 + (k8 & 3) * 32);
        ah[k8] = ptx::make_kmajor_sw128_desc(a2_addr + off);
        al[k8] = ptx::make_kmajor_sw128_desc(a2_addr + a2_piece + off);
      }
      constexpr uint64_t kBufStep = uint64_t(2 * a2_piece) >> 4;   // second A2 buffer, in descriptor address units
      FFT_WAIT(&sh.w_full, 0, 0x611);
      for (long long t = 0; t < my_mtiles; ++t) {
        const uint32_t bi = uint32_t(t % NB2), u = uint32_t(t / NB2);
        FFT_WAIT(&sh.a2_full[bi], u & 1, 0x604);
        FFT_WAIT(&sh.d2_empty, (uint32_t(t) & 1) ^ 1, 0x605);
        ptx::tc_fence_after();
        const uint64_t bstep = bi ? kBufStep : 0;
#pragma unroll
        for (int k8 = 0; k8 < K / 8; ++k8) {   // small products first, as in stage 1
          ptx::mma_tf32_ss(tmem + kFftTmemD2, al[k8] + bstep, wh[k8], idesc, k8 != 0);
          ptx::mma_tf32_ss(tmem + kFftTmemD2, ah[k8] + bstep, wl[k8], idesc, 1);
        }
#pragma unroll
        for (int k8 = 0; k8 < K / 8; ++k8) ptx::mma_tf32_ss(tmem + kFftTmemD2, ah[k8] + bstep, wh[k8], idesc, 1);
        ptx::tc_commit(&sh.a2_empty[bi]);
        ptx::tc_commit(&sh.d2_full);
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ------------------------------------------------------------ split: raw lines -> (hi, lo) -> tensor memory A1
    const int q = warp & 3;
    const int m = q * 32 + lane;
    const int sl = m / R, beta = m % R;           // stage-1 lane = (sub-line sl, beta), beta fastest
    const int g = sl / RX, bsel = sl % RX;        // line of the cube within the M-tile; which butterfly output
    const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16);
    long long t = 0;
    for (long long i = 0; i < my_stages; ++i) {
      const uint32_t s = uint32_t(i % p.raw_stages), phs = uint32_t(i / p.raw_stages) & 1;
      FFT_WAIT_WARP(&sh.raw_full[s], phs, 0x701);
      const uint8_t* stage = smem_rawring + size_t(s) * p.stage_bytes;
      for (int mt = 0; mt < p.mtiles_per_stage; ++mt, ++t) {
        // element m = R*l + beta of this lane's line sits at base + l*stride; its butterfly partner `half` further
        uint32_t base, stride, half;
        if (MODE == FFT_CONTIG) {
          base = uint32_t(g * p.N + beta) * 8u;
          stride = uint32_t(R) * 8u;
          half = uint32_t(NL) * 8u;
        } else {
          const int c = mt * Lg + g;                // column within the stage
          const uint32_t swz = (COLS == 16) ? uint32_t(beta & 7) : uint32_t((beta >> 1) & 3);   // TMA swizzle of the row
          base = uint32_t(beta) * kRowBytes + ((uint32_t(c >> 1) ^ swz) << 4) + uint32_t(c & 1) * 8u;
          stride = uint32_t(R) * kRowBytes;
          half = uint32_t(NL) * kRowBytes;
        }
        const uint32_t b = uint32_t(t & 1), phb = uint32_t(t >> 1) & 1;
        FFT_WAIT_WARP(&sh.a1_empty[b], phb ^ 1, 0x702);
        ptx::tc_fence_after();
        const uint32_t a_hi = lane_addr + kFftTmemA1 + b * 128, a_lo = a_hi + K;
#pragma unroll
        for (int l0 = 0; l0 < R; l0 += 16) {      // 16 complex = 32 reals per tensor-memory store
          uint32_t x[32], lo[32];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const uint2 v = *reinterpret_cast<const uint2*>(stage + base + uint32_t(l0 + j) * stride);
            if (RX == 1) {
              x[2 * j] = v.x; x[2 * j + 1] = v.y;
            } else {
              const uint2 w = *reinterpret_cast<const uint2*>(stage + base + half + uint32_t(l0 + j) * stride);
              const float ur = __uint_as_float(v.x), ui = __uint_as_float(v.y);
              const float vr = __uint_as_float(w.x), vi = __uint_as_float(w.y);
              if (bsel == 0) {
                x[2 * j] = __float_as_uint(ur + vr); x[2 * j + 1] = __float_as_uint(ui + vi);
              } else {
                const float2 tw = __ldg(p.twiddle2 + (l0 + j) * R + beta);
                const float dr = ur - vr, di = ui - vi;
                x[2 * j] = __float_as_uint(dr * tw.x - di * tw.y); x[2 * j + 1] = __float_as_uint(dr * tw.y + di * tw.x);
              }
            }
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float r = __uint_as_float(x[j]) - __uint_as_float(x[j] & 0xffffe000u);
            lo[j] = (__float_as_uint(r) + 0x1000u) & 0xffffe000u;
          }
          ptx::tmem_st_32x32(a_hi + l0 * 2, x);
          ptx::tmem_st_32x32(a_lo + l0 * 2, lo);
        }
        ptx::tc_wait_st();
        ptx::tc_fence_before();
        // the raw stage is refilled by TMA (async proxy): order this thread's reads before that write
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(&sh.a1_full[b]);
          ptx::mbar_arrive(&sh.raw_empty[s]);
        }
      }
    }
  } else if (warp >= 8 && warp < 16) {
    // ------------------------------------------------------------ drain stage 1: sum halves, twiddle, split, write A2
    // Two warp groups share the work by k1: group c takes the 16 values k1 = 16c .. 16c+15 (one 32-column chunk of
    // each accumulator half).  For R = 16 there is one chunk and the second group has nothing to do.
    const int grp = (warp - 8) >> 2;
    if (grp < K / 32) {
      const int q = warp & 3;
      const int m = q * 32 + lane;
      const int sl = m / R, beta = m % R;
      const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16) + kFftTmemD1 + grp * 32;
      // A2 row of (sl, k1): CONTIG sl*R + k1 ; STRIDED k1*SL + sl (so that stage-2 stores of one k2 touch neighbouring lines)
      const int row_mul_k1 = (MODE == FFT_CONTIG) ? 1 : SL;
      const int row_base = ((MODE == FFT_CONTIG) ? sl * R : sl) + grp * 16 * row_mul_k1;
      // K column (beta, q) -> panel beta/16, 16-byte chunk (beta%16)/2, half beta%2
      const uint32_t a2_col = uint32_t(beta >> 4) * (128u * 128u) + uint32_t(beta & 1) * 8u;
      const uint32_t a2_chunk = uint32_t(beta & 15) >> 1;
      float twr[16], twi[16];                        // T[16*grp + j][beta], kept for the whole kernel
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float2 w = __ldg(p.twiddle + (grp * 16 + j) * R + beta);
        twr[j] = w.x; twi[j] = w.y;
      }
      for (long long t = 0; t < my_mtiles; ++t) {
        FFT_WAIT_WARP(&sh.d1_full, uint32_t(t) & 1, 0x801);
        ptx::tc_fence_after();
        uint32_t v0[32];
        ptx::tmem_ld_32x32(lane_addr, v0);
        ptx::tc_wait_ld();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.d1_empty);
        float cre[16], cim[16];                       // C[k1] for this lane's beta
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float br = __uint_as_float(v0[2 * j]);
          const float bi = __uint_as_float(v0[2 * j + 1]);
          cre[j] = br * twr[j] - bi * twi[j];
          cim[j] = br * twi[j] + bi * twr[j];
        }
        // stage 2 of the previous M-tile must be done reading A2
        const uint32_t bi = uint32_t(t % NB2), u = uint32_t(t / NB2);
        FFT_WAIT_WARP(&sh.a2_empty[bi], (u & 1) ^ 1, 0x802);
        uint8_t* a2buf = smem_a2 + size_t(bi) * 2 * a2_piece;
        int rb = row_base;
        asm volatile("" : "+r"(rb));                  // recompute the 16 store addresses per tile instead of keeping them live
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int row = rb + j * row_mul_k1;
          const uint32_t off = a2_col + uint32_t(row) * 128u + ((a2_chunk ^ uint32_t(row & 7)) << 4);
          const uint32_t hr = __float_as_uint(cre[j]), hi_ = __float_as_uint(cim[j]);
          const float lr = cre[j] - __uint_as_float(hr & 0xffffe000u);
          const float li = cim[j] - __uint_as_float(hi_ & 0xffffe000u);
          *reinterpret_cast<uint2*>(a2buf + off) = make_uint2(hr, hi_);
          *reinterpret_cast<uint2*>(a2buf + a2_piece + off) =
              make_uint2((__float_as_uint(lr) + 0x1000u) & 0xffffe000u, (__float_as_uint(li) + 0x1000u) & 0xffffe000u);
        }
        ptx::fence_proxy_async_smem();                // generic writes -> visible to the MMA's shared-memory reads
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.a2_full[bi]);
      }
    }
  } else if (warp >= 16) {
    // ------------------------------------------------------------ drain stage 2: sum halves, store in natural order
    const int q = warp & 3;
    const int m = q * 32 + lane;
    const int sl = (MODE == FFT_CONTIG) ? m / R : m % SL;
    const int k1 = (MODE == FFT_CONTIG) ? m % R : m / SL;
    const int g = sl / RX, bsel = sl % RX;
    const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16) + kFftTmemD2;
    long long t = 0, istage = 0;
    for (long long sidx = blockIdx.x; sidx < p.num_stages; sidx += gridDim.x, ++istage) {
      uint8_t* stage = smem_rawring + size_t(istage % p.raw_stages) * p.stage_bytes;   // STAGE_OUT: results return here
      for (int mt = 0; mt < p.mtiles_per_stage; ++mt, ++t) {
        float2* dst;              // &out[line][RX*k1 + bsel]; output k = RX*(k1 + R*k2) + bsel is k2*k2_stride further
        long long k2_stride;
        bool ok;
        if (MODE == FFT_CONTIG) {
          const long long line = sidx * Lg + g;
          ok = line < p.rows;
          dst = reinterpret_cast<float2*>(p.out) + line * p.N + (RX * k1 + bsel);
          k2_stride = RX * R;
        } else {
          const long long ct = sidx % p.c_tiles, bt = sidx / p.c_tiles;
          const long long col = ct * COLS + mt * Lg + g;
          ok = col < p.C;
          dst = reinterpret_cast<float2*>(p.out) + (bt * p.N + (RX * k1 + bsel)) * p.C + col;
          k2_stride = (long long)(RX * R) * p.C;
        }
        FFT_WAIT_WARP(&sh.d2_full, uint32_t(t) & 1, 0x901);
        ptx::tc_fence_after();
#pragma unroll
        for (int ch = 0; ch < K / 32; ++ch) {
          uint32_t v0[32];
          ptx::tmem_ld_32x32(lane_addr + ch * 32, v0);
          ptx::tc_wait_ld();
          if (ch == K / 32 - 1) {
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sh.d2_empty);
          }
          if (STAGE_OUT) {
            // element (row k, column c) of the stage, in the layout TMA wrote the input in (same swizzle)
            const int c = mt * Lg + g;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int k = RX * (k1 + R * (ch * 16 + j)) + bsel;
              const uint32_t swz = (COLS == 16) ? uint32_t(k & 7) : uint32_t((k >> 1) & 3);
              const uint32_t off = uint32_t(k) * kRowBytes + ((uint32_t(c >> 1) ^ swz) << 4) + uint32_t(c & 1) * 8u;
              *reinterpret_cast<uint2*>(stage + off) = make_uint2(v0[2 * j], v0[2 * j + 1]);
            }
          } else if (ok) {
            float2* pd = dst + (long long)(ch * 16) * k2_stride;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              *pd = make_float2(__uint_as_float(v0[2 * j]), __uint_as_float(v0[2 * j + 1]));
              pd += k2_stride;
              asm volatile("" : "+l"(pd));            // one running pointer, not sixteen precomputed ones
            }
          }
        }
      }
      if (STAGE_OUT) {
        // all M-tiles of the stage are back in shared memory: one thread sends the rows out and, once the copy
        // engine has read them, hands the stage to the producer for the next load
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.out_ready);
        if (warp == 16) {
          FFT_WAIT_WARP(&sh.out_ready, uint32_t(istage) & 1, 0x902);
          if (lane == 0) {
            const long long ct = sidx % p.c_tiles, bt = sidx / p.c_tiles;
            for (int r0 = 0; r0 < p.N; r0 += 256) {
              if (p.out_blocked)
                ptx::tma_store_3d(&map_out, stage + size_t(r0) * kRowBytes, 0, r0,
                                  int((ct % p.blk_tiles) * p.blk_rows + ct / p.blk_tiles));
              else
                ptx::tma_store_3d(&map_out, stage + size_t(r0) * kRowBytes, int(ct * 2 * COLS), r0, int(bt));
            }
            ptx::tma_store_commit();
            ptx::tma_store_wait_read();
            ptx::mbar_arrive(&sh.raw_empty[istage % p.raw_stages]);
          }
          __syncwarp();
        }
      }
    }
    if (STAGE_OUT && warp == 16 && lane == 0) ptx::tma_store_wait_all();
  }

role_done:
#ifdef DFT3D_PROFILE_WAITS
  if (p.profile && lane == 0 && (warp <= 2 || (warp & 3) == 0)) {
    // one reporter per role: codes 0x5xx producer, 0x6xx MMA, 0x7xx split, 0x8xx drain 1, 0x9xx drain 2
    long long* dst = p.profile + size_t(blockIdx.x) * 128;
    for (int i = 5; i < 10; ++i)
      for (int j = 0; j < 8; ++j)
        if (prof_wait[i][j]) dst[i * 8 + j] = prof_wait[i][j];
    if (warp == 0) dst[0] = clock64() - prof_start;
  }
#endif
  if (warp == 0 && lane == 0 && sh.abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) { }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, 512);
}

#undef FFT_WAIT
#undef FFT_WAIT_WARP

}  // namespace dft3d
