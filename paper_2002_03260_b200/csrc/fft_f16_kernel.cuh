// The fused FFT axis kernel of fft_kernel.cuh (paper Section III-B, Eq. 17-18: GEMM, phase adjustment, GEMM, all on
// chip) with fp16 pieces instead of TF32 pieces: x = hi + lo and F_R = W_hi + W_lo with 11-bit significands as
// before, multiplied by tcgen05.mma kind::f16 (K = 16 per instruction).  Compared with the TF32 kernel this halves
// the tensor instructions, the tensor-memory stores of the stage-1 operand, the shared-memory bytes of the tables
// and of the stage-2 operand, and so leaves room (tensor memory and shared memory) to double-buffer both
// accumulators and the stage-2 operand at every size.
//
// fp16's exponent range is handled with exact powers of two:
//   * the tables hold 1024 * F_R (real form);
//   * every line (after the radix-2 butterfly, if there is one) is multiplied by its own 2^(13 - e), e = ilogb(largest
//     |component| of the line), so every stage-1 operand component lies below 2^14.  A split thread holds its R
//     elements of the line in registers, so e costs a maximum and a shuffle reduction over the lanes of the line;
//   * a stage-1 result is at most R*sqrt(2) times the largest operand component; the twiddle factors carry
//     2^-(10 + log2(R) - 1), which undoes the table's 1024 and brings the stage-2 operand below 2^15.5 again;
//   * the store multiplies by 2^(log2(R) - 1 - 10) (times 1/n for a scaled inverse) and by the line's 2^(e - E), which
//     the split warps leave in a small tagged ring in shared memory for the warps that drain stage 2.
//
// Geometry, warp roles, barriers and the radix-2 pre-pass are those of fft_kernel.cuh; the differences are the
// operand formats and the second buffer of each accumulator:
//   tensor memory columns: D1 buffers at 0 and 64, D2 buffers at 128 and 192, A1 buffers (hi R columns, lo R columns,
//                          two K-adjacent fp16 values per column) at 256 and 320
//   shared memory:         [W: 2 pieces x 2R rows x 128 B] [A2: 2 buffers x (hi, lo) x 128 rows x 128 B] [raw ring]
#pragma once
#include <cuda_fp16.h>
#include "fft_kernel.cuh"

namespace dft3d {

constexpr int kF16TmemD1 = 0, kF16TmemD2 = 128, kF16TmemA1 = 256;

struct FftF16Params {
  FftParams base;               // twiddle: T[k1][beta] * 2^-(10 + log2(R) - 1), unscaled otherwise
  float out_mul;                // 2^(log2(R) - 1 - 10), times 1/n for a scaled inverse
};

constexpr int kFft16ScaleRing = 16;   // M-tiles whose line scales can be pending between the split and the last drain

struct FftF16Shared {
  uint64_t raw_full[4], raw_empty[4];
  uint64_t a1_full[2], a1_empty[2];
  uint64_t d1_full[2], d1_empty[2];
  uint64_t a2_full[2], a2_empty[2];
  uint64_t d2_full[2], d2_empty[2];
  uint64_t w_full;
  uint64_t out_ready;
  uint32_t tmem_base;
  volatile int abort_flag;
  // per M-tile and (sub-)line: (tile number + 1) << 32 | float bits of 2^(e - E); written by the split warps
  volatile unsigned long long line_scale[kFft16ScaleRing][8];
};

__host__ __device__ constexpr int fft16_w_bytes(int R) { return 2 * 2 * R * 128; }
constexpr int kFft16A2Piece = 128 * 128;
constexpr int kFft16RawBytes = 128 * 1024;
__host__ __device__ constexpr size_t fft16_smem_bytes(int R) {
  return size_t(fft16_w_bytes(R)) + 4 * size_t(kFft16A2Piece) + kFft16RawBytes + 1024 + 2048;
}

#define F16_WAIT(bar, parity, code)                                 \
  {                                                                 \
    FFT_PROF_BEGIN                                                  \
    if (!bounded_wait((bar), (parity), &sh.abort_flag)) {           \
      sh.abort_flag = 1;                                            \
      atomicCAS(p.status, 0u, (unsigned)(code));                    \
      goto role_done;                                               \
    }                                                               \
    FFT_PROF_END(code)                                              \
  }
#define F16_WAIT_WARP(bar, parity, code)                                                  \
  {                                                                                       \
    FFT_PROF_BEGIN                                                                        \
    if (!__all_sync(0xffffffffu, bounded_wait((bar), (parity), &sh.abort_flag) ? 1 : 0)) { \
      sh.abort_flag = 1;                                                                  \
      atomicCAS(p.status, 0u, (unsigned)(code));                                          \
      goto role_done;                                                                     \
    }                                                                                     \
    FFT_PROF_END(code)                                                                    \
  }

// (re, im) -> packed fp16 pairs: hi = round to nearest, lo = the remainder rounded to fp16
__device__ __forceinline__ void split_half2(float re, float im, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(re, im);
  const float2 hf = __half22float2(h);
  const __half2 l = __floats2half2_rn(re - hf.x, im - hf.y);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

template <int MODE, int R, int RX, int COLS, int STAGE_OUT>
__global__ void __launch_bounds__(kFftThreads, 1)
fft_f16_axis_kernel(const __grid_constant__ CUtensorMap map_data, const __grid_constant__ CUtensorMap map_w,
                    const __grid_constant__ CUtensorMap map_out, const FftF16Params pp) {
  const FftParams& p = pp.base;
  extern __shared__ uint8_t smem_raw_[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_) + 1023) & ~uintptr_t(1023));
  constexpr int K = 2 * R;             // reals per contraction
  constexpr int NB = 2 * R;            // MMA N: the 2R output reals (k, re/im) of one stage
  constexpr int KS = K / 16;           // K = 16 steps per product
  constexpr int kWPiece = NB * 128;    // bytes of one table piece in shared memory
  constexpr int a2_piece = kFft16A2Piece;
  uint8_t* smem_w = smem;
  uint8_t* smem_a2 = smem_w + fft16_w_bytes(R);            // buffer i = [hi piece][lo piece] at i * 2 * a2_piece
  uint8_t* smem_rawring = smem_a2 + 4 * a2_piece;
  FftF16Shared& sh = *reinterpret_cast<FftF16Shared*>(smem_rawring + kFft16RawBytes);
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
  constexpr int kD1Warps = 4 * (K / 32);

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) {
      ptx::mbar_init(&sh.raw_full[i], 1);
      ptx::mbar_init(&sh.raw_empty[i], 4 * p.mtiles_per_stage + (STAGE_OUT ? 1 : 0));
    }
    ptx::mbar_init(&sh.out_ready, 4);
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&sh.a1_full[i], 4); ptx::mbar_init(&sh.a1_empty[i], 1);
      ptx::mbar_init(&sh.d1_full[i], 1); ptx::mbar_init(&sh.d1_empty[i], kD1Warps);
      ptx::mbar_init(&sh.a2_full[i], kD1Warps); ptx::mbar_init(&sh.a2_empty[i], 1);
      ptx::mbar_init(&sh.d2_full[i], 1); ptx::mbar_init(&sh.d2_empty[i], 4);
    }
    ptx::mbar_init(&sh.w_full, 1);
    sh.abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (tid < kFft16ScaleRing * 8) sh.line_scale[tid >> 3][tid & 7] = 0ull;
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

  long long my_stages = 0;
  if ((long long)blockIdx.x < p.num_stages) my_stages = (p.num_stages - 1 - blockIdx.x) / gridDim.x + 1;
  const long long my_mtiles = my_stages * p.mtiles_per_stage;

  // the split warps keep a whole line slice in registers: they take what the producer / issuer group can spare
  // (setmaxnreg is a warp-group-wide instruction: one call site per group, executed by all four of its warps; an
  // increase can only take what decreases of the same CTA released: 72 + 120 + 3 x 96 = 5 x 96)
  if (warp < 4) {
  ptx::setmaxnreg_dec<72>();
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      ptx::mbar_arrive_expect_tx(&sh.w_full, uint32_t(fft16_w_bytes(R)));
      for (int pc = 0; pc < 2; ++pc)                // [piece][2R rows][64 halves]
        ptx::tma_load_2d(smem_w + pc * kWPiece, &map_w, &sh.w_full, 0, pc * NB);
      long long i = 0;
      for (long long sidx = blockIdx.x; sidx < p.num_stages; sidx += gridDim.x, ++i) {
        const uint32_t s = uint32_t(i % p.raw_stages), ph = uint32_t(i / p.raw_stages) & 1;
        F16_WAIT(&sh.raw_empty[s], ph ^ 1, 0x501);
        ptx::mbar_arrive_expect_tx(&sh.raw_full[s], uint32_t(p.stage_bytes));
        uint8_t* dst = smem_rawring + size_t(s) * p.stage_bytes;
        if (MODE == FFT_CONTIG) {
          ptx::tma_load_3d(dst, &map_data, &sh.raw_full[s], 0, 0, int(sidx * Lg));
        } else {
          const long long ct = sidx % p.c_tiles, bt = sidx / p.c_tiles;
          for (int r0 = 0; r0 < p.N; r0 += 256) {
            if (p.in_blocked)
              ptx::tma_load_4d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s],
                               int(ct % p.blk_ratio) * 2 * COLS, int(bt), int(ct / p.blk_ratio), r0);
            else
              ptx::tma_load_3d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s], int(ct * 2 * COLS), r0, int(bt));
          }
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
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_f16(128, NB);
      const uint32_t w_addr = ptx::smem_u32(smem_w);
      // operand descriptors: a K = 16 step advances the start address by 32 bytes = 2 descriptor units
      const uint64_t wh = ptx::make_kmajor_sw128_desc(w_addr);
      const uint64_t wl = ptx::make_kmajor_sw128_desc(w_addr + kWPiece);
      F16_WAIT(&sh.w_full, 0, 0x601);
      for (long long t = 0; t < my_mtiles; t += 2) {
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          if (t + b < my_mtiles) {
            const uint32_t phb = uint32_t(t >> 1) & 1;
            F16_WAIT(&sh.a1_full[b], phb, 0x602);
            F16_WAIT(&sh.d1_empty[b], phb ^ 1, 0x603);
            ptx::tc_fence_after();
            const uint32_t a_hi = tmem + kF16TmemA1 + b * 64, a_lo = a_hi + R;
            const uint32_t d = tmem + kF16TmemD1 + b * 64;
#pragma unroll
            for (int k = 0; k < KS; ++k) {
              ptx::mma_f16_ts(d, a_hi + k * 8, wh + 2 * k, idesc, k != 0);
              ptx::mma_f16_ts(d, a_lo + k * 8, wh + 2 * k, idesc, 1);
              ptx::mma_f16_ts(d, a_hi + k * 8, wl + 2 * k, idesc, 1);
            }
            ptx::tc_commit(&sh.a1_empty[b]);
            ptx::tc_commit(&sh.d1_full[b]);
          }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ MMA issuer, stage 2 (A from shared memory)
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_f16(128, NB);
      const uint32_t w_addr = ptx::smem_u32(smem_w);
      const uint32_t a2_addr = ptx::smem_u32(smem_a2);
      const uint64_t wh = ptx::make_kmajor_sw128_desc(w_addr);
      const uint64_t wl = ptx::make_kmajor_sw128_desc(w_addr + kWPiece);
      const uint64_t ah = ptx::make_kmajor_sw128_desc(a2_addr);
      const uint64_t al = ptx::make_kmajor_sw128_desc(a2_addr + a2_piece);
      constexpr uint64_t kBufStep = uint64_t(2 * a2_piece) >> 4;   // second A2 buffer, in descriptor address units
      F16_WAIT(&sh.w_full, 0, 0x611);
      for (long long t = 0; t < my_mtiles; t += 2) {
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          if (t + b < my_mtiles) {
            const uint32_t phb = uint32_t(t >> 1) & 1;
            F16_WAIT(&sh.a2_full[b], phb, 0x604);
            F16_WAIT(&sh.d2_empty[b], phb ^ 1, 0x605);
            ptx::tc_fence_after();
            const uint64_t bstep = b ? kBufStep : 0;
            const uint32_t d = tmem + kF16TmemD2 + b * 64;
#pragma unroll
            for (int k = 0; k < KS; ++k) {
              ptx::mma_f16_ss(d, ah + bstep + 2 * k, wh + 2 * k, idesc, k != 0);
              ptx::mma_f16_ss(d, al + bstep + 2 * k, wh + 2 * k, idesc, 1);
              ptx::mma_f16_ss(d, ah + bstep + 2 * k, wl + 2 * k, idesc, 1);
            }
            ptx::tc_commit(&sh.a2_empty[b]);
            ptx::tc_commit(&sh.d2_full[b]);
          }
        }
      }
    }
  }
  } else if (warp < 8) {
    // ------------------------------------------------------------ split: raw lines -> scaled (hi, lo) fp16 pairs -> A1
    ptx::setmaxnreg_inc<120>();
    const int q = warp & 3;
    const int m = q * 32 + lane;
    const int sl = m / R, beta = m % R;           // stage-1 lane = (sub-line sl, beta), beta fastest
    const int g = sl / RX, bsel = sl % RX;        // line of the cube within the M-tile; which butterfly output
    const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16);
    long long t = 0;
    for (long long i = 0; i < my_stages; ++i) {
      const uint32_t s = uint32_t(i % p.raw_stages), phs = uint32_t(i / p.raw_stages) & 1;
      F16_WAIT_WARP(&sh.raw_full[s], phs, 0x701);
      const uint8_t* stage = smem_rawring + size_t(s) * p.stage_bytes;
      for (int mt = 0; mt < p.mtiles_per_stage; ++mt, ++t) {
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
        // this lane's R elements (after the butterfly when RX == 2), kept in registers: the line's scale comes from
        // their largest magnitude, reduced over the R lanes (all beta) of the (sub-)line
        float xr[R], xi[R];
        float mx = 0.0f;
#pragma unroll
        for (int l = 0; l < R; ++l) {
          const uint2 v = *reinterpret_cast<const uint2*>(stage + base + uint32_t(l) * stride);
          if (RX == 1) {
            xr[l] = __uint_as_float(v.x); xi[l] = __uint_as_float(v.y);
          } else {
            const uint2 w = *reinterpret_cast<const uint2*>(stage + base + half + uint32_t(l) * stride);
            const float ur = __uint_as_float(v.x), ui = __uint_as_float(v.y);
            const float vr = __uint_as_float(w.x), vi = __uint_as_float(w.y);
            if (bsel == 0) {
              xr[l] = ur + vr; xi[l] = ui + vi;
            } else {
              const float2 tw = __ldg(p.twiddle2 + l * R + beta);
              const float dr = ur - vr, di = ui - vi;
              xr[l] = dr * tw.x - di * tw.y; xi[l] = dr * tw.y + di * tw.x;
            }
          }
          mx = fmaxf(mx, fmaxf(fabsf(xr[l]), fabsf(xi[l])));
        }
        // the raw stage is refilled by TMA (async proxy): order this thread's reads before that write
        ptx::fence_proxy_async_smem();
#pragma unroll
        for (int o = R / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) ptx::mbar_arrive(&sh.raw_empty[s]);
        float in_scale = 1.0f;
        {
          float inv = 1.0f;
          if (mx > 0.0f && mx < 3.0e38f) {
            const int e = max(ilogbf(mx), 13 - 126);    // the scale stops growing at 2^126 (subnormal-sized data)
            in_scale = ldexpf(1.0f, 13 - e);
            inv = ldexpf(1.0f, e - 13);
          }
          if (beta == 0)
            sh.line_scale[t % kFft16ScaleRing][sl] = ((unsigned long long)(t + 1) << 32) | __float_as_uint(inv);
        }
        const uint32_t b = uint32_t(t & 1), phb = uint32_t(t >> 1) & 1;
        F16_WAIT_WARP(&sh.a1_empty[b], phb ^ 1, 0x702);
        ptx::tc_fence_after();
        const uint32_t a_hi = lane_addr + kF16TmemA1 + b * 64, a_lo = a_hi + R;
#pragma unroll
        for (int l0 = 0; l0 < R; l0 += 16) {      // 16 complex = 16 packed columns per tensor-memory store
          uint32_t hw[16], lw[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) split_half2(xr[l0 + j] * in_scale, xi[l0 + j] * in_scale, hw[j], lw[j]);
          ptx::tmem_st_32x16(a_hi + l0, hw);
          ptx::tmem_st_32x16(a_lo + l0, lw);
        }
        ptx::tc_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.a1_full[b]);
      }
    }
  } else if (warp >= 8 && warp < 16) {
    // ------------------------------------------------------------ drain stage 1: twiddle, split, write A2
    // Two warp groups share the work by k1: group c takes the 16 values k1 = 16c .. 16c+15 (one 32-column chunk of
    // the accumulator).  For R = 16 there is one chunk and the second group has nothing to do.
    const int grp = (warp - 8) >> 2;
    if (grp < K / 32) {
      const int q = warp & 3;
      const int m = q * 32 + lane;
      const int sl = m / R, beta = m % R;
      const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16) + kF16TmemD1 + grp * 32;
      // A2 row of (sl, k1): CONTIG sl*R + k1 ; STRIDED k1*SL + sl (so that stage-2 stores of one k2 touch neighbouring lines)
      const int row_mul_k1 = (MODE == FFT_CONTIG) ? 1 : SL;
      const int row_base = ((MODE == FFT_CONTIG) ? sl * R : sl) + grp * 16 * row_mul_k1;
      // K position (beta, re/im) = halves 2*beta, 2*beta+1 of the row: 16-byte chunk beta/4, word beta%4
      const uint32_t a2_chunk = uint32_t(beta) >> 2;
      const uint32_t a2_word = uint32_t(beta & 3) * 4u;
      float twr[16], twi[16];                        // scaled T[16*grp + j][beta], kept for the whole kernel
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float2 w = __ldg(p.twiddle + (grp * 16 + j) * R + beta);
        twr[j] = w.x; twi[j] = w.y;
      }
      for (long long t = 0; t < my_mtiles; ++t) {
        const uint32_t b = uint32_t(t & 1), phb = uint32_t(t >> 1) & 1;
        F16_WAIT_WARP(&sh.d1_full[b], phb, 0x801);
        ptx::tc_fence_after();
        uint32_t v0[32];
        ptx::tmem_ld_32x32(lane_addr + b * 64, v0);
        ptx::tc_wait_ld();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.d1_empty[b]);
        uint32_t ch[16], cl[16];                      // C[k1] for this lane's beta, as packed fp16 pieces
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float br = __uint_as_float(v0[2 * j]);
          const float bi = __uint_as_float(v0[2 * j + 1]);
          split_half2(br * twr[j] - bi * twi[j], br * twi[j] + bi * twr[j], ch[j], cl[j]);
        }
        // stage 2 of the M-tile two back must be done reading this A2 buffer
        F16_WAIT_WARP(&sh.a2_empty[b], phb ^ 1, 0x802);
        uint8_t* a2buf = smem_a2 + size_t(b) * 2 * a2_piece;
        int rb = row_base;
        asm volatile("" : "+r"(rb));                  // recompute the 16 store addresses per tile instead of keeping them live
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int row = rb + j * row_mul_k1;
          const uint32_t off = uint32_t(row) * 128u + ((a2_chunk ^ uint32_t(row & 7)) << 4) + a2_word;
          *reinterpret_cast<uint32_t*>(a2buf + off) = ch[j];
          *reinterpret_cast<uint32_t*>(a2buf + a2_piece + off) = cl[j];
        }
        ptx::fence_proxy_async_smem();                // generic writes -> visible to the MMA's shared-memory reads
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.a2_full[b]);
      }
    }
  } else if (warp >= 16) {
    // ------------------------------------------------------------ drain stage 2: undo the scales, store in natural order
    const int q = warp & 3;
    const int m = q * 32 + lane;
    const int sl = (MODE == FFT_CONTIG) ? m / R : m % SL;
    const int k1 = (MODE == FFT_CONTIG) ? m % R : m / SL;
    const int g = sl / RX, bsel = sl % RX;
    const uint32_t lane_addr = tmem + (uint32_t(q * 32) << 16) + kF16TmemD2;
    const float om1 = pp.out_mul;
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
        const uint32_t b = uint32_t(t & 1), phb = uint32_t(t >> 1) & 1;
        F16_WAIT_WARP(&sh.d2_full[b], phb, 0x901);
        ptx::tc_fence_after();
        // this line's scale; the split warps wrote it long ago (the tag guards against reading a slot too early)
        float out_mul2;
        {
          unsigned long long sv;
          bool seen;
          const long long t0 = clock64();
          for (;;) {
            sv = sh.line_scale[t % kFft16ScaleRing][sl];
            seen = (sv >> 32) == (unsigned long long)(t + 1);
            if (seen || sh.abort_flag || clock64() - t0 > 4000000000LL) break;
          }
          if (!__all_sync(0xffffffffu, seen ? 1 : 0)) {
            sh.abort_flag = 1;
            atomicCAS(p.status, 0u, 0x903u);
            goto role_done;
          }
          out_mul2 = __uint_as_float(uint32_t(sv));
        }
#pragma unroll
        for (int ch = 0; ch < K / 32; ++ch) {
          uint32_t v0[32];
          ptx::tmem_ld_32x32(lane_addr + b * 64 + ch * 32, v0);
          ptx::tc_wait_ld();
          if (ch == K / 32 - 1) {
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sh.d2_empty[b]);
          }
          float f[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) f[j] = (__uint_as_float(v0[j]) * om1) * out_mul2;
          if (STAGE_OUT) {
            // element (row k, column c) of the stage, in the layout TMA wrote the input in (same swizzle)
            const int c = mt * Lg + g;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int k = RX * (k1 + R * (ch * 16 + j)) + bsel;
              const uint32_t swz = (COLS == 16) ? uint32_t(k & 7) : uint32_t((k >> 1) & 3);
              const uint32_t off = uint32_t(k) * kRowBytes + ((uint32_t(c >> 1) ^ swz) << 4) + uint32_t(c & 1) * 8u;
              *reinterpret_cast<float2*>(stage + off) = make_float2(f[2 * j], f[2 * j + 1]);
            }
          } else if (ok) {
            float2* pd = dst + (long long)(ch * 16) * k2_stride;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              *pd = make_float2(f[2 * j], f[2 * j + 1]);
              pd += k2_stride;
              asm volatile("" : "+l"(pd));            // one running pointer, not sixteen precomputed ones
            }
          }
        }
      }
      if (STAGE_OUT) {
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.out_ready);
        if (warp == 16) {
          F16_WAIT_WARP(&sh.out_ready, uint32_t(istage) & 1, 0x902);
          if (lane == 0) {
            const long long ct = sidx % p.c_tiles, bt = sidx / p.c_tiles;
            for (int r0 = 0; r0 < p.N; r0 += 256) {
              if (p.out_blocked)
                ptx::tma_store_3d(&map_out, stage + size_t(r0) * kRowBytes, 0, r0, int(ct));
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

#undef F16_WAIT
#undef F16_WAIT_WARP

}  // namespace dft3d
