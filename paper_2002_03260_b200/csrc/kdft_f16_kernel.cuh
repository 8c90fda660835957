// KDFT axis kernel with fp16 pieces: the same tile, pipeline and complex-as-real mapping as kdft_kernel.cuh, but
// the split x = hi + lo, W = W_hi + W_lo uses fp16 pieces (11-bit significands, like TF32) and
// tcgen05.mma kind::f16, which contracts K = 16 per instruction at twice the TF32 rate: half the MMAs and half
// the table bytes for the same three products (hi*hi, lo*hi, hi*lo) and the same fp32 accumulation.
//
// fp16 has a narrow exponent range, so the operands are scaled by powers of two (exact):
//   * the table holds 1024 * W (entries in [-1024, 1024]; the lo piece of all but vanishing entries stays normal);
//   * the data is multiplied by 2^k with k chosen from the largest input magnitude, which every pass records for
//     its successor (amax_out) and a small reduction kernel provides for the first pass; the largest scaled value
//     lies in [2^13, 2^14).  An entry more than 2^18 below the largest loses relative precision (its lo piece
//     becomes subnormal: absolute error 2^-25 of a scaled unit, i.e. 2^-38 of the largest entry), which is far
//     below fp32 rounding in the norm-wise sense the transform is judged in.
//   The epilogue multiplies by 2^-10 * 2^-k (and 1/n for a scaled inverse).
// A stage covers 64 reals of the contraction (128-byte rows of the fp16 table); the raw fp32 data stage is 32 KB.
#pragma once
#include <cuda_fp16.h>
#include "kdft_kernel.cuh"
#include "split_f16.cuh"

namespace dft3d {

constexpr int kF16BlockK = 64;          // reals of the contraction per pipeline stage
constexpr int kF16BytesStageA = kTileM * kF16BlockK * 4;   // raw fp32 data of one stage: 32 KB
// The raw data of a stage arrives as two halves of 32 reals (16 KB each) with a barrier pair of their own, so that the
// second half (and the next stage's first) is on its way while the split warps convert the first: a double buffer in
// the room of one stage.
constexpr int kF16HalvesA = 2;
constexpr int kF16BytesHalfA = kF16BytesStageA / 2;
constexpr size_t kKdftF16SmemBytes = size_t(kStagesB) * kBytesStageB + size_t(kF16BytesStageA) + 1024 + 512;

struct KdftF16Params {
  int k2, bn, n_tiles, chunk_kb;        // as KdftParams; chunk_kb counts 64-real stages
  long long m_tiles, rows, batches, C;
  int lpb, bpt;
  long long c_tiles;
  float* out;
  unsigned int* status;
  long long* profile;
  float out_mul;                        // 2^-10, times 1/n for a scaled inverse
  int n_group;                          // table panels (n-tiles) that are live at a time; the tiles go
                                        // panel group by panel group, all lines within a group (0 or n_tiles: one group)
  const unsigned int* amax_in;          // float bits: largest |input| (an upper bound is enough)
  unsigned int* amax_out;               // float bits: receives the largest |output| (atomic max)
  WaitControl wc;
};

struct KdftF16Shared {
  uint64_t b_full[kStagesB], b_empty[kStagesB];
  uint64_t a_full[kF16HalvesA], a_empty[kF16HalvesA];
  uint64_t t_full[kStagesT], t_empty[kStagesT];
  uint64_t acc_full, acc_empty;
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;
};

// largest magnitude of a float array (grid-stride, one atomic per warp); `result` must start at zero
__global__ void amax_kernel(const float4* x, long long n4, unsigned int* result) {
  float m = 0.0f;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    const float4 v = x[i];
    m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0 && m > 0.0f) atomicMax(result, __float_as_uint(m));
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
kdft_f16_axis_kernel(const __grid_constant__ CUtensorMap map_data, const __grid_constant__ CUtensorMap map_w,
                 const KdftF16Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_b = smem;
  uint8_t* smem_a = smem + size_t(kStagesB) * kBytesStageB;
  KdftF16Shared& sh = *reinterpret_cast<KdftF16Shared*>(smem_a + size_t(kF16BytesStageA));

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < kStagesB; ++i) { ptx::mbar_init(&sh.b_full[i], 1); ptx::mbar_init(&sh.b_empty[i], 1); }
    for (int i = 0; i < kF16HalvesA; ++i) { ptx::mbar_init(&sh.a_full[i], 1); ptx::mbar_init(&sh.a_empty[i], 4); }
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
  // tile order: panel group by panel group (see KdftF16Params::n_group); one group = panel fastest over all line tiles
  const long long ng = (p.n_group > 0 && p.n_group < p.n_tiles && p.n_tiles % p.n_group == 0) ? p.n_group : p.n_tiles;
  const long long tiles_per_group = p.m_tiles * ng;
  const int num_kb = (p.k2 + kF16BlockK - 1) / kF16BlockK;   // a ragged last stage is zero-filled by TMA on both operands
  const uint32_t bytes_b = 2u * uint32_t(p.bn) * 128u;            // two pieces, bn rows of 64 halves

  // power-of-two scale that brings the largest input magnitude into [2^13, 2^14): fp16 pieces then neither
  // overflow nor lose more than fp16's own subnormal floor (2^-25 of a scaled unit) on small entries
  float in_scale = 1.0f, out_mul2 = 1.0f;
  {
    const float a = __uint_as_float(*p.amax_in);
    if (a > 0.0f && a < 3.0e38f) {
      // below 2^-113 the scale stops growing (2^126 is the largest power of two that is safe to multiply by);
      // nothing is lost: such data are multiples of 2^-149, i.e. of 2^-23 after scaling, which the two pieces hold
      const int e = max(ilogbf(a), -113);
      in_scale = ldexpf(1.0f, 13 - e);
      out_mul2 = ldexpf(1.0f, e - 13);
    }
  }

  if (warp < 4) {
    // warp group 0: producer and MMA issuer need few registers; hand the rest to the epilogue
    ptx::setmaxnreg_dec<DFT3D_REGS_WG0>();
    if (warp == 0) {
      // ------------------------------------------------------------ TMA producer
      if (lane == 0 && !p.wc.silent_producer) {
        uint32_t ib = 0, ia = 0;   // running stage counters
        for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
          const long long mt = (t % tiles_per_group) / ng;
          const int nt = int((t / tiles_per_group) * ng + t % ng);
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
              ptx::tma_load_3d(smem_b + size_t(s) * kBytesStageB, &map_w, &sh.b_full[s], kb * kF16BlockK, nt * p.bn, 0);
              ++ib;
            }
#pragma unroll
            for (int h = 0; h < kF16HalvesA; ++h) {
              const uint32_t s = ia % kF16HalvesA, ph = (ia / kF16HalvesA) & 1;
              DFT3D_WAIT(&sh.a_empty[s], ph ^ 1, 0x102);
              ptx::mbar_arrive_expect_tx(&sh.a_full[s], kF16BytesHalfA);
              if (MODE == KDFT_CONTIG)     // a 128-byte-wide half (the 128B swizzle spans 32 floats)
                ptx::tma_load_2d(smem_a + size_t(s) * kF16BytesHalfA, &map_data, &sh.a_full[s], kb * kF16BlockK + 32 * h, ay);
              else                         // 16 rows j of the stage's 32
                ptx::tma_load_3d(smem_a + size_t(s) * kF16BytesHalfA, &map_data, &sh.a_full[s], ax,
                                 kb * (kF16BlockK / 2) + 16 * h, az);
              ++ia;
            }
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------ MMA issuer
      if (lane == 0) {
        const uint32_t idesc = ptx::make_idesc_f16(kTileM, p.bn);
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
            const uint32_t b_lo = b_hi + uint32_t(p.bn) * 128u;
            const uint32_t a_hi = tmem + kAccCols + st * 64;
            const uint32_t a_lo = a_hi + 32;
#pragma unroll
            for (int k = 0; k < kF16BlockK / 16; ++k) {   // K = 16 per MMA: 8 packed columns of A, 32 bytes of each B row
              const uint64_t dhi = ptx::make_kmajor_sw128_desc(b_hi + k * 32);
              const uint64_t dlo = ptx::make_kmajor_sw128_desc(b_lo + k * 32);
              ptx::mma_f16_ts(tmem, a_hi + k * 8, dhi, idesc, (k != 0 || !chunk_first) ? 1u : 0u);
              ptx::mma_f16_ts(tmem, a_lo + k * 8, dhi, idesc, 1);
              ptx::mma_f16_ts(tmem, a_hi + k * 8, dlo, idesc, 1);
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
    if (MODE == KDFT_STRIDED) strided_off = (m / p.lpb) * (kF16BlockK / 4) * p.lpb + (m % p.lpb);   // 16 rows per half
    const uint64_t scale2 = pack2(in_scale, in_scale);
    uint32_t ia = 0, it = 0;
    for (long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const uint32_t st = it % kStagesT, pht = (it / kStagesT) & 1;
        uint32_t ph[32], pl[32];                 // 64 scaled values as fp16 pairs: hi pieces, lo pieces
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t sa = ia % kF16HalvesA, pha = (ia / kF16HalvesA) & 1;
          DFT3D_WAIT_WARP(&sh.a_full[sa], pha, 0x301);
          const uint8_t* stage = smem_a + size_t(sa) * kF16BytesHalfA;
          uint32_t x[32];
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
            for (int j = 0; j < 16; ++j) {
              const uint2 v = colp[j * p.lpb];
              x[2 * j] = v.x; x[2 * j + 1] = v.y;
            }
          }
          // the half is refilled by TMA (async proxy): order this thread's reads before that write
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&sh.a_empty[sa]);
          ++ia;
#pragma unroll
          for (int i = 0; i < 16; ++i)   // element 2i in the low half of each fp16 pair; packed fp32 instructions
            split_half2(mul2(pack2_bits(x[2 * i], x[2 * i + 1]), scale2), ph[h * 16 + i], pl[h * 16 + i]);
        }
        DFT3D_WAIT_WARP(&sh.t_empty[st], pht ^ 1, 0x302);
        ptx::tc_fence_after();
        ptx::tmem_st_32x32(lane_addr + kAccCols + st * 64, ph);
        ptx::tmem_st_32x32(lane_addr + kAccCols + st * 64 + 32, pl);
        ptx::tc_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.t_full[st]);
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
      const long long mt = (t % tiles_per_group) / ng;
      const int nt = int((t / tiles_per_group) * ng + t % ng);
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
      // ---- undo the scales, note the largest magnitude for the next pass, store this lane's 128 reals
      const int c0 = nt * p.bn + half * 128;   // first real output column held by this thread
      float amax = 0.0f;
#pragma unroll
      for (int i = 0; i < 128; ++i) acc[i] = (acc[i] * p.out_mul) * out_mul2;   // two exact-unless-underflow steps
      if (cols_active && c0 < p.k2) {
        if (MODE == KDFT_CONTIG) {
          const long long row = mt * kTileM + m;
          if (row < p.rows) {
            float4* dst = reinterpret_cast<float4*>(p.out + row * (long long)p.k2 + c0);
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + 4 * i < p.k2) {
                dst[i] = make_float4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
                amax = fmaxf(fmaxf(amax, fmaxf(fabsf(acc[4 * i]), fabsf(acc[4 * i + 1]))),
                             fmaxf(fabsf(acc[4 * i + 2]), fabsf(acc[4 * i + 3])));
              }
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
              if (c0 / 2 + i < J) {
                *reinterpret_cast<float2*>(dst + i * k_stride) = make_float2(acc[2 * i], acc[2 * i + 1]);
                amax = fmaxf(amax, fmaxf(fabsf(acc[2 * i]), fabsf(acc[2 * i + 1])));
              }
          }
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if (lane == 0 && amax > 0.0f) atomicMax(p.amax_out, __float_as_uint(amax));
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
