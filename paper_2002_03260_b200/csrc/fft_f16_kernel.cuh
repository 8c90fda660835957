// The fused FFT axis kernel (paper Section III-B, Eq. 17-18: GEMM, phase adjustment, GEMM, all on chip) with fp16
// pieces and tile-parallel warp groups.
//
// Arithmetic: as in fft_kernel.cuh (n = R*l + beta, k = k1 + R*k2, complex-as-real 2R x 2R matrices, three products
// hi*hi, lo*hi, hi*lo per K step, fp32 accumulation in tensor memory), but x = hi + lo and F_R = W_hi + W_lo use fp16
// pieces (11-bit significands, as TF32 has) and tcgen05.mma kind::f16 (K = 16 per instruction): half the tensor
// instructions, half the tensor-memory stores of the stage-1 operand, half the shared-memory bytes of the tables and
// of the stage-2 operand.
//
// fp16's exponent range is handled with exact powers of two:
//   * the tables hold 1024 * F_R (real form);
//   * every line (after the radix-2 butterfly, if there is one) is multiplied by its own 2^(13 - e), e = the exponent
//     of its largest |component|, so every stage-1 operand component lies below 2^14.  A thread holds its R elements
//     of the line in registers, so e costs a maximum and one reduction over the lanes of the line;
//   * a stage-1 result is at most R*sqrt(2) times the largest operand component; the twiddle factors carry
//     2^-(10 + log2(R) - 1), which undoes the table's 1024 and keeps the stage-2 operand below 2^15.5;
//   * the store multiplies by 2^(log2(R) - 1 - 10) (times 1/n for a scaled inverse) and by the line's 2^(e - 13).
// An element more than 2^18 below its line's largest keeps less than full relative precision (its lo piece becomes
// subnormal: absolute error 2^-38 of the line's largest element), which is invisible in the norm-wise error.
//
// Lengths N = RX*R*R.  RX = 2 (512, 2048) and RX = 4 (4096 = 4*32*32, a three-factor split) apply Eq. 17 once more with
// P = N/RX before the two GEMM stages: the thread of sub-line b forms  y_b[m] = (sum_q x[m + q*N/RX] * w_RX^(b*q)) *
// exp(s*2*pi*i*b*m/N)  for m < R*R (a radix-RX butterfly on the CUDA cores: additions, swaps and one complex
// multiplication), and X[RX*k + b] is entry k of the R*R-point transform of y_b.
//
// Organisation.  The per-tile chain  split -> MMA 1 -> drain 1 (+twiddle) -> MMA 2 -> drain 2 (+store)  is latency
// bound when every link is one warp group (the TF32 kernel's design: each group sees one warp per scheduler).  Here
// four identical worker groups each take every fourth M-tile through ALL the links, so each scheduler always has four
// independent warps to pick from, and the two MMA issuer threads serve the groups in tile order:
//   warp 0      TMA producer (raw stages, tables)
//   warp 1, 2   MMA issuers, stage 1 (A from tensor memory) and stage 2 (A from shared memory)
//   warp 3      STAGE_OUT only: sends finished stages out as TMA stores
//   warps 4-19  worker groups g = 0..3 (tile t belongs to group t mod 4)
// Tensor memory, per group g at column 128*g: D1 at +0 (2R columns), A1 at +64 (hi R columns, lo R columns, two
// K-adjacent fp16 values per column); D2 reuses A1's columns (stage 1 has consumed them by then).
// Shared memory: [W: 2 pieces x 2R rows x 128 B] [A2: 2 buffers x (hi, lo) x 128 rows x 128 B, used in tile order]
// [twiddles R x R complex64 (and those of the radix-2 step)] [raw ring 128 KB] [barriers].
// A mbarrier wait tells phases apart by parity only, so nobody may wait on a barrier two phases ahead: every barrier
// here is waited on in consecutive phases by construction (per-group barriers by that group and the issuers in tile
// order; a2_empty[h] by group h^2 for every tile of group h; raw_full[s] needs (4 / tiles per stage) to divide the
// ring length, which the host guarantees).
#pragma once
#include <cuda_fp16.h>
#include "fft_kernel.cuh"
#include "split_f16.cuh"

namespace dft3d {

struct FftF16Params {
  FftParams base;               // twiddle: T[k1][beta] * 2^-(10 + log2(R) - 1), unscaled otherwise
  float out_mul;                // 2^(log2(R) - 1 - 10), times 1/n for a scaled inverse
  float quarter_turn;           // RX == 4: the sign s of the exponent (exp(s*2*pi*i/4) = s*i)
};

// Two axes in one launch (fft_f16_fused_kernel below): the CTAs of the axis-1 pass write n0-planes of their result
// into a ring of `ring` planes, the CTAs of the axis-2 pass read them from there, and these counters order the two.
// All zero for the one-axis kernels.
struct FftFuse {
  unsigned int* written;     // [planes] warps that have stored their share of plane p (writer side adds, reader side waits)
  unsigned int* consumed;    // [planes] warps whose share of plane p has arrived in shared memory (reader side adds)
  unsigned int written_target, consumed_target;
  int ring;                  // planes in the ring; plane p lives in slot p % ring
  long long ring_rows;       // reader: rows (lines) of the whole ring, ring * n1
  int ctas_writer;           // CTAs 0 .. ctas_writer-1 run the axis-1 pass, the others the axis-2 pass
  int evict_hints;           // 1: L2 eviction hints (input and output stream: evict first; ring: evict last)
};
enum : int { FUSE_NONE = 0, FUSE_WRITER = 1, FUSE_READER = 2 };

struct FftF16Shared {
  uint64_t raw_full[4], raw_empty[4], out_ready[4];
  uint64_t split_done[4];      // STAGE_OUT with tiles that share lines: every tile of the stage has read its input
  uint64_t a1_full[4], d1_full[4], a2_full[4], a2_empty[4], d2_full[4], sc_full[4];
  uint64_t w_full;
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;
  float line_scale[4][8];      // per group, 2^(e - 13) of the tile's (sub-)lines, from the split to the store (where a
                               // thread's stage-2 lane belongs to another sub-line than its stage-1 lane)
};

__host__ __device__ constexpr int fft16_w_bytes(int R) { return 2 * 2 * R * 128; }
__host__ __device__ constexpr int fft16_tw_bytes(int R) { return R * R * 8; }
constexpr int kFft16A2Piece = 128 * 128;
constexpr int kFft16RawBytes = 128 * 1024;
__host__ __device__ constexpr size_t fft16_smem_bytes(int R, int RX) {   // RX == 2: a second twiddle table (radix-2 step)
  return size_t(fft16_w_bytes(R)) + 4 * size_t(kFft16A2Piece) + size_t(RX == 2 ? 2 : 1) * fft16_tw_bytes(R) +
         kFft16RawBytes + 1024 + 1024;
}

#ifndef FFT16_REGS_WG0
#define FFT16_REGS_WG0 64
#define FFT16_REGS_WORK 104
#endif
#define F16_WAIT(bar, parity, code)                                 \
  {                                                                 \
    FFT_PROF_BEGIN                                                  \
    if (!bounded_wait((bar), (parity), &sh.abort_flag, sh.wait_limit)) {           \
      sh.abort_flag = 1;                                            \
      atomicCAS(p.status, 0u, (unsigned)(code));                    \
      goto role_done;                                               \
    }                                                               \
    FFT_PROF_END(code)                                              \
  }
#define F16_WAIT_WARP(bar, parity, code)                                                  \
  {                                                                                       \
    FFT_PROF_BEGIN                                                                        \
    if (!__all_sync(0xffffffffu, bounded_wait((bar), (parity), &sh.abort_flag, sh.wait_limit) ? 1 : 0)) { \
      sh.abort_flag = 1;                                                                  \
      atomicCAS(p.status, 0u, (unsigned)(code));                                          \
      goto role_done;                                                                     \
    }                                                                                     \
    FFT_PROF_END(code)                                                                    \
  }

// Waits until a counter in global memory that other CTAs add to has reached `target` (bounded like every other wait).
__device__ __forceinline__ bool bounded_wait_counter(const unsigned int* counter, unsigned int target,
                                                     volatile int* abort_flag, long long limit) {
  const long long t0 = clock64();
  for (uint32_t spin = 0;; ++spin) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    if ((spin & 0xf) == 0xf) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) return false;
    }
    __nanosleep(200);
  }
}

// The body of one CTA: CTA number `cta` of `ncta` takes the stages cta, cta + ncta, ...  FUSE: see FftFuse.
template <int MODE, int R, int RX, int COLS, int STAGE_OUT, int FUSE>
__device__ __forceinline__ void fft_f16_axis_body(const CUtensorMap* map_data_p, const CUtensorMap* map_w_p,
                                                  const CUtensorMap* map_out_p, const FftF16Params& pp,
                                                  const FftFuse& fz, const int cta, const int ncta) {
  const CUtensorMap& map_data = *map_data_p;
  const CUtensorMap& map_w = *map_w_p;
  const CUtensorMap& map_out = *map_out_p;
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
  float2* smem_tw = reinterpret_cast<float2*>(smem_a2 + 4 * a2_piece);
  float2* smem_tw2 = smem_tw + R * R;                      // RX == 2 only: exp(s*2*pi*i*m/N), m < R*R
  uint8_t* smem_rawring = reinterpret_cast<uint8_t*>(smem_tw) + (RX == 2 ? 2 : 1) * fft16_tw_bytes(R);
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

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) {
      ptx::mbar_init(&sh.raw_full[i], 1);
      ptx::mbar_init(&sh.raw_empty[i], STAGE_OUT ? 1 : 4 * p.mtiles_per_stage);   // the store warp / the split warps
      ptx::mbar_init(&sh.sc_full[i], 4);
      ptx::mbar_init(&sh.out_ready[i], 4 * p.mtiles_per_stage);
      ptx::mbar_init(&sh.split_done[i], 4 * p.mtiles_per_stage);
      ptx::mbar_init(&sh.a1_full[i], 4);
      ptx::mbar_init(&sh.d1_full[i], 1);
      ptx::mbar_init(&sh.a2_full[i], 4);
      ptx::mbar_init(&sh.a2_empty[i], 1);
      ptx::mbar_init(&sh.d2_full[i], 1);
    }
    ptx::mbar_init(&sh.w_full, 1);
    sh.abort_flag = 0;
    sh.wait_limit = p.wc.limit_clocks > 0 ? p.wc.limit_clocks : kDefaultWaitClocks;
    ptx::fence_mbar_init();
  }
  for (int i = tid; i < R * R; i += kFftThreads) smem_tw[i] = __ldg(p.twiddle + i);
  if (RX == 2)
    for (int i = tid; i < R * R; i += kFftThreads) smem_tw2[i] = __ldg(p.twiddle2 + i);
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
  if ((long long)cta < p.num_stages) my_stages = (p.num_stages - 1 - cta) / ncta + 1;
  const long long my_mtiles = my_stages * p.mtiles_per_stage;

  // Registers: the workers keep a line slice in registers and take what the first group can spare.  setmaxnreg is a
  // warp-group-wide instruction (one call site per group, executed by all four of its warps), and an increase can
  // only take what decreases of the same CTA released: 64 + 4 x 104 = 5 x 96.
  if (warp < 4) {
    ptx::setmaxnreg_dec<FFT16_REGS_WG0>();
    if (warp == 0) {
      // ---------------------------------------------------------- TMA producer
      if (lane == 0 && !p.wc.silent_producer) {
        ptx::mbar_arrive_expect_tx(&sh.w_full, uint32_t(fft16_w_bytes(R)));
        for (int pc = 0; pc < 2; ++pc)                // [piece][2R rows][64 halves]
          ptx::tma_load_2d(smem_w + pc * kWPiece, &map_w, &sh.w_full, 0, pc * NB);
        long long i = 0;
        long long plane_ok = -1;                      // FUSE: the plane the last counter wait was for
        // FUSE with hints: the stream from HBM leaves L2 first, the ring stays
        const bool hints = FUSE != FUSE_NONE && fz.evict_hints;
        const uint64_t pol_load = hints ? (FUSE == FUSE_WRITER ? ptx::l2_policy_evict_first() : ptx::l2_policy_evict_last()) : 0;
        for (long long sidx = cta; sidx < p.num_stages; sidx += ncta, ++i) {
          const uint32_t s = uint32_t(i % p.raw_stages), ph = uint32_t(i / p.raw_stages) & 1;
          F16_WAIT(&sh.raw_empty[s], ph ^ 1, 0x501);
          if (FUSE != FUSE_NONE) {
            // writer: the plane that last lived in this stage's ring slot must have been read completely before
            // anything of this stage is stored there; the load below gates this CTA's stores (the workers store only
            // after they have seen it land).  Reader: the plane must have been written completely.
            const long long plane = sidx / p.fuse_stages_per_plane;
            const long long need = (FUSE == FUSE_WRITER) ? plane - fz.ring : plane;
            if (need >= 0 && need != plane_ok) {
              const unsigned int* counter = (FUSE == FUSE_WRITER ? fz.consumed : fz.written) + need;
              const unsigned int target = FUSE == FUSE_WRITER ? fz.consumed_target : fz.written_target;
              if (!bounded_wait_counter(counter, target, &sh.abort_flag, sh.wait_limit)) {
                sh.abort_flag = 1;
                atomicCAS(p.status, 0u, 0x502u);
                goto role_done;
              }
              plane_ok = need;
              // the loads that follow read, through the async proxy, what other CTAs wrote with ordinary stores
              asm volatile("fence.proxy.async.global;" ::: "memory");
            }
          }
          ptx::mbar_arrive_expect_tx(&sh.raw_full[s], uint32_t(p.stage_bytes));
          uint8_t* dst = smem_rawring + size_t(s) * p.stage_bytes;
          if (MODE == FFT_CONTIG) {
            const long long row0 = sidx * Lg;
            if (hints) ptx::tma_load_3d_hint(dst, &map_data, &sh.raw_full[s], 0, 0, int(row0 % fz.ring_rows), pol_load);
            else ptx::tma_load_3d(dst, &map_data, &sh.raw_full[s], 0, 0, int(FUSE == FUSE_READER ? row0 % fz.ring_rows : row0));
          } else {
            const long long ct = sidx % p.c_tiles, bt = sidx / p.c_tiles;
            for (int r0 = 0; r0 < p.N; r0 += 256) {
              if (p.in_blocked && p.blk_pair > 1)
                ptx::tma_load_5d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s], 0, 0, int(bt), r0 / p.blk_pair,
                                 int(ct));
              else if (p.in_blocked && hints)
                ptx::tma_load_4d_hint(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s],
                                      int(ct % p.blk_ratio) * 2 * COLS, int(bt), r0, int(ct / p.blk_ratio), pol_load);
              else if (p.in_blocked)
                ptx::tma_load_4d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s],
                                 int(ct % p.blk_ratio) * 2 * COLS, int(bt), r0, int(ct / p.blk_ratio));
              else if (p.col_tiles_row)   // a slice of the last axis: tile ct % tiles of row ct / tiles of the full array
                ptx::tma_load_3d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s],
                                 int(2 * ((ct / p.col_tiles_row) * p.col_pitch + p.col_off + (ct % p.col_tiles_row) * COLS)),
                                 r0, int(bt));
              else
                ptx::tma_load_3d(dst + size_t(r0) * kRowBytes, &map_data, &sh.raw_full[s], int(ct * 2 * COLS), r0, int(bt));
            }
            const long long nidx = sidx + ncta;
            if (p.l2_prefetch && nidx < p.num_stages) {
              const long long nct = nidx % p.c_tiles, nbt = nidx / p.c_tiles;
              for (int r0 = 0; r0 < p.N; r0 += 256)
                ptx::tma_prefetch_l2_3d(&map_data, int(nct * 2 * COLS), r0, int(nbt));
            }
          }
        }
      }
    } else if (warp == 1) {
      // ---------------------------------------------------------- MMA issuer, stage 1: D1[g] = A1[g] (tensor memory) x W
      if (lane == 0) {
        const uint32_t idesc = ptx::make_idesc_f16(128, NB);
        const uint32_t w_addr = ptx::smem_u32(smem_w);
        // operand descriptors: a K = 16 step advances the start address by 32 bytes = 2 descriptor units
        const uint64_t wh = ptx::make_kmajor_sw128_desc(w_addr);
        const uint64_t wl = ptx::make_kmajor_sw128_desc(w_addr + kWPiece);
        F16_WAIT(&sh.w_full, 0, 0x601);
        for (long long t = 0; t < my_mtiles; ++t) {
          const uint32_t g = uint32_t(t) & 3, pk = uint32_t(t >> 2) & 1;
          F16_WAIT(&sh.a1_full[g], pk, 0x602);
          ptx::tc_fence_after();
          const uint32_t d = tmem + g * 128;
          const uint32_t a_hi = d + 64, a_lo = a_hi + R;
          // the small products first: the tensor core truncates when it adds into its accumulator, by up to one
          // ulp of the accumulator, so the fewer additions happen once the large hi*hi terms are in, the better
#pragma unroll
          for (int k = 0; k < KS; ++k) {
            ptx::mma_f16_ts(d, a_lo + k * 8, wh + 2 * k, idesc, k != 0);
            ptx::mma_f16_ts(d, a_hi + k * 8, wl + 2 * k, idesc, 1);
          }
#pragma unroll
          for (int k = 0; k < KS; ++k) ptx::mma_f16_ts(d, a_hi + k * 8, wh + 2 * k, idesc, 1);
          ptx::tc_commit(&sh.d1_full[g]);
        }
      }
    } else if (warp == 2) {
      // ---------------------------------------------------------- MMA issuer, stage 2: D2[g] = A2[t & 1] (shared memory) x W
      if (lane == 0) {
        const uint32_t idesc = ptx::make_idesc_f16(128, NB);
        const uint32_t idesc_wide = ptx::make_idesc_f16(128, 2 * NB);
        const uint32_t w_addr = ptx::smem_u32(smem_w);
        const uint32_t a2_addr = ptx::smem_u32(smem_a2);
        const uint64_t wh = ptx::make_kmajor_sw128_desc(w_addr);
        const uint64_t wl = ptx::make_kmajor_sw128_desc(w_addr + kWPiece);
        const uint64_t ah0 = ptx::make_kmajor_sw128_desc(a2_addr);
        const uint64_t al0 = ptx::make_kmajor_sw128_desc(a2_addr + a2_piece);
        constexpr uint64_t kBufStep = uint64_t(2 * a2_piece) >> 4;   // second A2 buffer, in descriptor address units
        F16_WAIT(&sh.w_full, 0, 0x611);
        for (long long t = 0; t < my_mtiles; ++t) {
          const uint32_t g = uint32_t(t) & 3, pk = uint32_t(t >> 2) & 1;
          F16_WAIT(&sh.a2_full[g], pk, 0x604);
          ptx::tc_fence_after();
          const uint64_t ah = ah0 + ((t & 1) ? kBufStep : 0), al = al0 + ((t & 1) ? kBufStep : 0);
          // The lo piece of the table follows the hi piece row by row in shared memory, so [W_hi | W_lo] is one
          // operand of 2*NB rows: hi x [W_hi | W_lo] is ONE MMA of N = 2*NB (the data operand is read once, not
          // twice), and the hi*hi sums (columns 0..NB-1) stay apart from the small products (columns NB..2NB-1, where
          // lo x W_hi is added), which the store adds in round-to-nearest fp32.  D2 takes the group's whole tensor
          // memory: D1 has been drained, A1 consumed.
          const uint32_t d = tmem + g * 128;
#pragma unroll
          for (int k = 0; k < KS; ++k) {
            ptx::mma_f16_ss(d, ah + 2 * k, wh + 2 * k, idesc_wide, k != 0);
            ptx::mma_f16_ss(d + NB, al + 2 * k, wh + 2 * k, idesc, 1);
          }
          ptx::tc_commit(&sh.a2_empty[g]);
          ptx::tc_commit(&sh.d2_full[g]);
        }
      }
    } else if (STAGE_OUT) {
      // ---------------------------------------------------------- warp 3: finished stages leave as TMA stores
      long long istage = 0;
      for (long long sidx = cta; sidx < p.num_stages; sidx += ncta, ++istage) {
        const uint32_t s = uint32_t(istage % p.raw_stages), ph = uint32_t(istage / p.raw_stages) & 1;
        F16_WAIT_WARP(&sh.out_ready[s], ph, 0x902);
        if (lane == 0) {
          const uint8_t* stage = smem_rawring + size_t(s) * p.stage_bytes;
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
          ptx::mbar_arrive(&sh.raw_empty[s]);
        }
        __syncwarp();
      }
      if (lane == 0) ptx::tma_store_wait_all();
    }
  } else {
    // ------------------------------------------------------------ worker groups: every fourth M-tile, start to end
    ptx::setmaxnreg_inc<FFT16_REGS_WORK>();
    const int g = (warp - 4) >> 2;              // group = tile number mod 4
    const int q = warp & 3;                     // lane quarter of tensor memory this warp may touch
    const int m = q * 32 + lane;
    // stage-1 lane = (sub-line sl1, beta), beta fastest; stage-2 lane = (sub-line sl2, k1)
    const int sl1 = m / R, beta = m % R;
    // Which line of the stage and which butterfly output a sub-line is.  CONTIG: the RX sub-lines of a line sit in one
    // M-tile.  STRIDED with RX >= 2: an M-tile holds the SAME butterfly output of SL neighbouring lines (tiles RX*u ..
    // RX*u + RX-1 are the RX outputs of lines u*SL ...), so that a stage-2 store still covers SL neighbouring columns of
    // one output row (32 bytes) instead of SL/2.
    constexpr bool kPairTiles = (MODE == FFT_STRIDED) && (RX >= 2);
    const int g1 = kPairTiles ? sl1 : sl1 / RX;         // line within the tile (kPairTiles: within the pair of tiles)
    const int bsel1_fixed = sl1 % RX;
    // stage-2 lanes.  CONTIG: (line, k1, butterfly output), output fastest, so that the lanes of a warp store
    // consecutive outputs X[RX*k1 + b] of one line; STRIDED: (k1, sub-line), sub-line fastest (neighbouring columns).
    const int sl2 = (MODE == FFT_CONTIG) ? (m / (RX * R)) * RX + (m % RX) : m % SL;
    const int k1 = (MODE == FFT_CONTIG) ? (m % (RX * R)) / RX : m / SL;
    const int g2 = kPairTiles ? sl2 : sl2 / RX;
    const int bsel2_fixed = sl2 % RX;
    const uint32_t tm_d1 = tmem + (uint32_t(q * 32) << 16) + g * 128;
    const uint32_t tm_a1 = tm_d1 + 64;          // A1 (hi | lo); D2 takes the whole 128 columns
    // A2 row (= stage-2 lane) of (sub-line, k1): CONTIG line*RX*R + RX*k1 + b ; STRIDED k1*SL + sl.
    // K position (beta, re/im) = halves 2*beta, 2*beta+1 of the row: 16-byte chunk beta/4 (XORed with row % 8 by the
    // 128-byte swizzle), word beta%4.  row % 8 takes kSwzPer different values as k1 runs: offsets for each of them.
    constexpr int row_mul_k1 = (MODE == FFT_CONTIG) ? RX : SL;
    constexpr int kSwzPer = (row_mul_k1 >= 8) ? 1 : 8 / row_mul_k1;
    uint32_t a2_off[kSwzPer];                   // byte offset of (row of k1 = v, this beta) minus v * row_mul_k1 * 128
    {
      const int row_base = (MODE == FFT_CONTIG) ? (sl1 / RX) * RX * R + (sl1 % RX) : sl1;
      const uint32_t a2_chunk = uint32_t(beta) >> 2;
      const uint32_t a2_word = uint32_t(beta & 3) * 4u;
#pragma unroll
      for (int v = 0; v < kSwzPer; ++v) {
        const uint32_t r = uint32_t(row_base + v * row_mul_k1) & 7u;
        a2_off[v] = uint32_t(row_base) * 128u + ((a2_chunk ^ r) << 4) + a2_word;
      }
    }
    const float om1 = pp.out_mul;
    const bool st_hints = FUSE != FUSE_NONE && fz.evict_hints;
    const uint64_t pol_store = st_hints ? (FUSE == FUSE_WRITER ? ptx::l2_policy_evict_last() : ptx::l2_policy_evict_first()) : 0;

    for (long long t = g; t < my_mtiles; t += 4) {
      const long long istage = t / p.mtiles_per_stage;
      const int mt = int(t % p.mtiles_per_stage);
      const long long sidx = (long long)cta + istage * ncta;
      const uint32_t s = uint32_t(istage % p.raw_stages), phs = uint32_t(istage / p.raw_stages) & 1;
      const uint32_t pk = uint32_t(t >> 2) & 1;
      uint8_t* stage = smem_rawring + size_t(s) * p.stage_bytes;
      const int bsel1 = kPairTiles ? (mt % RX) : bsel1_fixed, bsel2 = kPairTiles ? (mt % RX) : bsel2_fixed;
      const int col0 = kPairTiles ? (mt / RX) * SL : mt * Lg;     // first column of the stage this tile's lines occupy

      // ---- split: this lane's R elements (after the butterfly when RX == 2) -> scaled fp16 pieces -> A1
      F16_WAIT_WARP(&sh.raw_full[s], phs, 0x701);
      float inv_scale;
      {
        uint32_t base, stride, half;
        if (MODE == FFT_CONTIG) {
          base = uint32_t(g1 * p.N + beta) * 8u;
          stride = uint32_t(R) * 8u;
          half = uint32_t(NL) * 8u;
        } else {
          const int c = col0 + g1;                  // column within the stage
          const uint32_t swz = (COLS == 16) ? uint32_t(beta & 7) : (COLS == 8 ? uint32_t((beta >> 1) & 3) : 0u);   // TMA swizzle of the row (none for 32-byte rows)
          base = uint32_t(beta) * kRowBytes + ((uint32_t(c >> 1) ^ swz) << 4) + uint32_t(c & 1) * 8u;
          stride = uint32_t(R) * kRowBytes;
          half = uint32_t(NL) * kRowBytes;
        }
        float xr[R], xi[R];
        float mxf = 0.0f;                           // largest magnitude of this lane's elements
#pragma unroll
        for (int l = 0; l < R; ++l) {
          const uint2 v = *reinterpret_cast<const uint2*>(stage + base + uint32_t(l) * stride);
          if (RX == 1) {
            xr[l] = __uint_as_float(v.x); xi[l] = __uint_as_float(v.y);
          } else if (RX == 4) {
            // radix-4 butterfly: u_q = x[m + q*N/4]; y_0 = (u0+u2)+(u1+u3), y_2 = (u0+u2)-(u1+u3),
            // y_1 = (u0-u2) + w(u1-u3), y_3 = (u0-u2) - w(u1-u3) with w = exp(s*2*pi*i/4) = s*i; then the twiddle
            const uint2 v1 = *reinterpret_cast<const uint2*>(stage + base + half + uint32_t(l) * stride);
            const uint2 v2 = *reinterpret_cast<const uint2*>(stage + base + 2 * half + uint32_t(l) * stride);
            const uint2 v3 = *reinterpret_cast<const uint2*>(stage + base + 3 * half + uint32_t(l) * stride);
            const float u0r = __uint_as_float(v.x), u0i = __uint_as_float(v.y), u1r = __uint_as_float(v1.x), u1i = __uint_as_float(v1.y);
            const float u2r = __uint_as_float(v2.x), u2i = __uint_as_float(v2.y), u3r = __uint_as_float(v3.x), u3i = __uint_as_float(v3.y);
            float yr, yi;
            if ((bsel1 & 1) == 0) {
              const float ar = u0r + u2r, ai = u0i + u2i, cr = u1r + u3r, ci = u1i + u3i;
              yr = bsel1 == 0 ? ar + cr : ar - cr;
              yi = bsel1 == 0 ? ai + ci : ai - ci;
            } else {
              const float br = u0r - u2r, bi = u0i - u2i, dr = u1r - u3r, di = u1i - u3i;
              const float wr = -pp.quarter_turn * di, wi = pp.quarter_turn * dr;       // (s*i) * d
              yr = bsel1 == 1 ? br + wr : br - wr;
              yi = bsel1 == 1 ? bi + wi : bi - wi;
            }
            if (bsel1 == 0) {
              xr[l] = yr; xi[l] = yi;
            } else {
              const float2 tw = __ldg(p.twiddle2 + (bsel1 - 1) * NL + l * R + beta);   // exp(s*2*pi*i*b*m/N)
              xr[l] = yr * tw.x - yi * tw.y; xi[l] = yr * tw.y + yi * tw.x;
            }
          } else {
            const uint2 w = *reinterpret_cast<const uint2*>(stage + base + half + uint32_t(l) * stride);
            const float ur = __uint_as_float(v.x), ui = __uint_as_float(v.y);
            const float vr = __uint_as_float(w.x), vi = __uint_as_float(w.y);
            if (bsel1 == 0) {
              xr[l] = ur + vr; xi[l] = ui + vi;
            } else {
              const float2 tw = smem_tw2[l * R + beta];
              const float dr = ur - vr, di = ui - vi;
              xr[l] = dr * tw.x - di * tw.y; xi[l] = dr * tw.y + di * tw.x;
            }
          }
          mxf = fmaxf(mxf, fmaxf(fabsf(xr[l]), fabsf(xi[l])));
        }
        if (!STAGE_OUT) {
          // the raw stage is refilled by TMA (async proxy): order this thread's reads before that write
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            ptx::mbar_arrive(&sh.raw_empty[s]);
            if (FUSE == FUSE_READER) {
              // this warp's share of the plane has left the ring (the load had landed before raw_full completed)
              __threadfence();
              atomicAdd(fz.consumed + sidx / p.fuse_stages_per_plane, 1u);
            }
          }
        } else if (kPairTiles) {
          // the results return into the raw stage, and the RX tiles of a group of lines all read ALL rows of those
          // lines: none of them may store before the others have read (the tile without twiddles is well ahead)
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&sh.split_done[s]);
        }
        // the line's largest magnitude over its R lanes (all beta), then 2^(13 - e) and 2^(e - 13) from the exponent
        // field f = e + 127, clamped so that both are normal floats (lines of subnormal-sized data lose nothing:
        // after the largest safe scaling, 2^126, they are multiples of 2^-23)
        // (as bits: non-negative floats order like integers)
        const uint32_t mx = __reduce_max_sync(R == 32 ? 0xffffffffu : (0xffffu << (lane & 16)), __float_as_uint(mxf));
        const uint32_t f = max(mx >> 23, 14u);
        const float in_scale = __uint_as_float((267u - f) << 23);
        const uint64_t scale2 = pack2(in_scale, in_scale);
        inv_scale = __uint_as_float((f - 13u) << 23);
        if (MODE == FFT_STRIDED || RX >= 2) {
          // the stage-2 lanes of this thread belong to another (sub-)line: exchange through shared memory
          // (a bounded mbarrier rather than a named barrier: a warp that gave up a wait must not strand the others)
          if (beta == 0) sh.line_scale[g][sl1] = inv_scale;
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&sh.sc_full[g]);
          F16_WAIT_WARP(&sh.sc_full[g], pk, 0x703);
          inv_scale = sh.line_scale[g][sl2];
        }
#pragma unroll
        for (int l0 = 0; l0 < R; l0 += 16) {        // 16 complex = 16 packed columns per tensor-memory store
          uint32_t hw[16], lw[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) split_half2(mul2(pack2(xr[l0 + j], xi[l0 + j]), scale2), hw[j], lw[j]);
          ptx::tmem_st_32x16(tm_a1 + l0, hw);
          ptx::tmem_st_32x16(tm_a1 + R + l0, lw);
        }
        ptx::tc_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.a1_full[g]);
      }

      // ---- drain stage 1: twiddle, split, write the stage-2 operand (buffer t & 1)
      F16_WAIT_WARP(&sh.d1_full[g], pk, 0x801);
      ptx::tc_fence_after();
      {
        uint8_t* a2buf = smem_a2 + size_t(t & 1) * 2 * a2_piece;
#pragma unroll
        for (int c = 0; c < K / 32; ++c) {          // 16 values of k1 per chunk of 32 accumulator columns
          uint32_t v0[32];
          ptx::tmem_ld_32x32(tm_d1 + c * 32, v0);
          ptx::tc_wait_ld();
          uint32_t ch[16], cl[16];                  // C[k1] for this lane's beta, as packed fp16 pieces
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 tw = smem_tw[(c * 16 + j) * R + beta];
            const float br = __uint_as_float(v0[2 * j]);
            const float bi = __uint_as_float(v0[2 * j + 1]);
            split_half2(pack2(br * tw.x - bi * tw.y, br * tw.y + bi * tw.x), ch[j], cl[j]);
          }
          if (c == 0 && t >= 2) {
            // stage 2 of tile t - 2 (group g ^ 2) must be done reading this buffer
            F16_WAIT_WARP(&sh.a2_empty[g ^ 2], uint32_t((t - 2) >> 2) & 1, 0x802);
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int k1i = c * 16 + j;
            uint8_t* dst2 = a2buf + a2_off[k1i % kSwzPer] + k1i * row_mul_k1 * 128;
            *reinterpret_cast<uint32_t*>(dst2) = ch[j];
            *reinterpret_cast<uint32_t*>(dst2 + a2_piece) = cl[j];
          }
        }
        ptx::tc_fence_before();
        ptx::fence_proxy_async_smem();                // generic writes -> visible to the MMA's shared-memory reads
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh.a2_full[g]);
      }

      // ---- drain stage 2: undo the scales, store in natural order
      {
        float2* dst;              // &out[line][RX*k1 + bsel]; output k = RX*(k1 + R*k2) + bsel is k2*k2_stride further
        long long k2_stride;
        bool ok;
        if (MODE == FFT_CONTIG) {
          const long long line = sidx * Lg + g2;
          ok = line < p.rows;
          dst = reinterpret_cast<float2*>(p.out) + line * p.N + (RX * k1 + bsel2);
          k2_stride = RX * R;
        } else {
          const long long ct = sidx % p.c_tiles, bt = sidx / p.c_tiles;
          const long long col = ct * COLS + col0 + g2;
          ok = col < p.C;
          if (p.out_blocked) {
            // block [k][COLS] number n2tile*blk_rows + i1 of the blocked intermediate: pieces of one block are close
            // together, so plain stores from registers do (the L2 merges them into full lines)
            // (blk_pair = P > 1: P neighbouring rows i1 interleave their pieces, T[n2 tile][i1 / P][k][i1 % P][COLS])
            const long long i1 = ct / p.blk_tiles, P = p.blk_pair;
            const long long blk = (ct % p.blk_tiles) * (p.blk_rows / P) + i1 / P;
            dst = reinterpret_cast<float2*>(p.out) + ((blk * p.N + (RX * k1 + bsel2)) * P + i1 % P) * COLS + (col0 + g2);
            k2_stride = (long long)(RX * R) * COLS * P;
          } else {
            const long long slot = (FUSE == FUSE_WRITER) ? bt % fz.ring : bt;
            dst = reinterpret_cast<float2*>(p.out) + (slot * p.N + (RX * k1 + bsel2)) * p.out_pitch + p.out_off + col;
            k2_stride = (long long)(RX * R) * p.out_pitch;
          }
        }
        // one factor when the product of the two is a normal float (always, except for subnormal-sized data)
        float om = om1 * inv_scale, om_b = 1.0f;
        if (!(om >= 1.1754944e-38f)) { om = om1; om_b = inv_scale; }
        F16_WAIT_WARP(&sh.d2_full[g], pk, 0x901);
        if (STAGE_OUT && kPairTiles) F16_WAIT_WARP(&sh.split_done[s], phs, 0x903);
        ptx::tc_fence_after();
        const uint64_t om2 = pack2(om, om);
#pragma unroll
        for (int ch = 0; ch < K / 32; ++ch) {
          uint32_t va[32], vb[32];                    // hi*hi sums and the small products of the same outputs
          ptx::tmem_ld_32x32(tm_d1 + ch * 32, va);
          ptx::tmem_ld_32x32(tm_d1 + NB + ch * 32, vb);
          ptx::tc_wait_ld();
          float f[32];
#pragma unroll
          for (int j = 0; j < 16; ++j)
            unpack2(mul2(add2(pack2(__uint_as_float(va[2 * j]), __uint_as_float(va[2 * j + 1])),
                              pack2(__uint_as_float(vb[2 * j]), __uint_as_float(vb[2 * j + 1]))), om2),
                    f[2 * j], f[2 * j + 1]);
          if (om_b != 1.0f) {
#pragma unroll
            for (int j = 0; j < 32; ++j) f[j] *= om_b;
          }
          if (STAGE_OUT) {
            // element (row k, column c) of the stage, in the layout TMA wrote the input in (same swizzle)
            const int c = col0 + g2;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int k = RX * (k1 + R * (ch * 16 + j)) + bsel2;
              const uint32_t swz = (COLS == 16) ? uint32_t(k & 7) : (COLS == 8 ? uint32_t((k >> 1) & 3) : 0u);
              const uint32_t off = uint32_t(k) * kRowBytes + ((uint32_t(c >> 1) ^ swz) << 4) + uint32_t(c & 1) * 8u;
              *reinterpret_cast<float2*>(stage + off) = make_float2(f[2 * j], f[2 * j + 1]);
            }
          } else if (ok) {
            if (MODE == FFT_CONTIG) {
              float2* pd = dst + ch * 16 * (RX * R);  // compile-time stride: immediate offsets
              if (st_hints) {
#pragma unroll
                for (int j = 0; j < 16; ++j) ptx::st_global_v2_hint(pd + j * (RX * R), f[2 * j], f[2 * j + 1], pol_store);
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) pd[j * (RX * R)] = make_float2(f[2 * j], f[2 * j + 1]);
              }
            } else {
              float2* pd = dst + (long long)(ch * 16) * k2_stride;
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                if (st_hints) ptx::st_global_v2_hint(pd, f[2 * j], f[2 * j + 1], pol_store);
                else *pd = make_float2(f[2 * j], f[2 * j + 1]);
                pd += k2_stride;
                asm volatile("" : "+l"(pd));          // one running pointer, not sixteen precomputed ones
              }
            }
          }
        }
        ptx::tc_fence_before();                       // the next tile's split overwrites these columns
        if (FUSE == FUSE_WRITER) {
          // this warp's stores of the tile are out: make them visible, then count the warp in for the plane
          __threadfence();
          __syncwarp();
          if (lane == 0) atomicAdd(fz.written + sidx / p.fuse_stages_per_plane, 1u);
        }
        if (STAGE_OUT) {
          ptx::fence_proxy_async_smem();              // generic writes -> visible to the TMA store
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&sh.out_ready[s]);
        }
      }
    }
  }

role_done:
#ifdef DFT3D_PROFILE_WAITS
  if (p.profile && lane == 0 && (warp <= 3 || (warp & 3) == 0)) {
    // one reporter per role / group: rows 5..9 by wait code, column by code & 7; workers add up over the groups
    long long* dst = p.profile + size_t(cta) * 128;
    for (int i = 5; i < 10; ++i)
      for (int j = 0; j < 8; ++j)
        if (prof_wait[i][j]) atomicAdd(reinterpret_cast<unsigned long long*>(dst + i * 8 + j), (unsigned long long)prof_wait[i][j]);
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

// one axis per launch
template <int MODE, int R, int RX, int COLS, int STAGE_OUT>
__global__ void __launch_bounds__(kFftThreads, 1)
fft_f16_axis_kernel(const __grid_constant__ CUtensorMap map_data, const __grid_constant__ CUtensorMap map_w,
                    const __grid_constant__ CUtensorMap map_out, const FftF16Params pp) {
  const FftFuse none = {};
  fft_f16_axis_body<MODE, R, RX, COLS, STAGE_OUT, FUSE_NONE>(&map_data, &map_w, &map_out, pp, none, int(blockIdx.x),
                                                            int(gridDim.x));
}

// Axes 1 and 2 of a 3D transform in ONE launch (Eq. 17 applied axis after axis, Section IV-D's closing remark): the
// first `ctas_writer` CTAs run the axis-1 pass (strided, COLS-line stages) plane by plane into a ring of a few
// n0-planes, the others run the axis-2 pass (contiguous) out of that ring into the output.  The ring is small enough
// to stay in L2, so the intermediate between the two axes is written and read back there instead of in HBM: 32 bytes
// of HBM traffic per point and transform instead of 48.  Both kinds of CTA take their stages in plane order, and a
// stage waits only for stages that come before it in that order (a reader for the writers of its plane, a writer for
// the readers of the plane that used its ring slot last), so with all CTAs resident (one per SM, grid <= SM count)
// nobody waits for somebody who waits for them.  Both axes have the same length R*R (same table and twiddles).
template <int R, int COLS>
__global__ void __launch_bounds__(kFftThreads, 1)
fft_f16_fused_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_w,
                     const __grid_constant__ CUtensorMap map_ring, const FftF16Params writer, const FftF16Params reader,
                     const FftFuse fz) {
  if (int(blockIdx.x) < fz.ctas_writer)
    fft_f16_axis_body<FFT_STRIDED, R, 1, COLS, 0, FUSE_WRITER>(&map_in, &map_w, &map_in, writer, fz, int(blockIdx.x),
                                                               fz.ctas_writer);
  else
    fft_f16_axis_body<FFT_CONTIG, R, 1, COLS, 0, FUSE_READER>(&map_ring, &map_w, &map_ring, reader, fz,
                                                              int(blockIdx.x) - fz.ctas_writer,
                                                              int(gridDim.x) - fz.ctas_writer);
}

}  // namespace dft3d
