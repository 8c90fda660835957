// The KDFT axis kernel with fp16 pieces (kdft_f16_kernel.cuh) on PAIRS of CTAs: tcgen05.mma cta_group::2.
//
// Two CTAs of a cluster (the two SMs of a TPC) work on one 256-lane x 256-column tile: each CTA owns 128 lanes (its own
// raw data stages, split warps, tensor-memory A stages, accumulator and epilogue) and loads only HALF of every table
// stage (128 of the 256 output columns); the leader CTA's single MMA thread issues M = 256 instructions that read
// A from both CTAs' tensor memory and B from both CTAs' shared memory and write each CTA's own accumulator.  Per SM
// this halves the table bytes brought into shared memory and the bytes each MMA reads from it, which is what held the
// one-CTA kernel at ~0.75 of the tensor peak (96 KB of operands per 1536 issue clocks = 62 B/clk/SM).
//
// Signals.  To the leader (its shared memory, reached through mapa): b_full (both CTAs' table loads complete their
// bytes on the leader's barrier), t_full (4 split warps of each CTA), acc_empty (8 epilogue warps of each CTA).
// From the leader to both CTAs (tcgen05.commit with a CTA mask): b_empty, t_empty, acc_full.  Raw data barriers are
// local.  Both CTAs meet at a cluster barrier after set-up and before they release tensor memory; every other wait
// is bounded as in the one-CTA kernel.
#pragma once
#include <cuda_fp16.h>
#include "kdft_f16_kernel.cuh"

namespace dft3d {

constexpr int kX2StagesB = 4;                       // table stages per CTA (half a tile: 2 pieces x 128 rows x 128 B)
constexpr int kX2BytesStageB = 2 * 128 * 128;
constexpr int kX2StagesA = 2;                       // raw fp32 data stages (32 KB each)

struct KdftX2Shared {
  uint64_t b_full[kX2StagesB], b_empty[kX2StagesB];
  uint64_t a_full[kX2StagesA], a_empty[kX2StagesA];
  uint64_t t_full[kStagesT], t_empty[kStagesT];
  uint64_t acc_full, acc_empty;
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_limit;
};
constexpr size_t kKdftX2SmemBytes = size_t(kX2StagesB) * kX2BytesStageB + size_t(kX2StagesA) * kF16BytesStageA +
                                    sizeof(KdftX2Shared) + 1024;

namespace ptx {
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same variable in the CTA of the given rank
__device__ __forceinline__ uint32_t map_to_cta(const void* local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose bytes complete on a barrier given by its shared::cluster address
// (the leader's): the pair form of the tiled load, no multicast
__device__ __forceinline__ void tma_load_3d_pair(void* smem_dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x,
                                                 int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D (both CTAs' tensor memory, 128 lanes each) (+)= A (both CTAs' tensor memory) * B^T (both CTAs' shared memory halves)
__device__ __forceinline__ void mma_f16_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t"
      "}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this shared-memory offset in both CTAs of the pair once all earlier MMAs are complete
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
}  // namespace ptx

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
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kKdftThreads, 1)
kdft_f16x2_axis_kernel(const __grid_constant__ CUtensorMap map_data, const __grid_constant__ CUtensorMap map_w,
                 const KdftF16Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_b = smem;
  uint8_t* smem_a = smem + size_t(kX2StagesB) * kX2BytesStageB;
  KdftX2Shared& sh = *reinterpret_cast<KdftX2Shared*>(smem_a + size_t(kX2StagesA) * kF16BytesStageA);
  const uint32_t rank = ptx::cluster_ctarank();      // 0 = leader (issues the MMAs), 1 = its peer

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < kX2StagesB; ++i) { ptx::mbar_init(&sh.b_full[i], 1); ptx::mbar_init(&sh.b_empty[i], 1); }
    for (int i = 0; i < kX2StagesA; ++i) { ptx::mbar_init(&sh.a_full[i], 1); ptx::mbar_init(&sh.a_empty[i], 4); }
    for (int i = 0; i < kStagesT; ++i) { ptx::mbar_init(&sh.t_full[i], 8); ptx::mbar_init(&sh.t_empty[i], 1); }   // both CTAs' split warps
    ptx::mbar_init(&sh.acc_full, 1);
    ptx::mbar_init(&sh.acc_empty, 2 * kEpilogueWarps);                                                           // both CTAs' epilogues
    sh.abort_flag = 0;
    sh.wait_limit = p.wc.limit_clocks > 0 ? p.wc.limit_clocks : kDefaultWaitClocks;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(&sh.tmem_base, kTmemCols);
    ptx::tmem_relinquish_pair();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&map_data);
    ptx::prefetch_tensormap(&map_w);
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();            // the peer's barriers are initialised before anything is signalled across
  ptx::tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  // pair tiles: 256 lanes (two M-tiles, one per CTA) x one N-tile; an odd M-tile count leaves the last peer a phantom
  // tile (its loads are out of bounds and zero-filled, its stores masked)
  const long long total_pairs = ((p.m_tiles + 1) / 2) * p.n_tiles;
  // Order of the tile pairs: within a group of n_group table panels all line tiles, panel fastest; then the next group.
  // The pairs that run at the same time then share n_group panels (n_group * 4 MiB at 2048 points) instead of all of
  // them, which keeps the table in L2 at the price of reading the data once per group.
  const long long ng = (p.n_group > 0 && p.n_group < p.n_tiles && p.n_tiles % p.n_group == 0) ? p.n_group : p.n_tiles;
  const long long pairs_per_group = ((p.m_tiles + 1) / 2) * ng;
  const long long pair0 = blockIdx.x >> 1, pair_step = gridDim.x >> 1;
  const int num_kb = (p.k2 + kF16BlockK - 1) / kF16BlockK;   // a ragged last stage is zero-filled by TMA on both operands

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
      if (lane == 0) {
        uint32_t ib = 0, ia = 0;   // running stage counters
        uint32_t leader_b_full[kX2StagesB];
#pragma unroll
        for (int i = 0; i < kX2StagesB; ++i) leader_b_full[i] = ptx::map_to_cta(&sh.b_full[i], 0);
        for (long long tp = pair0; tp < total_pairs; tp += pair_step) {
          const long long mt = 2 * ((tp % pairs_per_group) / ng) + rank;
          const int nt = int((tp / pairs_per_group) * ng + tp % ng);
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
              // this CTA's half of the table stage (columns nt*256 + 128*rank ...); the bytes of both halves complete
              // on the leader's barrier, which the leader arms for the whole stage
              const uint32_t s = ib % kX2StagesB, ph = (ib / kX2StagesB) & 1;
              DFT3D_WAIT(&sh.b_empty[s], ph ^ 1, 0x101);
              if (rank == 0) ptx::mbar_arrive_expect_tx(&sh.b_full[s], 2u * kX2BytesStageB);
              ptx::tma_load_3d_pair(smem_b + size_t(s) * kX2BytesStageB, &map_w, leader_b_full[s], kb * kF16BlockK,
                                    nt * 256 + int(rank) * 128, 0);
              ++ib;
            }
            {
              const uint32_t s = ia % kX2StagesA, ph = (ia / kX2StagesA) & 1;
              DFT3D_WAIT(&sh.a_empty[s], ph ^ 1, 0x102);
              ptx::mbar_arrive_expect_tx(&sh.a_full[s], kF16BytesStageA);
              if (MODE == KDFT_CONTIG) {   // two 128-byte-wide halves (the 128B swizzle spans 32 floats)
                ptx::tma_load_2d(smem_a + size_t(s) * kF16BytesStageA, &map_data, &sh.a_full[s], kb * kF16BlockK, ay);
                ptx::tma_load_2d(smem_a + size_t(s) * kF16BytesStageA + kF16BytesStageA / 2, &map_data, &sh.a_full[s],
                                 kb * kF16BlockK + 32, ay);
              } else
                ptx::tma_load_3d(smem_a + size_t(s) * kF16BytesStageA, &map_data, &sh.a_full[s], ax, kb * (kF16BlockK / 2), az);
              ++ia;
            }
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------ MMA issuer
      if (lane == 0 && rank == 0) {
        const uint32_t idesc = ptx::make_idesc_f16(2 * kTileM, 256);
        uint32_t ib = 0, it = 0, chunk_count = 0;
#ifdef DFT3D_PROFILE_WAITS
        long long w_acc = 0, w_b = 0, w_t = 0, t_begin = clock64(), tq;
#define PW_BEGIN tq = clock64();
#define PW_END(v) v += clock64() - tq;
#else
#define PW_BEGIN
#define PW_END(v)
#endif
        for (long long tp = pair0; tp < total_pairs; tp += pair_step) {
          for (int kb = 0; kb < num_kb; ++kb) {
            const bool chunk_first = (kb % p.chunk_kb) == 0;
            if (chunk_first) {
              // the tensor-core accumulator restarts from zero every chunk (see the epilogue)
              PW_BEGIN
              DFT3D_WAIT(&sh.acc_empty, (chunk_count & 1) ^ 1, 0x201);
              PW_END(w_acc)
              ptx::tc_fence_after();
            }
            const uint32_t sb = ib % kX2StagesB, phb = (ib / kX2StagesB) & 1;
            const uint32_t st = it % kStagesT, pht = (it / kStagesT) & 1;
            PW_BEGIN
            DFT3D_WAIT(&sh.b_full[sb], phb, 0x202);
            PW_END(w_b)
            PW_BEGIN
            DFT3D_WAIT(&sh.t_full[st], pht, 0x203);
            PW_END(w_t)
            ptx::tc_fence_after();
            const uint32_t b_hi = ptx::smem_u32(smem_b + size_t(sb) * kX2BytesStageB);   // same offset in the peer
            const uint32_t b_lo = b_hi + 128u * 128u;
            const uint32_t a_hi = tmem + kAccCols + st * 64;
            const uint32_t a_lo = a_hi + 32;
#pragma unroll
            for (int k = 0; k < kF16BlockK / 16; ++k) {   // K = 16 per MMA: 8 packed columns of A, 32 bytes of each B row
              const uint64_t dhi = ptx::make_kmajor_sw128_desc(b_hi + k * 32);
              const uint64_t dlo = ptx::make_kmajor_sw128_desc(b_lo + k * 32);
              ptx::mma_f16_ts_pair(tmem, a_hi + k * 8, dhi, idesc, (k != 0 || !chunk_first) ? 1u : 0u);
              ptx::mma_f16_ts_pair(tmem, a_lo + k * 8, dhi, idesc, 1);
              ptx::mma_f16_ts_pair(tmem, a_hi + k * 8, dlo, idesc, 1);
            }
            ptx::tc_commit_pair(&sh.b_empty[sb]);
            ptx::tc_commit_pair(&sh.t_empty[st]);
            ++ib;
            ++it;
            if ((kb + 1) % p.chunk_kb == 0 || kb + 1 == num_kb) {
              ptx::tc_commit_pair(&sh.acc_full);
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
    if (MODE == KDFT_STRIDED) strided_off = (m / p.lpb) * (kF16BlockK / 2) * p.lpb + (m % p.lpb);
    const uint64_t scale2 = pack2(in_scale, in_scale);
    uint32_t ia = 0, it = 0;
    for (long long tp = pair0; tp < total_pairs; tp += pair_step) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const uint32_t sa = ia % kX2StagesA, pha = (ia / kX2StagesA) & 1;
        const uint32_t st = it % kStagesT, pht = (it / kStagesT) & 1;
        DFT3D_WAIT_WARP(&sh.a_full[sa], pha, 0x301);
        uint32_t ph[32], pl[32];                 // 64 scaled values as fp16 pairs: hi pieces, lo pieces
        const uint8_t* stage = smem_a + size_t(sa) * kF16BytesStageA;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t x[32];
          if (MODE == KDFT_CONTIG) {
            const uint4* rowp = reinterpret_cast<const uint4*>(stage + h * (kF16BytesStageA / 2) + m * 128);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const uint4 v = rowp[c ^ (m & 7)];
              x[4 * c] = v.x; x[4 * c + 1] = v.y; x[4 * c + 2] = v.z; x[4 * c + 3] = v.w;
            }
          } else {
            const uint2* colp = reinterpret_cast<const uint2*>(stage) + strided_off;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const uint2 v = colp[(h * 16 + j) * p.lpb];
              x[2 * j] = v.x; x[2 * j + 1] = v.y;
            }
          }
          if (h == 1) {
            // the stage is refilled by TMA (async proxy): order this thread's reads before that write
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sh.a_empty[sa]);
          }
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
        if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(&sh.t_full[st], 0));
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
    for (long long tp = pair0; tp < total_pairs; tp += pair_step) {
      const long long mt = 2 * ((tp % pairs_per_group) / ng) + rank;
      const int nt = int((tp / pairs_per_group) * ng + tp % ng);
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
        if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(&sh.acc_empty, 0));
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
  ptx::cluster_sync_all();            // neither CTA lets go of its shared / tensor memory while the other may touch it
  if (warp == 1) ptx::tmem_dealloc_pair(tmem, kTmemCols);
}

#undef DFT3D_WAIT
#undef DFT3D_WAIT_WARP

}  // namespace dft3d
