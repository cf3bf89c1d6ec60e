// MXFP4 x MXFP4 block-scaled GEMM on the 5th-generation tensor cores (stage 3).
//
//   Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} qx[s,j,i] * qw[m,j,i]
//
// the low-bit matrix multiplication Q(XP) Q(P^-1 W^T) of the paper's Sec. 3.
//
// Persistent CTAs, one per SM, each walking a strided list of 128 x BN output
// tiles.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (one elected
// lane) and tensor-memory owner, warps 2..5 = epilogue.  A K-step is 256
// elements = 128 bytes of packed codes per row = one 128-byte swizzle atom,
// i.e. four tcgen05.mma of K = 64.  The E8M0 scale bytes travel as 512-byte
// atoms (128 rows x 4 blocks), are copied shared -> tensor memory with
// tcgen05.cp and read by the MMA from there.
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace batq {

constexpr int kGemmThreads = 192;
constexpr int kBM = 128;
constexpr int kBKBytes = 128;  // 256 four-bit elements

template <int BN>
struct GemmCfg {
  static constexpr int kABytes = kBM * kBKBytes;       // 16 KiB
  static constexpr int kBBytes = BN * kBKBytes;
  static constexpr int kSfaBytes = 1024;                 // 128 rows x 8 blocks
  static constexpr int kSfbBytes = (BN / 128) * 1024;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr int kAccStages = (BN == 256) ? 1 : 2;
  static constexpr int kAccCols = BN * kAccStages;
  static constexpr int kSfColsPerStage = 8 + 2 * (BN / 32);  // A: 2 chunks x 4, B: 2 chunks x BN/32
  static constexpr int kTmemCols = 512;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024;  // + alignment slack
  static constexpr uint32_t kTxBytes = kStageBytes;
  static_assert(kAccCols + kStages * kSfColsPerStage <= kTmemCols, "tensor memory budget");
};

struct GemmParams {
  const uint8_t* sfa;  // activation scales, BATQ_SF_MMA layout
  const uint8_t* sfb;  // weight scales, BATQ_SF_MMA layout
  void* y;
  int64_t ldy;
  int32_t s;           // rows of X (tokens)
  int32_t m;           // rows of W (output features)
  int32_t k_bytes;     // n / 2
  int32_t katoms;      // KA = 2*ceil(k/8)
  int32_t k_steps;     // ceil(n / 256)
  int32_t m_tiles;     // ceil(s / 128)
  int32_t n_tiles;     // ceil(m / BN)
  int32_t sfa_row_tiles;  // ceil(s / 128)
  int32_t sfb_row_tiles;  // ceil(m / 128)
};

// Instruction descriptor of tcgen05.mma kind::mxf4.block_scale:
//   [4,6) B scale id   [7,10) A format (E2M1 = 1)   [10,13) B format   [15] A major (0 = K)
//   [16] B major       [17,23) N >> 3               [23] scale format (1 = UE8M0)
//   [24,29) M >> 4     [29,31) A scale id           [31] K size (0 = 64)
__host__ __device__ constexpr uint32_t mxf4_idesc(int M, int N) {
  return (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) | (1u << 23) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

template <int BN, bool OUT_BF16>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_mxfp4_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const GemmParams p) {
  using Cfg = GemmCfg<BN>;
  extern __shared__ uint8_t gemm_smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t acc_full_bar[2];
  __shared__ __align__(8) uint64_t acc_empty_bar[2];
  __shared__ __align__(8) uint64_t drain_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(gemm_smem_raw) + 1023) & ~uintptr_t(1023));

  if (tid == 0) {
    for (int i = 0; i < Cfg::kStages; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&acc_full_bar[i]), 1);
      mbar_init(smem_u32(&acc_empty_bar[i]), 4);
    }
    mbar_init(smem_u32(&drain_bar), 1);
    abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_b);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  const int total_tiles = p.m_tiles * p.n_tiles;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int mt = tile % p.m_tiles;
        const int nt = tile / p.m_tiles;
        const int m0 = mt * kBM;
        const int n0 = nt * BN;
        for (int kt = 0; kt < p.k_steps; ++kt) {
          ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, &abort_flag);
          if (!ok) break;
          uint8_t* st = smem + stage * Cfg::kStageBytes;
          const uint32_t bar = smem_u32(&full_bar[stage]);
          mbar_arrive_expect_tx(bar, Cfg::kTxBytes);
          tma_load_2d(smem_u32(st), &tmap_a, kt * kBKBytes, m0, bar);
          tma_load_2d(smem_u32(st + Cfg::kABytes), &tmap_b, kt * kBKBytes, n0, bar);
          bulk_g2s(smem_u32(st + Cfg::kABytes + Cfg::kBBytes),
                   p.sfa + (static_cast<int64_t>(mt) * p.katoms + 2 * kt) * 512, 1024, bar);
#pragma unroll
          for (int rt = 0; rt < BN / 128; ++rt) {
            const int row_tile = min(nt * (BN / 128) + rt, p.sfb_row_tiles - 1);
            bulk_g2s(smem_u32(st + Cfg::kABytes + Cfg::kBBytes + Cfg::kSfaBytes + rt * 1024),
                     p.sfb + (static_cast<int64_t>(row_tile) * p.katoms + 2 * kt) * 512, 1024, bar);
          }
          ++issued;
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Given up: let the copies already in flight land before the CTA exits.
        const int pending = min(issued, Cfg::kStages);
        for (int i = 0; i < pending; ++i) {
          if (--stage < 0) { stage = Cfg::kStages - 1; phase ^= 1u; }
          const uint32_t bar = smem_u32(&full_bar[stage]);
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(bar, phase) && global_timer_ns() - t0 < 100000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc0 = mxf4_idesc(kBM, BN);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = it % Cfg::kAccStages;
        const uint32_t acc_phase = (it / Cfg::kAccStages) & 1u;
        ok = mbar_wait(smem_u32(&acc_empty_bar[acc]), acc_phase ^ 1u, &abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kt = 0; kt < p.k_steps; ++kt) {
          ok = mbar_wait(smem_u32(&full_bar[stage]), phase, &abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          uint8_t* st = smem + stage * Cfg::kStageBytes;
          const uint32_t sf_col = tmem_base + Cfg::kAccCols + stage * Cfg::kSfColsPerStage;
          const uint32_t sfa_col = sf_col;           // chunk c at +4c
          const uint32_t sfb_col = sf_col + 8;       // chunk c at +c*(BN/32), row tile rt at +4rt
          const uint32_t sfa_smem = smem_u32(st + Cfg::kABytes + Cfg::kBBytes);
          const uint32_t sfb_smem = sfa_smem + Cfg::kSfaBytes;
#pragma unroll
          for (int c = 0; c < 2; ++c)
            tc_cp_32x128b_warpx4(sfa_col + 4 * c, make_smem_desc(sfa_smem + c * 512, 0, 128, 0));
#pragma unroll
          for (int rt = 0; rt < BN / 128; ++rt)
#pragma unroll
            for (int c = 0; c < 2; ++c)
              tc_cp_32x128b_warpx4(sfb_col + c * (BN / 32) + 4 * rt,
                                   make_smem_desc(sfb_smem + rt * 1024 + c * 512, 0, 128, 0));
          const uint64_t adesc = make_smem_desc(smem_u32(st), 16, 1024, 2);
          const uint64_t bdesc = make_smem_desc(smem_u32(st + Cfg::kABytes), 16, 1024, 2);
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint32_t c = kb >> 1;
            const uint32_t sfid = (kb & 1) * 2;  // byte pair inside the 32-bit scale column
            const uint32_t idesc = idesc0 | (sfid << 29) | (sfid << 4);
            tc_mma_mxf4(d_tmem, adesc + 2 * kb, bdesc + 2 * kb, idesc, (sfa_col + 4 * c) | (sfid << 30),
                        (sfb_col + c * (BN / 32)) | (sfid << 30), (kt | kb) != 0 ? 1u : 0u);
          }
          tc_commit(smem_u32(&empty_bar[stage]));  // frees the stage once these MMAs have read it
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(smem_u32(&acc_full_bar[acc]));
      }
      // All tensor-core work of this CTA done (or abandoned) before the memory is released.
      tc_commit(smem_u32(&drain_bar));
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(smem_u32(&drain_bar), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
    }
  } else {
    // ---------------------------------------------------------------- epilogue warps
    const int quad = warp & 3;  // tensor-memory lanes [32*quad, 32*quad + 32) belong to this warp
    int it = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
      const int mt = tile % p.m_tiles;
      const int nt = tile / p.m_tiles;
      const int acc = it % Cfg::kAccStages;
      const uint32_t acc_phase = (it / Cfg::kAccStages) & 1u;
      bool ok = mbar_wait(smem_u32(&acc_full_bar[acc]), acc_phase, &abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const int row = mt * kBM + quad * 32 + lane;
      const uint32_t taddr = tmem_base + acc * BN + (static_cast<uint32_t>(quad * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(taddr + c0, r);
        tmem_ld_wait();
        const int col0 = nt * BN + c0;
        if (row < p.s && col0 < p.m) {
          if (OUT_BF16) {
            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<int64_t>(row) * p.ldy + col0;
            if (col0 + 32 <= p.m) {
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                uint32_t w[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                  const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * h]),
                                                                 __uint_as_float(r[8 * v + 2 * h + 1]));
                  w[h] = *reinterpret_cast<const uint32_t*>(&b);
                }
                reinterpret_cast<uint4*>(yp)[v] = make_uint4(w[0], w[1], w[2], w[3]);
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (col0 + i < p.m) yp[i] = __float2bfloat16_rn(__uint_as_float(r[i]));
            }
          } else {
            float* yp = reinterpret_cast<float*>(p.y) + static_cast<int64_t>(row) * p.ldy + col0;
            if (col0 + 32 <= p.m) {
#pragma unroll
              for (int v = 0; v < 8; ++v)
                reinterpret_cast<uint4*>(yp)[v] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (col0 + i < p.m) yp[i] = __uint_as_float(r[i]);
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty_bar[acc]));
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

}  // namespace batq
