// MXFP8 (E4M3) activations x MXFP4 (E2M1) weights, block-scaled GEMM (stage 3 of the W4A8
// configurations of Sec. 4):
//
//   Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} q8x[s,j,i] * q4w[m,j,i]
//
// tcgen05.mma kind::mxf8f6f4 takes both element types in 8-bit containers: the activations are
// one byte per code already; the packed 4-bit weight codes are widened on the way into shared
// memory by the TMA unit itself (tensor-map type 16U4_ALIGN16B: every 8 bytes of 16 packed codes
// land in a 16-byte slot), so HBM and L2 still carry 0.5 byte per weight.  A K-step is 128
// elements = one 128-byte swizzle row of either operand = four MMAs of K = 32, each with one
// scale byte per row (the four bytes of one 32-bit scale column; one 512-byte atom per 128 rows
// and K-step).  Otherwise the kernel is organised like gemm_mxfp4.cuh: persistent CTAs, warp 0 =
// TMA producer, warp 1 = MMA issuer and tensor-memory owner, warps 2..5 = epilogue, accumulators
// double buffered in tensor memory for the 128-wide tile.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_mxfp4.cuh"
#include "ptx.cuh"

namespace batq {

constexpr int kW4A8KElems = 128;   // elements per K-step

template <int BN>
struct W4A8Cfg {
  static constexpr int kABytes = kBM * 128;               // E4M3 codes, 128 per row
  static constexpr int kBBytes = BN * 128;                // E2M1 codes in 8-bit containers, 128 per row
  static constexpr int kSfbAtoms = (BN + 127) / 128;
  static constexpr int kSfBytes = ((512 + kSfbAtoms * 512 + 1023) / 1024) * 1024;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfBytes;
  static constexpr int kStages = (BN == 256) ? 4 : 5;
  static constexpr int kAccStages = (BN == 256) ? 1 : 2;
  static constexpr int kAccCols = BN * kAccStages;
  static constexpr int kSfColsPerStage = 4 + 4 * kSfbAtoms;
  static constexpr int kTmemCols = 512;
  static constexpr int kStagingBufs = (BN == 256) ? 1 : 2;
  static constexpr int kStagingBytes = 4 * kStagingBufs * 4096;
  static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024;
  static_assert(BN == 128 || BN == 256, "tile width");
  static_assert(kAccCols + kStages * kSfColsPerStage <= kTmemCols, "tensor memory budget");
  static_assert(kSmemBytes <= 232448, "shared memory budget");
  static_assert(kStageBytes % 1024 == 0, "stage alignment");
};

struct W4A8Params {
  const uint8_t* sfa;     // activation scales, BATQ_SF_MMA layout
  const uint8_t* sfb;     // weight scales, BATQ_SF_MMA layout
  int32_t s, m;
  int32_t katoms;         // 2*ceil(k/8) atoms per 128-row tile
  int32_t k_steps;        // n / 128
  int32_t m_tiles, n_tiles;
  int32_t sfb_row_tiles;  // ceil(m / 128)
  int32_t m16;            // columns covered by the TMA store (see GemmParams)
  int32_t b_row_tx;       // bytes one weight row of a K-step adds to the barrier's transaction count
  void* y;
  int64_t ldy;
};

// Instruction descriptor of tcgen05.mma kind::mxf8f6f4.block_scale (same fields as mxf4_idesc; the
// 8-bit-container kinds number their formats E4M3 = 0, E5M2 = 1, E2M3 = 3, E3M2 = 4, E2M1 = 5).
__host__ __device__ constexpr uint32_t mxf8f6f4_idesc_e4m3_e2m1(int M, int N) {
  return (0u << 7) | (5u << 10) | (static_cast<uint32_t>(N >> 3) << 17) | (1u << 23) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem], 8-bit containers, one UE8M0 scale per 32 along K, K = 32.
__device__ __forceinline__ void tc_mma_mxf8f6f4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate)
      : "memory");
}

template <int BN, bool OUT_BF16>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_w4a8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_y, const W4A8Params p) {
  using Cfg = W4A8Cfg<BN>;
  extern __shared__ uint8_t w4a8_smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t acc_full_bar[2];
  __shared__ __align__(8) uint64_t acc_empty_bar[2];
  __shared__ __align__(8) uint64_t drain_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  grid_launch_dependents();
  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const int lane = tid & 31;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(w4a8_smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + Cfg::kStages * Cfg::kStageBytes;

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
    tma_prefetch_desc(&tmap_y);
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
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    bool ok = true;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t tx_bytes = static_cast<uint32_t>(Cfg::kABytes + BN * p.b_row_tx + 512 + Cfg::kSfbAtoms * 512);
    grid_dependency_wait();  // the quantised activations come from the kernel before this one
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int mt = tile % p.m_tiles;
      const int nt = tile / p.m_tiles;
      const int m0 = mt * kBM;
      const int n0 = nt * BN;
      const uint8_t* sfa_src = p.sfa + static_cast<int64_t>(mt) * p.katoms * 512;
      for (int kt = 0; kt < p.k_steps; ++kt) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, &abort_flag));
        if (!ok) break;
        const uint32_t st = smem_base + stage * Cfg::kStageBytes;
        const uint32_t bar = smem_u32(&full_bar[stage]);
        if (elect_one()) {
          mbar_arrive_expect_tx(bar, tx_bytes);
          tma_load_2d(st, &tmap_a, kt * 128, m0, bar);                               // bytes = E4M3 codes
          tma_load_2d(st + Cfg::kABytes, &tmap_b, kt * kW4A8KElems, n0, bar);        // x counts 4-bit elements
          bulk_g2s(st + Cfg::kABytes + Cfg::kBBytes, sfa_src + kt * 512, 512, bar);
#pragma unroll
          for (int rt = 0; rt < Cfg::kSfbAtoms; ++rt) {
            const int row_tile = min((n0 >> 7) + rt, p.sfb_row_tiles - 1);  // stay inside the buffer
            bulk_g2s(st + Cfg::kABytes + Cfg::kBBytes + 512 + rt * 512,
                     p.sfb + (static_cast<int64_t>(row_tile) * p.katoms + kt) * 512, 512, bar);
          }
        }
        ++issued;
        if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) {
      const int pending = min(issued, Cfg::kStages);
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = Cfg::kStages - 1; phase ^= 1u; }
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&full_bar[stage]), phase) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    constexpr uint32_t idesc0 = mxf8f6f4_idesc_e4m3_e2m1(kBM, BN);
    const uint32_t smem_base = smem_u32(smem);
    const uint64_t ab_desc0 = make_smem_desc(smem_base, 16, 1024, 2);
    const uint64_t sf_desc0 = make_smem_desc(smem_base + Cfg::kABytes + Cfg::kBBytes, 0, 128, 0);
    const uint32_t sf_tmem0 = tmem_base + Cfg::kAccCols;
    int stage = 0;
    uint32_t phase = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
      const int acc = it % Cfg::kAccStages;
      const uint32_t acc_phase = (it / Cfg::kAccStages) & 1u;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&acc_empty_bar[acc]), acc_phase ^ 1u, &abort_flag));
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + acc * BN;
      for (int kt = 0; kt < p.k_steps; ++kt) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&full_bar[stage]), phase, &abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t soff = static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
        const uint64_t adesc = ab_desc0 + soff;
        const uint64_t bdesc = adesc + (Cfg::kABytes >> 4);
        const uint64_t sfd = sf_desc0 + soff;
        const uint32_t sfa_col = sf_tmem0 + stage * Cfg::kSfColsPerStage;
        const uint32_t sfb_col = sfa_col + 4;
        if (elect_one()) {
          tc_cp_32x128b_warpx4(sfa_col, sfd);
#pragma unroll
          for (int rt = 0; rt < Cfg::kSfbAtoms; ++rt) tc_cp_32x128b_warpx4(sfb_col + 4 * rt, sfd + ((512 + rt * 512) >> 4));
#pragma unroll
          for (uint32_t kb = 0; kb < 4; ++kb)   // block kb of the K-step: byte kb of every scale column
            tc_mma_mxf8f6f4(d_tmem, adesc + 2 * kb, bdesc + 2 * kb, idesc0 | (kb << 29) | (kb << 4),
                            sfa_col | (kb << 30), sfb_col | (kb << 30), (kt | static_cast<int>(kb)) != 0 ? 1u : 0u);
          tc_commit(smem_u32(&empty_bar[stage]));
        }
        if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      if (elect_one()) tc_commit(smem_u32(&acc_full_bar[acc]));
    }
    if (lane == 0) {
      tc_commit(smem_u32(&drain_bar));
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(smem_u32(&drain_bar), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue warps
    const int quad = warp & 3;
    uint8_t* my_staging = staging + quad * (Cfg::kStagingBufs * 4096);
    constexpr int kChunkCols = OUT_BF16 ? 64 : 32;
    int buf = 0;
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
      const int row0 = mt * kBM + quad * 32;
      const uint32_t taddr = tmem_base + acc * BN + (static_cast<uint32_t>(quad * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += kChunkCols) {
        uint32_t w[32];
        if (OUT_BF16) {
          uint32_t r0[32], r1[32];
          tmem_ld_32x32b_x32(taddr + c0, r0);
          tmem_ld_32x32b_x32(taddr + c0 + 32, r1);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const __nv_bfloat162 a = __floats2bfloat162_rn(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
            const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
            w[i] = *reinterpret_cast<const uint32_t*>(&a);
            w[16 + i] = *reinterpret_cast<const uint32_t*>(&b);
          }
        } else {
          tmem_ld_32x32b_x32(taddr + c0, w);
          tmem_ld_wait();
        }
        const int col0 = nt * BN + c0;
        if (p.m16 < p.m && col0 < p.m && col0 + kChunkCols > p.m16 && row0 + lane < p.s) {
          if (OUT_BF16) {
            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<int64_t>(row0 + lane) * p.ldy + col0;
#pragma unroll
            for (int i = 0; i < kChunkCols; ++i)
              if (col0 + i >= p.m16 && col0 + i < p.m) {
                const uint32_t word = w[((i >> 5) << 4) + ((i & 31) >> 1)];
                const uint16_t hv = static_cast<uint16_t>((i & 1) ? (word >> 16) : (word & 0xFFFFu));
                yp[i] = *reinterpret_cast<const __nv_bfloat16*>(&hv);
              }
          } else {
            float* yp = reinterpret_cast<float*>(p.y) + static_cast<int64_t>(row0 + lane) * p.ldy + col0;
#pragma unroll
            for (int i = 0; i < kChunkCols; ++i)
              if (col0 + i >= p.m16 && col0 + i < p.m) yp[i] = __uint_as_float(w[i]);
          }
        }
        if (lane == 0) bulk_wait_group_read<Cfg::kStagingBufs - 1>();
        __syncwarp();
        uint8_t* sb = my_staging + buf * 4096 + lane * 128;
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<uint4*>(sb + ((q ^ (lane & 7)) << 4)) = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (row0 < p.s && col0 < p.m16) tma_store_2d(&tmap_y, col0, row0, smem_u32(my_staging + buf * 4096));
          bulk_commit_group();
        }
        buf = (buf + 1) % Cfg::kStagingBufs;
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty_bar[acc]));
    }
    if (lane == 0) bulk_wait_group<0>();
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

}  // namespace batq
