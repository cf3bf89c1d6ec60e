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
// tcgen05.cp and read by the MMA from there.  Accumulators are double
// buffered in tensor memory where the tile width allows (BN <= 192), so the
// epilogue of one tile overlaps the main loop of the next; the epilogue goes
// tensor memory -> registers -> swizzled shared staging -> TMA store, which
// also clips ragged tiles.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace batq {

constexpr int kGemmThreads = 192;
constexpr int kBM = 128;
constexpr int kBKBytes = 128;  // 256 four-bit elements

template <int BN>
struct GemmCfg {
  static constexpr int kABytes = kBM * kBKBytes;  // 16 KiB
  static constexpr int kBBytes = BN * kBKBytes;
  static constexpr int kSfaBytes = 1024;  // 128 rows x 8 blocks
  static constexpr int kSfbAtoms = (BN + 127) / 128;  // 128-row scale atoms a tile can touch
  static constexpr int kSfbBytes = kSfbAtoms * 1024;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
  static constexpr int kStages = (BN == 128) ? 5 : 4;
  static constexpr int kAccStages = (BN == 256) ? 1 : 2;
  static constexpr int kAccCols = BN * kAccStages;
  static constexpr int kSfColsPerStage = 8 + 2 * 4 * kSfbAtoms;  // A: 2 chunks x 4, B: 2 chunks x 4 per atom
  static constexpr int kTmemCols = 512;
  static constexpr int kStagingBufs = (BN == 256) ? 1 : 2;  // per epilogue warp, 4 KiB each
  static constexpr int kStagingBytes = 4 * kStagingBufs * 4096;
  static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024;  // + alignment slack
  static constexpr uint32_t kTxBytes = kStageBytes;
  static_assert(kAccCols + kStages * kSfColsPerStage <= kTmemCols, "tensor memory budget");
  static_assert(kSmemBytes <= 232448, "shared memory budget");
  static_assert(BN % 64 == 0 && BN <= 256, "tile width");
};

struct GemmParams {
  const uint8_t* sfa;  // activation scales, BATQ_SF_MMA layout
  const uint8_t* sfb;  // weight scales, BATQ_SF_MMA layout
  int32_t s;           // rows of X (tokens)
  int32_t m;           // rows of W (output features)
  int32_t katoms;      // KA = 2*ceil(k/8)
  int32_t k_steps;     // ceil(n / 256)
  int32_t m_tiles;     // ceil(s / 128)
  int32_t n_tiles;     // ceil(m / BN)
  int32_t sfb_row_tiles;  // ceil(m / 128)
  // The TMA store covers columns [0, m16), m16 = m rounded down to a multiple of 16 bytes
  // (its clipping is 16-byte granular); the epilogue writes the < 16-byte tail of each row directly.
  int32_t m16;
  void* y;
  int64_t ldy;
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
                  const __grid_constant__ CUtensorMap tmap_y, const GemmParams p) {
  using Cfg = GemmCfg<BN>;
  extern __shared__ uint8_t gemm_smem_raw[];
  __shared__ __align__(8) uint64_t pipe_bar[2 * Cfg::kStages];  // [0, kStages) full, [kStages, 2 kStages) empty
  uint64_t* const full_bar = pipe_bar;
  uint64_t* const empty_bar = pipe_bar + Cfg::kStages;
  __shared__ __align__(8) uint64_t acc_full_bar[2];
  __shared__ __align__(8) uint64_t acc_empty_bar[2];
  __shared__ __align__(8) uint64_t drain_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  // A kernel launched as a programmatic dependent of this one may be scheduled on every SM this
  // grid has left; it must still wait for this grid before it touches memory.
  grid_launch_dependents();
  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);  // warp-uniform for the compiler
  const int lane = tid & 31;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(gemm_smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + Cfg::kStages * Cfg::kStageBytes;  // 1024-aligned: kStageBytes % 1024 == 0

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

  // The producer and MMA warps run their loops with all 32 lanes (warp-uniform control flow and
  // operands, so descriptors and addresses live in uniform registers); one elected lane issues.
  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    bool ok = true;
    const uint32_t smem_base = smem_u32(smem);
    grid_dependency_wait();  // the quantised activations come from the kernel before this one
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int mt = tile % p.m_tiles;
      const int nt = tile / p.m_tiles;
      const int m0 = mt * kBM;
      const int n0 = nt * BN;
      const int sfb_tile0 = n0 >> 7;
      const uint8_t* sfa_src = p.sfa + static_cast<int64_t>(mt) * p.katoms * 512;
      for (int kt = 0; kt < p.k_steps; ++kt) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&full_bar[0]) + 8u * (Cfg::kStages + stage), phase ^ 1u, &abort_flag));
        if (!ok) break;
        const uint32_t st = smem_base + stage * Cfg::kStageBytes;
        const uint32_t bar = smem_u32(&full_bar[0]) + 8u * stage;
        if (elect_one()) {
          mbar_arrive_expect_tx(bar, Cfg::kTxBytes);
          tma_load_2d(st, &tmap_a, kt * kBKBytes, m0, bar);
          tma_load_2d(st + Cfg::kABytes, &tmap_b, kt * kBKBytes, n0, bar);
          bulk_g2s(st + Cfg::kABytes + Cfg::kBBytes, sfa_src + kt * 1024, 1024, bar);
#pragma unroll
          for (int rt = 0; rt < Cfg::kSfbAtoms; ++rt) {
            const int row_tile = min(sfb_tile0 + rt, p.sfb_row_tiles - 1);  // stay inside the buffer
            bulk_g2s(st + Cfg::kABytes + Cfg::kBBytes + Cfg::kSfaBytes + rt * 1024,
                     p.sfb + (static_cast<int64_t>(row_tile) * p.katoms + 2 * kt) * 512, 1024, bar);
          }
        }
        ++issued;
        if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) {
      // Given up: let the copies already in flight land before the CTA exits.
      const int pending = min(issued, Cfg::kStages);
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = Cfg::kStages - 1; phase ^= 1u; }
        const uint32_t bar = smem_u32(&full_bar[stage]);
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(bar, phase) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    constexpr uint32_t idesc0 = mxf4_idesc(kBM, BN);
    constexpr uint32_t idesc1 = idesc0 | (2u << 29) | (2u << 4);  // scale byte pair 2 instead of 0
    // Loop-invariant descriptor bases; a stage adds (stage * kStageBytes) >> 4 to the address field.
    const uint32_t smem_base = smem_u32(smem);
    const uint64_t ab_desc0 = make_smem_desc(smem_base, 16, 1024, 2);
    const uint64_t sf_desc0 = make_smem_desc(smem_base + Cfg::kABytes + Cfg::kBBytes, 0, 128, 0);
    const uint32_t sf_tmem0 = tmem_base + Cfg::kAccCols;
    const uint32_t full0 = smem_u32(&full_bar[0]);
    const uint32_t empty0 = smem_u32(&empty_bar[0]);

    // Scale factors of one stage: shared memory -> tensor memory (512-byte atoms).
    auto copy_scales = [&](int stage) {
      const uint64_t sfd = sf_desc0 + static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
      const uint32_t col = sf_tmem0 + stage * Cfg::kSfColsPerStage;
      if (elect_one()) {
        tc_cp_32x128b_warpx4(col, sfd);
        tc_cp_32x128b_warpx4(col + 4, sfd + 32);
#pragma unroll
        for (int rt = 0; rt < Cfg::kSfbAtoms; ++rt)
#pragma unroll
          for (int c = 0; c < 2; ++c)
            tc_cp_32x128b_warpx4(col + 8 + c * 4 * Cfg::kSfbAtoms + 4 * rt,
                                 sfd + ((Cfg::kSfaBytes + rt * 1024 + c * 512) >> 4));
      }
    };

    int stage = 0;
    uint32_t phase = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
      const int nt = tile / p.m_tiles;
      const uint32_t sfb_sub = static_cast<uint32_t>((nt * BN) & 127) >> 5;  // tile starts mid-atom (BN = 192)
      const int acc = it % Cfg::kAccStages;
      const uint32_t acc_phase = (it / Cfg::kAccStages) & 1u;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&acc_empty_bar[acc]), acc_phase ^ 1u, &abort_flag));
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + acc * BN;
      for (int kt = 0; kt < p.k_steps; ++kt) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(full0 + 8u * stage, phase, &abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        copy_scales(stage);
        const uint32_t soff = static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
        const uint64_t adesc = ab_desc0 + soff;
        const uint64_t bdesc = adesc + (Cfg::kABytes >> 4);
        const uint32_t sfa_col = sf_tmem0 + stage * Cfg::kSfColsPerStage;
        const uint32_t sfb_col = sfa_col + 8 + sfb_sub;
        if (elect_one()) {
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint32_t c = kb >> 1;
            const uint32_t sfid = (kb & 1) * 2;  // byte pair inside the 32-bit scale column
            tc_mma_mxf4(d_tmem, adesc + 2 * kb, bdesc + 2 * kb, (kb & 1) ? idesc1 : idesc0,
                        (sfa_col + 4 * c) | (sfid << 30), (sfb_col + c * 4 * Cfg::kSfbAtoms) | (sfid << 30),
                        (kt | kb) != 0 ? 1u : 0u);
          }
          tc_commit(empty0 + 8u * stage);  // frees the stage once these MMAs have read it
        }
        if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      if (elect_one()) tc_commit(smem_u32(&acc_full_bar[acc]));
    }
    // All tensor-core work of this CTA done (or abandoned) before the memory is released.
    if (lane == 0) {
      tc_commit(smem_u32(&drain_bar));
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(smem_u32(&drain_bar), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue warps
    const int quad = warp & 3;  // tensor-memory lanes [32*quad, 32*quad + 32) belong to this warp
    uint8_t* my_staging = staging + quad * (Cfg::kStagingBufs * 4096);
    constexpr int kChunkCols = OUT_BF16 ? 64 : 32;  // 128 bytes of output per row
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
        uint32_t w[32];  // one 128-byte output row segment
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
          // ragged row tail (< 16 bytes) that the TMA store does not cover
          if (OUT_BF16) {
            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<int64_t>(row0 + lane) * p.ldy + col0;
#pragma unroll
            for (int i = 0; i < kChunkCols; ++i)
              if (col0 + i >= p.m16 && col0 + i < p.m) {
                const uint32_t word = w[((i >> 5) << 4) + ((i & 31) >> 1)];
                const uint16_t h = static_cast<uint16_t>((i & 1) ? (word >> 16) : (word & 0xFFFFu));
                yp[i] = *reinterpret_cast<const __nv_bfloat16*>(&h);
              }
          } else {
            float* yp = reinterpret_cast<float*>(p.y) + static_cast<int64_t>(row0 + lane) * p.ldy + col0;
#pragma unroll
            for (int i = 0; i < kChunkCols; ++i)
              if (col0 + i >= p.m16 && col0 + i < p.m) yp[i] = __uint_as_float(w[i]);
          }
        }
        // the staging buffer about to be overwritten must have been read by its TMA store
        if (lane == 0) bulk_wait_group_read<Cfg::kStagingBufs - 1>();
        __syncwarp();
        uint8_t* sb = my_staging + buf * 4096 + lane * 128;
#pragma unroll
        for (int q = 0; q < 8; ++q)  // 128-byte swizzle: 16-byte chunk index XOR (row & 7)
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
    if (lane == 0) bulk_wait_group<0>();  // all stores complete before the CTA exits
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

}  // namespace batq
