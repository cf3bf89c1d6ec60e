// MXFP4 x MXFP4 block-scaled GEMM on CTA pairs with output tiles up to 448 features wide (stage 3,
// prefill shapes with many columns of tiles).
//
//   Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} qx[s,j,i] * qw[m,j,i]
//
// the low-bit matrix multiplication Q(XP) Q(P^-1 W^T) of the paper's Sec. 3.
//
// Why a second pair kernel.  gemm_mxfp4_pair.cuh keeps two accumulators in tensor memory (256 and
// 192 columns) so that a tile's epilogue runs under the next tile's MMAs; its tiles are at most
// 256 features wide, and at that width the kernel is bound by the bytes every SM pulls from L2
// (36 KiB per K-step for 128 x 256 outputs per SM), not by the tensor cores.  Here ONE tile takes
// both accumulators: 256 tokens x up to 448 features, two MMAs per 64 elements of K (N = 256 and
// N = bn - 256) that share the activation tile.  Per K-step a CTA then loads 49 KiB for 128 x 448
// outputs, 0.78 of the bytes per flop, and the tensor cores become the limit.  The price: the
// MMAs of a tile cannot start before the accumulators of the one before it have been read out
// (its loads can), so eight warps drain them instead of four and hand the accumulator back as
// soon as their columns sit in registers; the stores follow under the next tile's MMAs.
//
//   leader (cluster rank 0): rows [m0, m0+128),      weight rows [n0, n0+a/2) and [n0+a, n0+a+b/2)
//   peer   (cluster rank 1): rows [m0+128, m0+256),  weight rows [n0+a/2, n0+a) and [n0+a+b/2, n0+bn)
//
// with a = min(bn, 256), b = bn - a.  Work distribution, tile numbering, segments of column widths
// and barriers are those of gemm_mxfp4_pair.cuh (PairParams, PairWalk), with widths up to 448.
// The scale factors of a K-step go through ONE 40-column slot of tensor memory behind the
// accumulators (8 for the activations, 2 x 16 for four 128-row atoms of weight scales):
// tcgen05.cp and tcgen05.mma of one thread execute in issue order, so the copy for step k+1 cannot
// overtake the MMAs of step k that still read the slot.  No load carries a multicast qualifier.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "gemm_mxfp4_pair.cuh"
#include "ptx.cuh"

namespace batq {

constexpr int kWideEpiWarps = 8;
constexpr int kWideThreads = (2 + kWideEpiWarps) * 32;
constexpr int kWideMaxBn = 448;

struct WideCfg {
  static constexpr int kABytes = kBM * kBKBytes;          // 16 KiB: this CTA's 128 token rows
  static constexpr int kBBytes = (kWideMaxBn / 2) * kBKBytes;  // 28 KiB: this CTA's half of both parts
  static constexpr int kSfaBytes = 1024;                  // 128 rows x 8 blocks
  static constexpr int kSfbAtoms = 4;                     // 448 weight rows from a multiple of 64 touch at most four
  static constexpr int kSfbBytes = kSfbAtoms * 1024;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;   // 49 KiB
  static constexpr int kStages = 4;
  static constexpr int kAccCols = 448;
  static constexpr int kSfCols = 8 + 2 * 4 * kSfbAtoms;   // 40
  static constexpr int kTmemCols = 512;
  static constexpr int kStagingBufBytes = 2048;             // 32 rows x 64 bytes, one per epilogue warp
  static constexpr int kStagingBytes = kWideEpiWarps * kStagingBufBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024;
  static_assert(kAccCols + kSfCols <= kTmemCols, "tensor memory budget");
  static_assert(kSmemBytes <= 232448, "shared memory budget");
  static_assert(kStageBytes % 1024 == 0, "stage alignment");
};

template <bool OUT_BF16>
__global__ void __launch_bounds__(kWideThreads, 1)
gemm_mxfp4_wide_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b32,
                       const __grid_constant__ CUtensorMap tmap_sfa, const __grid_constant__ CUtensorMap tmap_sfb,
                       const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ PairParams p) {
  using Cfg = WideCfg;
  extern __shared__ uint8_t wide_smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];   // used in the leader only
  __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];  // one set per CTA
  __shared__ __align__(8) uint64_t acc_full_bar;             // one per CTA
  __shared__ __align__(8) uint64_t acc_empty_bar[2];         // used in the leader only: columns [0, 256) and [256, 448)
  __shared__ __align__(8) uint64_t drain_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  // A kernel launched as a programmatic dependent of this one may be scheduled on every SM this
  // grid has left; it must still wait for this grid before it touches memory.
  grid_launch_dependents();
  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const int lane = tid & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(wide_smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + Cfg::kStages * Cfg::kStageBytes;

  if (tid == 0) {
    for (int i = 0; i < Cfg::kStages; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), 1);
    }
    mbar_init(smem_u32(&acc_full_bar), 1);
    for (int i = 0; i < 2; ++i) mbar_init(smem_u32(&acc_empty_bar[i]), 2 * kWideEpiWarps);  // the epilogue warps of both CTAs
    mbar_init(smem_u32(&drain_bar), 1);
    abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_b32);
    tma_prefetch_desc(&tmap_sfa);
    tma_prefetch_desc(&tmap_sfb);
    tma_prefetch_desc(&tmap_y);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the other CTA's barriers are initialised before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  const PairWalk walk0(p, pair, n_pairs);

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (both CTAs)
    bool ok = true;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0_leader = map_to_cta(smem_u32(&full_bar[0]), 0);
    int my_steps = 0;
    {
      PairWalk w = walk0;
      PairTile t;
      while (w.next(t)) my_steps += p.k_steps;
    }
    // K-step kt of tile t into ring stage `stage`.  `what`: 1 = the weight side (this CTA's half of
    // the B tile in boxes of 32 rows, weight scales; the leader also arms the barrier with the
    // bytes of both CTAs), 2 = the activation side (A tile, activation scales), 3 = both.
    auto issue = [&](const PairTile& t, int kt, int stage, int what) {
      const int m0 = t.mp * 256 + static_cast<int>(rank) * kBM;
      const int bna = min(t.bn, 256), bnb = t.bn - bna;
      const int ha = bna >> 1, hb = bnb >> 1;
      const uint32_t st = smem_base + stage * Cfg::kStageBytes;
      const uint32_t bar = full0_leader + 8u * stage;
      if (what & 1) {
        if (rank == 0)
          mbar_arrive_expect_tx(smem_u32(&full_bar[stage]),
                                2u * static_cast<uint32_t>(Cfg::kABytes + (ha + hb) * kBKBytes + Cfg::kSfaBytes + Cfg::kSfbBytes));
        const int a0 = t.n0 + static_cast<int>(rank) * ha;
        for (int r = 0; r < ha; r += 32)
          tma_load_2d_pair(st + Cfg::kABytes + r * kBKBytes, &tmap_b32, kt * kBKBytes, a0 + r, bar);
        const int b0 = t.n0 + bna + static_cast<int>(rank) * hb;
        for (int r = 0; r < hb; r += 32)
          tma_load_2d_pair(st + Cfg::kABytes + (ha + r) * kBKBytes, &tmap_b32, kt * kBKBytes, b0 + r, bar);
#pragma unroll
        for (int rt = 0; rt < Cfg::kSfbAtoms; ++rt)
          tma_load_2d_pair(st + Cfg::kABytes + Cfg::kBBytes + Cfg::kSfaBytes + rt * 1024, &tmap_sfb, 0,
                           ((t.n0 >> 7) + rt) * p.katoms + 2 * kt, bar);
      }
      if (what & 2) {
        tma_load_2d_pair(st, &tmap_a, kt * kBKBytes, m0, bar);
        tma_load_2d_pair(st + Cfg::kABytes + Cfg::kBBytes, &tmap_sfa, 0, (m0 >> 7) * p.katoms + 2 * kt, bar);
      }
    };
    // The first `prefill` steps of the pair, side `what`, into stages 0, 1, ...
    const int prefill = min(my_steps, Cfg::kStages);
    auto issue_prefill = [&](int what) {
      PairWalk w = walk0;
      PairTile t;
      int g = 0;
      while (g < prefill && w.next(t))
        for (int kt = 0; kt < p.k_steps && g < prefill; ++kt, ++g) issue(t, kt, g, what);
    };
    // The weights do not depend on the kernel that quantises the activations: fill the ring's
    // weight side first, then wait for that kernel (programmatic dependent launch; an ordinary
    // launch does not wait here), then add the activation side.
    if (elect_one()) issue_prefill(1);
    __syncwarp();
    grid_dependency_wait();
    if (elect_one()) issue_prefill(2);
    __syncwarp();
    int stage = prefill % Cfg::kStages;
    uint32_t phase = (prefill == Cfg::kStages) ? 1u : 0u;
    {
      PairWalk w = walk0;
      PairTile t;
      int g = 0;
      while (ok && w.next(t)) {
        for (int kt = 0; kt < p.k_steps; ++kt, ++g) {
          if (g < prefill) continue;
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, &abort_flag));
          if (!ok) break;
          if (elect_one()) issue(t, kt, stage, 3);
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
    if (!ok && lane == 0) {
      // Given up: the loads of both CTAs are counted on the leader's barriers, so neither CTA can
      // wait for its own; give the copies already in flight ample time to land instead.
      const uint64_t t0 = global_timer_ns();
      while (global_timer_ns() - t0 < 1000000ull) {}
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    if (rank == 0) {
      const uint32_t smem_base = smem_u32(smem);
      const uint64_t ab_desc0 = make_smem_desc(smem_base, 16, 1024, 2);
      const uint64_t sf_desc0 = make_smem_desc(smem_base + Cfg::kABytes + Cfg::kBBytes, 0, 128, 0);
      const uint32_t sf_tmem0 = tmem_base + Cfg::kAccCols;
      const uint32_t full0 = smem_u32(&full_bar[0]);
      const uint32_t empty0 = smem_u32(&empty_bar[0]);

      int stage = 0;
      uint32_t phase = 0;
      uint32_t n_tile = 0;
      bool ok = true;
      PairWalk w = walk0;
      PairTile t;
      while (ok && w.next(t)) {
        const int bna = min(t.bn, 256), bnb = t.bn - bna;
        const uint32_t ia0 = mxf4_idesc(256, bna);
        const uint32_t ia1 = ia0 | (2u << 29) | (2u << 4);
        const uint32_t ib0 = mxf4_idesc(256, bnb > 0 ? bnb : 64);
        const uint32_t ib1 = ib0 | (2u << 29) | (2u << 4);
        const uint32_t sfb_sub = static_cast<uint32_t>(t.n0 & 127) >> 5;
        const uint32_t b_part_b = static_cast<uint32_t>(((bna >> 1) * kBKBytes) >> 4);  // part b's rows in the B tile
        // One accumulator in two parts, handed back separately by the epilogue of the tile before
        // this one: columns [0, 256) first.  The first K-step issues its four MMAs on part a, then
        // waits for part b.
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&acc_empty_bar[0]), (n_tile & 1u) ^ 1u, &abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        // One K-step.  FIRST (the tile's first: the accumulators start from zero, and part b's MMAs
        // wait for part b of the accumulator) and TWO (the tile has a part b) are compile-time: the
        // elected lane's instruction stream between two MMAs holds no run-time branch.
        auto k_step = [&](auto first_c, auto two_c) {
          constexpr bool FIRST = decltype(first_c)::value;
          constexpr bool TWO = decltype(two_c)::value;
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(full0 + 8u * stage, phase, &abort_flag));
          if (!ok) return;
          tc_fence_after_sync();
          const uint32_t soff = static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
          const uint64_t adesc = ab_desc0 + soff;
          const uint64_t bdesc = adesc + (Cfg::kABytes >> 4);
          const uint64_t sfd = sf_desc0 + soff;
          const uint32_t sfa_col = sf_tmem0;
          const uint32_t sfb_col = sfa_col + 8 + sfb_sub;
          if (elect_one()) {
            tc_cp_32x128b_warpx4_pair(sfa_col, sfd);
            tc_cp_32x128b_warpx4_pair(sfa_col + 4, sfd + 32);
#pragma unroll
            for (int rt = 0; rt < Cfg::kSfbAtoms; ++rt)
#pragma unroll
              for (int c = 0; c < 2; ++c)
                tc_cp_32x128b_warpx4_pair(sfa_col + 8 + c * 4 * Cfg::kSfbAtoms + 4 * rt,
                                          sfd + ((Cfg::kSfaBytes + rt * 1024 + c * 512) >> 4));
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
              const uint32_t c = kb >> 1;
              const uint32_t sfid = (kb & 1) * 2;
              const uint32_t sa = (sfa_col + 4 * c) | (sfid << 30);
              const uint32_t sb = (sfb_col + c * 4 * Cfg::kSfbAtoms) | (sfid << 30);
              tc_mma_mxf4_pair(tmem_base, adesc + 2 * kb, bdesc + 2 * kb, (kb & 1) ? ia1 : ia0, sa, sb,
                               (FIRST && kb == 0) ? 0u : 1u);
              if (TWO && !FIRST)   // weight rows 256.. of the tile: eight scale columns (256 rows) further on
                tc_mma_mxf4_pair(tmem_base + 256, adesc + 2 * kb, bdesc + b_part_b + 2 * kb, (kb & 1) ? ib1 : ib0, sa,
                                 sb + 8, 1u);
            }
          }
          if (TWO && FIRST) {   // part a's MMAs are under way, now part b
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&acc_empty_bar[1]), (n_tile & 1u) ^ 1u, &abort_flag));
            if (!ok) return;
            tc_fence_after_sync();
            if (elect_one()) {
#pragma unroll
              for (int kb = 0; kb < 4; ++kb) {
                const uint32_t c = kb >> 1;
                const uint32_t sfid = (kb & 1) * 2;
                tc_mma_mxf4_pair(tmem_base + 256, adesc + 2 * kb, bdesc + b_part_b + 2 * kb, (kb & 1) ? ib1 : ib0,
                                 (sfa_col + 4 * c) | (sfid << 30), (sfb_col + 8 + c * 4 * Cfg::kSfbAtoms) | (sfid << 30),
                                 kb != 0 ? 1u : 0u);
              }
            }
          }
          if (elect_one()) tc_commit_pair(empty0 + 8u * stage, 3);  // frees the stage in both CTAs
          __syncwarp();
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        };
        using yes = std::integral_constant<bool, true>;
        using no = std::integral_constant<bool, false>;
        if (bnb > 0) {
          k_step(yes{}, yes{});
          for (int kt = 1; kt < p.k_steps && ok; ++kt) k_step(no{}, yes{});
        } else {
          k_step(yes{}, no{});
          for (int kt = 1; kt < p.k_steps && ok; ++kt) k_step(no{}, no{});
        }
        if (!ok) break;
        if (bnb == 0) {   // part b unused by this tile: take its barrier's phase along
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&acc_empty_bar[1]), (n_tile & 1u) ^ 1u, &abort_flag));
          if (!ok) break;
        }
        if (!ok) break;
        if (elect_one()) tc_commit_pair(smem_u32(&acc_full_bar), 3);
        ++n_tile;
      }
      if (lane == 0) {
        tc_commit_pair_local(smem_u32(&drain_bar));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&drain_bar), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
      __syncwarp();
    }
  } else {
    // ---------------------------------------------------------------- epilogue warps (both CTAs)
    // Two warps per lane quadrant of tensor memory; they take alternate chunks of 32 columns.  With
    // bf16 output a warp first moves ALL its columns of the tile into registers (rounded and
    // packed: 16 words per chunk, at most seven chunks), hands the accumulator back, and only then
    // writes them out through its staging buffer (32 rows x 64 bytes) and TMA stores -- under the
    // next tile's MMAs.  With fp32 output the columns do not fit the register file: the warp works
    // chunk by chunk.  The accumulator goes back in two parts, columns [0, 256) first: the next tile's
    // first MMAs only write those.
    const int quad = warp & 3;
    const int part = (warp - 2) >> 2;
    uint8_t* my_staging = staging + (warp - 2) * Cfg::kStagingBufBytes;
    constexpr int kBoxCols = OUT_BF16 ? 32 : 16;   // columns of a 64-byte row
    constexpr int kMaxChunks = 7;                  // 2 x 7 x 32 = 448 columns
    const uint32_t acc_empty_leader = map_to_cta(smem_u32(&acc_empty_bar[0]), 0);
    auto release = [&](int which) {   // this warp has read its columns of part `which`
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * which);
    };
    uint32_t n_tile = 0;
    PairWalk wk = walk0;
    PairTile t;
    // Rows [row0, row0 + 32) x columns [col0, col0 + kBoxCols) of y from 16 words per lane (one row
    // per lane).
    auto write_box = [&](const uint32_t* w, int row0, int col0) {
      if (p.m16 < p.m && col0 < p.m && col0 + kBoxCols > p.m16 && row0 + lane < p.s) {
        if (OUT_BF16) {
          __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(p.y) + static_cast<int64_t>(row0 + lane) * p.ldy + col0;
#pragma unroll
          for (int i = 0; i < kBoxCols; ++i)
            if (col0 + i >= p.m16 && col0 + i < p.m) {
              const uint32_t word = w[i >> 1];
              const uint16_t hv = static_cast<uint16_t>((i & 1) ? (word >> 16) : (word & 0xFFFFu));
              yp[i] = *reinterpret_cast<const __nv_bfloat16*>(&hv);
            }
        } else {
          float* yp = reinterpret_cast<float*>(p.y) + static_cast<int64_t>(row0 + lane) * p.ldy + col0;
#pragma unroll
          for (int i = 0; i < kBoxCols; ++i)
            if (col0 + i >= p.m16 && col0 + i < p.m) yp[i] = __uint_as_float(w[i]);
        }
      }
      if (lane == 0) bulk_wait_group_read<0>();   // the store before this one has read the buffer
      __syncwarp();
      uint8_t* sb = my_staging + lane * 64;
#pragma unroll
      for (int q = 0; q < 4; ++q)   // 64-byte swizzle: 16-byte chunk index XOR ((row / 2) & 3)
        *reinterpret_cast<uint4*>(sb + ((q ^ ((lane >> 1) & 3)) << 4)) = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        if (row0 < p.s && col0 < p.m16) tma_store_2d(&tmap_y, col0, row0, smem_u32(my_staging));
        bulk_commit_group();
      }
    };
    while (wk.next(t)) {
      bool ok = mbar_wait(smem_u32(&acc_full_bar), n_tile & 1u, &abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const int row0 = t.mp * 256 + static_cast<int>(rank) * kBM + quad * 32;
      // part a sits in columns [0, 256), part b from column 256 on: tile column c0 = accumulator column c0
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
      if (OUT_BF16) {
        uint32_t w[kMaxChunks][16];
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
          const int c0 = (2 * i + part) * 32;
          if (i == 4) release(0);   // chunks 0..3 of a warp are the columns below 256
          if (c0 < t.bn) {
            uint32_t r[32];
            tmem_ld_32x32b_x32(taddr + c0, r);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const __nv_bfloat162 a = __floats2bfloat162_rn(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
              w[i][j] = *reinterpret_cast<const uint32_t*>(&a);
            }
          }
        }
        release(1);
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
          const int c0 = (2 * i + part) * 32;
          if (c0 < t.bn) write_box(w[i], row0, t.n0 + c0);
        }
      } else {
        bool released = false;
#pragma unroll 1
        for (int c0 = part * 32; c0 < t.bn; c0 += 64) {
          uint32_t w[32];
          if (c0 >= 256 && !released) { release(0); released = true; }
          tmem_ld_32x32b_x32(taddr + c0, w);
          tmem_ld_wait();
          write_box(w, row0, t.n0 + c0);
          write_box(w + 16, row0, t.n0 + c0 + 16);
        }
        if (!released) release(0);
        release(1);
      }
      ++n_tile;
    }
    if (lane == 0) bulk_wait_group<0>();
  }

  // Neither CTA may leave (or release tensor memory) while the other can still read its shared
  // memory or signal its barriers.
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, Cfg::kTmemCols);
  }
}

}  // namespace batq
