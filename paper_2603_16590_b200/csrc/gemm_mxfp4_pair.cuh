// MXFP4 x MXFP4 block-scaled GEMM on CTA pairs (stage 3, prefill shapes).
//
//   Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} qx[s,j,i] * qw[m,j,i]
//
// the low-bit matrix multiplication Q(XP) Q(P^-1 W^T) of the paper's Sec. 3.
//
// Same pipeline as gemm_mxfp4.cuh, but two CTAs on the two SMs of a pair (a cluster of 2) share
// one 256-token output tile: each CTA owns 128 token rows (its A tile, its accumulator rows in
// its own tensor memory) and stages only half of the tile's weight rows; one thread of the leader
// CTA issues tcgen05.mma.cta_group::2, which reads A and the two halves of B from both shared
// memories.
//
//   leader (cluster rank 0): rows [m0, m0+128),      weight rows [n0, n0+bn/2)
//   peer   (cluster rank 1): rows [m0+128, m0+256),  weight rows [n0+bn/2, n0+bn)
//
// Work distribution.  Tiles are numbered column of tiles after column (all 256-token row blocks
// of one range of output features are consecutive) and pair p of P takes tiles p, p + P, ...: at
// any time the pairs work on a few neighbouring columns and all row blocks, in step along K, so
// every weight tile is requested by many pairs at once and every activation tile by the others
// -- measured, that sharing in L2 is worth a quarter of the throughput against a distribution in
// which each pair walks its own stretch of a row.  Column widths come in up to kPairMaxSegs
// segments of consecutive columns; inside a segment the columns are all equally wide (64, 128,
// 192 or 256) or alternately wa and wb wide (256 and 192: 224 on average).  The host picks the
// segments by walking candidates through a cost model, so that the pairs' last tiles end together
// (e.g. 6144 features at 2048 tokens: nine columns of 256, twelve of 192, six of 256 give every
// pair at most three tiles and never two 256-wide ones in a row).  The last column is as narrow
// as the layer's edge allows.  Every column starts at a multiple of 64 features: the MMA takes
// the weight scales from an even column of tensor memory only (one column = 32 weight rows; an
// odd one raises a misaligned-address fault).
//
// Accumulators live in two slots of tensor memory, columns [0, 256) and [256, 448).  A tile wider
// than 192 needs slot 0; a narrower one takes the slot the tile before it did not use, so that
// its MMAs run under that tile's epilogue.  (Two 256-wide tiles in a row share slot 0: the second
// waits for the first one's epilogue.)
//
// The scale factors of a K-step go through two alternating 24-column slots of tensor memory
// behind the accumulators: tcgen05.cp and tcgen05.mma of one thread execute in issue order, so the
// copy for step k+2 cannot overtake the MMAs of step k that still read the slot.
//
// Barriers.  full[stage] lives in the leader and counts the bytes of both CTAs' loads (the
// peer's TMA loads name the leader's barrier); empty[stage] and acc_full[] exist in both CTAs
// and are signalled by the leader's tcgen05.commit with a CTA mask; acc_empty[] lives in the
// leader and collects the epilogue warps of both CTAs.  No load carries a multicast qualifier.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_mxfp4.cuh"
#include "ptx.cuh"

namespace batq {

constexpr int kPairThreads = 192;
constexpr int kPairUnitCols = 64;   // output features per scheduling unit
constexpr int kPairMaxSegs = 4;     // segments of columns with one width pattern each

struct PairCfg {
  static constexpr int kABytes = kBM * kBKBytes;          // 16 KiB: this CTA's 128 token rows
  static constexpr int kBBytes = 128 * kBKBytes;          // room for this CTA's half of the widest tile
  static constexpr int kSfaBytes = 1024;                  // 128 rows x 8 blocks
  static constexpr int kSfbAtoms = 3;                     // 128-row scale tiles a tile can touch (256 columns from row 64)
  static constexpr int kSfbBytes = kSfbAtoms * 1024;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
  static constexpr int kStages = 5;
  static constexpr int kSlot1Col = 256;                   // accumulator slot 0: [0, 256), slot 1: [256, 448)
  static constexpr int kSlot1Width = 192;
  static constexpr int kAccCols = 448;
  static constexpr int kSfCols = 8 + 2 * 4 * kSfbAtoms;   // scale columns of one K-step
  static constexpr int kSfSlots = 2;
  static constexpr int kTmemCols = 512;
  static constexpr int kStagingBufs = 2;
  static constexpr int kStagingBytes = 4 * kStagingBufs * 4096;
  static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024;
  static_assert(kAccCols + kSfSlots * kSfCols <= kTmemCols, "tensor memory budget");
  static_assert(kSmemBytes <= 232448, "shared memory budget");
  static_assert(kStageBytes % 1024 == 0, "stage alignment");
};

// Columns [col0, col0 + cols) of tiles: they start at feature n0 and are alternately wa and wb wide
// (wa == wb: all equally wide).
struct PairSeg {
  int32_t col0, cols, n0;
  int16_t wa, wb;
};
struct PairParams {
  int32_t s;              // rows of X (tokens)
  int32_t m;              // rows of W (output features)
  int32_t katoms;         // KA = 2*ceil(k/8): 512-byte scale atoms per 128-row tile
  int32_t k_steps;        // ceil(n / 256)
  int32_t m_pairs;        // ceil(s / 256)
  int32_t n_cols;         // columns of tiles
  int32_t n_segs;         // segments in use
  PairSeg seg[kPairMaxSegs];
  int32_t m16;            // as in GemmParams: columns covered by the TMA store
  void* y;
  int64_t ldy;
};

// The tiles of one pair, in order.  Every warp role walks the same sequence.
struct PairTile {
  int mp;    // 256-token row block
  int n0;    // first output feature (a multiple of 64)
  int bn;    // width: the column's, less (a multiple of 64) in the last column
};
struct PairWalk {
  const PairParams* p;
  int tile, total, step;
  __host__ __device__ __forceinline__ PairWalk(const PairParams& params, int pair, int n_pairs)
      : p(&params), tile(pair), total(params.m_pairs * params.n_cols), step(n_pairs) {}
  __host__ __device__ __forceinline__ bool next(PairTile& t) {
    if (tile >= total) return false;
    const int nt = tile / p->m_pairs;
    t.mp = tile - nt * p->m_pairs;
    int sg = 0;
    while (sg + 1 < p->n_segs && nt >= p->seg[sg + 1].col0) ++sg;
    const PairSeg& g = p->seg[sg];
    const int i = nt - g.col0;
    t.n0 = g.n0 + (i >> 1) * (g.wa + g.wb) + (i & 1) * g.wa;
    const int w = (i & 1) ? g.wb : g.wa;
    const int rem = p->m - t.n0;
    t.bn = rem >= w ? w : ((rem + 63) / 64) * 64;
    tile += step;
    return true;
  }
};
// Which accumulator slot a tile takes, and the parity of that slot's barriers for it.
struct PairSlots {
  int prev, use0, use1;
  __host__ __device__ __forceinline__ PairSlots() : prev(1), use0(0), use1(0) {}
  __host__ __device__ __forceinline__ void take(int bn, int& slot, uint32_t& phase) {
    slot = bn > PairCfg::kSlot1Width ? 0 : (prev == 0 ? 1 : 0);
    phase = static_cast<uint32_t>(slot == 0 ? use0++ : use1++) & 1u;
    prev = slot;
  }
};

template <bool OUT_BF16>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_mxfp4_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b32,
                       const __grid_constant__ CUtensorMap tmap_sfa, const __grid_constant__ CUtensorMap tmap_sfb,
                       const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ PairParams p) {
  using Cfg = PairCfg;
  extern __shared__ uint8_t pair_smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];   // used in the leader only
  __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];  // one set per CTA
  __shared__ __align__(8) uint64_t acc_full_bar[2];          // one set per CTA
  __shared__ __align__(8) uint64_t acc_empty_bar[2];         // used in the leader only
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
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(pair_smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + Cfg::kStages * Cfg::kStageBytes;

  if (tid == 0) {
    for (int i = 0; i < Cfg::kStages; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&acc_full_bar[i]), 1);
      mbar_init(smem_u32(&acc_empty_bar[i]), 8);  // 4 epilogue warps of each CTA
    }
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
      const int half = t.bn >> 1;
      const uint32_t st = smem_base + stage * Cfg::kStageBytes;
      const uint32_t bar = full0_leader + 8u * stage;
      if (what & 1) {
        if (rank == 0)
          mbar_arrive_expect_tx(smem_u32(&full_bar[stage]),
                                2u * static_cast<uint32_t>(Cfg::kABytes + half * kBKBytes + Cfg::kSfaBytes + Cfg::kSfbBytes));
        const int b0 = t.n0 + static_cast<int>(rank) * half;
        for (int r = 0; r < half; r += 32)
          tma_load_2d_pair(st + Cfg::kABytes + r * kBKBytes, &tmap_b32, kt * kBKBytes, b0 + r, bar);
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
      uint32_t g = 0;  // K-steps issued so far: the scale slot alternates with it
      bool ok = true;
      PairWalk w = walk0;
      PairTile t;
      PairSlots slots;
      while (ok && w.next(t)) {
        const uint32_t idesc0 = mxf4_idesc(256, t.bn);
        const uint32_t idesc1 = idesc0 | (2u << 29) | (2u << 4);
        const uint32_t sfb_sub = static_cast<uint32_t>(t.n0 & 127) >> 5;
        int acc;
        uint32_t acc_phase;
        slots.take(t.bn, acc, acc_phase);
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&acc_empty_bar[acc]), acc_phase ^ 1u, &abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * Cfg::kSlot1Col;
        for (int kt = 0; kt < p.k_steps; ++kt, ++g) {
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(full0 + 8u * stage, phase, &abort_flag));
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t soff = static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
          const uint64_t adesc = ab_desc0 + soff;
          const uint64_t bdesc = adesc + (Cfg::kABytes >> 4);
          const uint64_t sfd = sf_desc0 + soff;
          const uint32_t sfa_col = sf_tmem0 + (g & 1u) * Cfg::kSfCols;
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
              tc_mma_mxf4_pair(d_tmem, adesc + 2 * kb, bdesc + 2 * kb, (kb & 1) ? idesc1 : idesc0,
                               (sfa_col + 4 * c) | (sfid << 30), (sfb_col + c * 4 * Cfg::kSfbAtoms) | (sfid << 30),
                               (kt | kb) != 0 ? 1u : 0u);
            }
            tc_commit_pair(empty0 + 8u * stage, 3);  // frees the stage in both CTAs
          }
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (elect_one()) tc_commit_pair(smem_u32(&acc_full_bar[acc]), 3);
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
    const int quad = warp & 3;
    uint8_t* my_staging = staging + quad * (Cfg::kStagingBufs * 4096);
    constexpr int kChunkCols = OUT_BF16 ? 64 : 32;
    const uint32_t acc_empty0_leader = map_to_cta(smem_u32(&acc_empty_bar[0]), 0);
    int buf = 0;
    PairWalk wk = walk0;
    PairTile t;
    PairSlots slots;
    while (wk.next(t)) {
      int acc;
      uint32_t acc_phase;
      slots.take(t.bn, acc, acc_phase);
      bool ok = mbar_wait(smem_u32(&acc_full_bar[acc]), acc_phase, &abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const int row0 = t.mp * 256 + static_cast<int>(rank) * kBM + quad * 32;
      const uint32_t taddr = tmem_base + acc * Cfg::kSlot1Col + (static_cast<uint32_t>(quad * 32) << 16);
      // Rows [row0, row0 + 32) x columns [col0, col0 + kChunkCols) of y from w (one row per lane).
      auto write_chunk = [&](const uint32_t (&w)[32], int col0) {
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
      };
      if (OUT_BF16) {
        // All columns of the tile into registers first (rounded and packed: 32 words per 64 columns,
        // at most four such chunks), then the accumulator goes back -- a tile that needs the same
        // slot next waits for these loads only -- and the stores follow.
        uint32_t w[4][32];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (64 * i < t.bn) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              uint32_t r[32];
              tmem_ld_32x32b_x32(taddr + 64 * i + 32 * h, r);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const __nv_bfloat162 a = __floats2bfloat162_rn(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
                w[i][16 * h + j] = *reinterpret_cast<const uint32_t*>(&a);
              }
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty0_leader + 8u * acc);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (64 * i < t.bn) write_chunk(w[i], t.n0 + 64 * i);
      } else {
#pragma unroll 1
        for (int c0 = 0; c0 < t.bn; c0 += kChunkCols) {
          uint32_t w[32];
          tmem_ld_32x32b_x32(taddr + c0, w);
          tmem_ld_wait();
          if (c0 + kChunkCols >= t.bn) {   // the last columns sit in registers: hand the accumulator back
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty0_leader + 8u * acc);
          }
          write_chunk(w, t.n0 + c0);
        }
      }
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
