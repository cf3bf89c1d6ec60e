// MXFP4 x MXFP4 GEMM for a handful of tokens (decode: s <= 128), stage 3 of the path
// where it is bound by streaming the weights from HBM once (0.53 bytes per weight).
//
//   Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} qx[s,j,i] * qw[m,j,i]
//
// the low-bit matrix multiplication Q(XP) Q(P^-1 W^T) of the paper's Sec. 3, with the
// operands swapped for the tensor cores: a CTA owns 128 weight rows (the 128-row MMA
// operand) and a slice of K; the tokens are the narrow MMA dimension (16, 32, 64 or 128
// columns), so no tensor-core row is spent on padding tokens.  The grid is
// (row tiles) x (K splits): enough CTAs, two per SM, to keep the whole memory system
// busy however few output features the layer has.  With more than one split every CTA
// keeps its partial tile for a reduction in split order (deterministic): up to 8 splits can form a
// thread-block cluster that reduce-scatters the tiles through distributed shared memory (CTA q
// adds and writes tokens q, q + splits, ...); otherwise the tiles go to scratch and the CTA that
// draws the last ticket of a row tile adds them.  Up to 16 tokens the cluster's CTAs PUSH: each
// stores the partial sums of token t straight into a receive buffer of CTA t mod splits (remote
// stores are posted, nothing waits for them), one cluster barrier, and every CTA adds what it
// received from local shared memory -- one barrier and no remote load instead of two barriers
// around a round of remote loads.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and tensor-memory owner,
// warps 2..5 = epilogue.  The weight stream does not depend on the activation
// quantiser, so the producer starts it before waiting for the preceding kernel
// (programmatic dependent launch); only the loads of the quantised activations wait.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_mxfp4.cuh"
#include "ptx.cuh"

namespace batq {

constexpr int kSmallThreads = 192;

template <int NTOK>
struct SmallCfg {
  static constexpr int kWBytes = 128 * kBKBytes;     // 16 KiB of weight codes per K-step
  static constexpr int kXBytes = NTOK * kBKBytes;    // activation codes
  static constexpr int kSfBytes = 1024;              // two 512-byte scale atoms (8 blocks), per operand
  static constexpr int kStageBytes = kWBytes + kXBytes + 2 * kSfBytes;
  static constexpr int kStages = (NTOK == 128) ? 3 : (NTOK == 64) ? 4 : 5;
  static constexpr int kSfColsPerStage = 16;         // W: 2 atoms x 4 columns, X: 2 atoms x 4 columns
  static constexpr int kTmemCols = (NTOK == 128) ? 256 : 128;
  // Receive buffer of the push reduction (16-token tile only): [source split][ceil(s / splits)][128] fp32,
  // at most (16 + 7 - 1) / 7 * 7 = 21 token slots of 512 bytes.  It is apart from the ring: a faster
  // CTA of the cluster writes into it while this CTA's MMAs may still read the ring.
  static constexpr int kRecvBytes = (NTOK == 16) ? 21 * 512 : 0;
  static constexpr int kSmemBytes = kStages * kStageBytes + kRecvBytes + 1024;
  static_assert(NTOK == 16 || NTOK == 32 || NTOK == 64 || NTOK == 128, "token tile");
  static_assert(kStages * kStageBytes >= NTOK * 128 * 4, "the partial tile of the cluster reduction fits the ring");
  static_assert(NTOK + kStages * kSfColsPerStage <= kTmemCols, "tensor memory budget");
  static_assert(2 * (kSmemBytes + 2048) <= 232448, "two CTAs per SM");
  static_assert(kStageBytes % 1024 == 0, "stage alignment");
};

struct SmallParams {
  const uint8_t* sfx;    // activation scales, BATQ_SF_MMA layout (one 128-row tile)
  const uint8_t* sfw;    // weight scales, BATQ_SF_MMA layout
  int32_t s;             // tokens (<= NTOK)
  int32_t m;             // weight rows = output features
  int32_t katoms;        // 2*ceil(k/8)
  int32_t k_steps;       // ceil(n / 256)
  int32_t splits;        // gridDim.y
  void* y;               // [s x m] fp32 or bf16, row stride ldy
  int64_t ldy;
  float* partial;        // [row tile][split][NTOK][128] fp32 (splits > 1, ticket mode)
  uint32_t* tickets;     // [row tiles], zero on entry, zero again on exit (splits > 1, ticket mode)
  int32_t cluster_reduce;  // 1: the splits of a row tile are one thread-block cluster (grid.y == cluster.y <= 8)
                           // and add their partial tiles through distributed shared memory instead
};

// 32 lanes x 16 consecutive 32-bit columns -> 16 registers per thread.
__device__ __forceinline__ void tmem_ld_32x32b_x16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int NTOK, bool OUT_BF16>
__global__ void __launch_bounds__(kSmallThreads, 2)
gemm_small_s_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                    const SmallParams p) {
  using Cfg = SmallCfg<NTOK>;
  extern __shared__ uint8_t small_smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t acc_full_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ uint32_t ticket_slot;
  __shared__ int abort_flag;

  // The next grid on the stream (the quantiser of the next layer) may be scheduled at once; it
  // writes nothing before its own grid_dependency_wait().
  grid_launch_dependents();
  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const int lane = tid & 31;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(small_smem_raw) + 1023) & ~uintptr_t(1023));

  if (tid == 0) {
    for (int i = 0; i < Cfg::kStages; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), 1);
    }
    mbar_init(smem_u32(&acc_full_bar), 1);
    abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_w);
    tma_prefetch_desc(&tmap_x);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  const int rt = blockIdx.x;                      // 128-row tile of W
  const int sp = blockIdx.y;                      // K split
  const int kt0 = static_cast<int>(static_cast<int64_t>(p.k_steps) * sp / p.splits);
  const int kt1 = static_cast<int>(static_cast<int64_t>(p.k_steps) * (sp + 1) / p.splits);
  const int n_steps = kt1 - kt0;                  // >= 1: the host keeps splits <= k_steps
  const bool by_cluster = p.cluster_reduce != 0 && p.splits > 1;
  bool epi_ok = false;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    const uint32_t smem_base = smem_u32(smem);
    const uint8_t* sfw_src = p.sfw + static_cast<int64_t>(rt) * p.katoms * 512;
    auto load_w = [&](int stage, int kt) {
      const uint32_t st = smem_base + stage * Cfg::kStageBytes;
      const uint32_t bar = smem_u32(&full_bar[stage]);
      mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
      tma_load_2d(st, &tmap_w, kt * kBKBytes, rt * 128, bar);
      bulk_g2s(st + Cfg::kWBytes + Cfg::kXBytes, sfw_src + static_cast<int64_t>(kt) * 1024, 1024, bar);
    };
    auto load_x = [&](int stage, int kt) {
      const uint32_t st = smem_base + stage * Cfg::kStageBytes;
      const uint32_t bar = smem_u32(&full_bar[stage]);
      tma_load_2d(st + Cfg::kWBytes, &tmap_x, kt * kBKBytes, 0, bar);
      bulk_g2s(st + Cfg::kWBytes + Cfg::kXBytes + Cfg::kSfBytes, p.sfx + static_cast<int64_t>(kt) * 1024, 1024, bar);
    };
    // Weights first: they do not depend on the kernel that quantises the activations.
    const int prefill = min(n_steps, Cfg::kStages);
    if (elect_one())
      for (int i = 0; i < prefill; ++i) load_w(i, kt0 + i);
    __syncwarp();
    grid_dependency_wait();
    if (elect_one())
      for (int i = 0; i < prefill; ++i) load_x(i, kt0 + i);
    __syncwarp();
    int stage = prefill % Cfg::kStages;
    uint32_t phase = (prefill == Cfg::kStages) ? 1u : 0u;
    bool ok = true;
    int issued = prefill;
    for (int i = prefill; i < n_steps; ++i) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, &abort_flag));
      if (!ok) break;
      if (elect_one()) {
        load_w(stage, kt0 + i);
        load_x(stage, kt0 + i);
      }
      ++issued;
      if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
    }
    if (!ok && lane == 0) {
      // Given up: let the copies already in flight land before the CTA exits.
      const int pending = min(issued, Cfg::kStages);
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = Cfg::kStages - 1; phase ^= 1u; }
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&full_bar[stage]), phase) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    constexpr uint32_t idesc0 = mxf4_idesc(128, NTOK);
    constexpr uint32_t idesc1 = idesc0 | (2u << 29) | (2u << 4);  // scale byte pair 2 instead of 0
    const uint32_t smem_base = smem_u32(smem);
    const uint64_t w_desc0 = make_smem_desc(smem_base, 16, 1024, 2);
    const uint64_t sf_desc0 = make_smem_desc(smem_base + Cfg::kWBytes + Cfg::kXBytes, 0, 128, 0);
    const uint32_t sf_tmem0 = tmem_base + NTOK;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int i = 0; i < n_steps; ++i) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&full_bar[stage]), phase, &abort_flag));
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t soff = static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
      const uint64_t wdesc = w_desc0 + soff;
      const uint64_t xdesc = wdesc + (Cfg::kWBytes >> 4);
      const uint64_t sfd = sf_desc0 + soff;
      const uint32_t sfw_col = sf_tmem0 + stage * Cfg::kSfColsPerStage;
      const uint32_t sfx_col = sfw_col + 8;
      if (elect_one()) {
        tc_cp_32x128b_warpx4(sfw_col, sfd);
        tc_cp_32x128b_warpx4(sfw_col + 4, sfd + 32);
        tc_cp_32x128b_warpx4(sfx_col, sfd + 64);
        tc_cp_32x128b_warpx4(sfx_col + 4, sfd + 96);
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
          const uint32_t c = kb >> 1;
          const uint32_t sfid = (kb & 1) * 2;
          tc_mma_mxf4(tmem_base, wdesc + 2 * kb, xdesc + 2 * kb, (kb & 1) ? idesc1 : idesc0,
                      (sfw_col + 4 * c) | (sfid << 30), (sfx_col + 4 * c) | (sfid << 30), (i | kb) != 0 ? 1u : 0u);
        }
        tc_commit(smem_u32(&empty_bar[stage]));
      }
      if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
    }
    if (lane == 0) {
      // Arrives when every MMA issued above is done -- also on the give-up path, so that the
      // tensor memory is idle before it is released.
      tc_commit(smem_u32(&acc_full_bar));
      if (!ok) {
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&acc_full_bar), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue warps
    // The accumulator row of a thread (NTOK values) is handled 16 tokens at a time, so that the
    // widest token tile needs no more registers than the narrowest.
    const int quad = warp & 3;  // tensor-memory lanes [32*quad, 32*quad + 32)
    const int row = quad * 32 + lane;              // weight row inside the tile
    const int64_t mrow = static_cast<int64_t>(rt) * 128 + row;
    mbar_wait(smem_u32(&acc_full_bar), 0, &abort_flag);
    // A wait that gave up has raised abort_flag before this barrier, so the four epilogue warps
    // agree on `ok` and take the barriers below together or not at all.
    named_barrier_sync(1, 128);
    const bool ok = *static_cast<volatile int*>(&abort_flag) == 0;
    auto store16 = [&](int c, const float (&val)[16]) {
      if (mrow < p.m) {
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          if (c + t < p.s) {
            if (OUT_BF16)
              reinterpret_cast<__nv_bfloat16*>(p.y)[(c + t) * p.ldy + mrow] = __float2bfloat16_rn(val[t]);
            else
              reinterpret_cast<float*>(p.y)[(c + t) * p.ldy + mrow] = val[t];
          }
        }
      }
    };
    if (ok) {
      tc_fence_after_sync();
      epi_ok = true;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
      float* part_smem = reinterpret_cast<float*>(smem);  // cluster mode: every MMA has completed, the ring is free
      float* mine = p.partial + (static_cast<int64_t>(rt) * p.splits + sp) * (NTOK * 128) + row;
#pragma unroll 1
      for (int c = 0; c < NTOK; c += 16) {
        if (c >= p.s) break;
        uint32_t v[16];
        tmem_ld_32x32b_x16(taddr + c, v);
        tmem_ld_wait();
        if (by_cluster && NTOK == 16) {
          // push: token t goes to CTA t mod splits, slot [this split][t / splits]
          const int per = (p.s + p.splits - 1) / p.splits;
          const uint32_t recv0 = smem_u32(smem + Cfg::kStages * Cfg::kStageBytes) + static_cast<uint32_t>(sp * per * 512 + row * 4);
#pragma unroll
          for (int t = 0; t < 16; ++t)
            if (t < p.s)
              st_shared_cluster_f32(map_to_cta(recv0 + static_cast<uint32_t>((t / p.splits) * 512), static_cast<uint32_t>(t % p.splits)),
                                    __uint_as_float(v[t]));
        } else if (by_cluster) {
#pragma unroll
          for (int t = 0; t < 16; ++t)
            if (c + t < p.s) part_smem[(c + t) * 128 + row] = __uint_as_float(v[t]);
        } else if (p.splits > 1) {
#pragma unroll
          for (int t = 0; t < 16; ++t)
            if (c + t < p.s) __stcg(mine + (c + t) * 128, __uint_as_float(v[t]));
        } else {
          float val[16];
#pragma unroll
          for (int t = 0; t < 16; ++t) val[t] = __uint_as_float(v[t]);
          store16(c, val);
        }
      }
      tc_fence_before_sync();

      if (!by_cluster && p.splits > 1) {
        __threadfence();
        named_barrier_sync(1, 128);
        if (warp == 2 && lane == 0) ticket_slot = atomicAdd(p.tickets + rt, 1u);
        named_barrier_sync(1, 128);
        if (ticket_slot == static_cast<uint32_t>(p.splits - 1)) {
          __threadfence();
          // Sum in split order (deterministic).  Loads are issued in independent batches -- over the
          // tokens when there are many, over the splits when there are few -- so that their latencies
          // overlap instead of adding up.
          const float* all = p.partial + static_cast<int64_t>(rt) * p.splits * (NTOK * 128) + row;
          if (p.s > 4) {
#pragma unroll 1
            for (int c = 0; c < NTOK; c += 16) {
              if (c >= p.s) break;
              float acc[16];
#pragma unroll
              for (int t = 0; t < 16; ++t) acc[t] = 0.0f;
              constexpr int QB = 4;  // splits per batch: 64 loads in flight
              for (int q0 = 0; q0 < p.splits; q0 += QB) {
                float part[QB][16];
#pragma unroll
                for (int qq = 0; qq < QB; ++qq)
#pragma unroll
                  for (int t = 0; t < 16; ++t)
                    part[qq][t] = (q0 + qq < p.splits && c + t < p.s)
                                      ? __ldcg(all + (q0 + qq) * (NTOK * 128) + (c + t) * 128) : 0.0f;
#pragma unroll
                for (int qq = 0; qq < QB; ++qq)
#pragma unroll
                  for (int t = 0; t < 16; ++t) acc[t] += part[qq][t];
              }
              store16(c, acc);
            }
          } else {
            float acc[16];
#pragma unroll
            for (int t = 0; t < 16; ++t) acc[t] = 0.0f;
            for (int q0 = 0; q0 < p.splits; q0 += 8) {
              float part[8][4];
#pragma unroll
              for (int qq = 0; qq < 8; ++qq)
#pragma unroll
                for (int t = 0; t < 4; ++t)
                  part[qq][t] = (q0 + qq < p.splits && t < p.s) ? __ldcg(all + (q0 + qq) * (NTOK * 128) + t * 128) : 0.0f;
#pragma unroll
              for (int qq = 0; qq < 8; ++qq)
#pragma unroll
                for (int t = 0; t < 4; ++t) acc[t] += part[qq][t];
            }
            store16(0, acc);
          }
          if (warp == 2 && lane == 0) p.tickets[rt] = 0;  // ready for the next call
        }
      }
    }
  }

  if (by_cluster) {
    // Every thread of every CTA of the cluster takes both barriers, whatever happened above.
    __syncthreads();
    cluster_sync_all();
    if (NTOK == 16) {
      // Push mode: everything this CTA owns has arrived in its receive buffer (the barrier above
      // orders the other CTAs' remote stores before this point); add in split order (deterministic).
      // No CTA touches another's shared memory any more, so no second barrier.
      if (warp >= 2 && epi_ok) {
        const int row = (warp & 3) * 32 + lane;
        const int64_t mrow = static_cast<int64_t>(rt) * 128 + row;
        const int per = (p.s + p.splits - 1) / p.splits;
        const float* recv = reinterpret_cast<const float*>(smem + Cfg::kStages * Cfg::kStageBytes) + row;
        for (int j = 0; sp + j * p.splits < p.s; ++j) {
          const int t = sp + j * p.splits;
          float part[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) part[q] = q < p.splits ? recv[(q * per + j) * 128] : 0.0f;
          float acc = part[0];
#pragma unroll
          for (int q = 1; q < 8; ++q) acc += part[q];
          if (mrow < p.m) {
            if (OUT_BF16)
              reinterpret_cast<__nv_bfloat16*>(p.y)[t * p.ldy + mrow] = __float2bfloat16_rn(acc);
            else
              reinterpret_cast<float*>(p.y)[t * p.ldy + mrow] = acc;
          }
        }
      }
    } else if (warp >= 2 && epi_ok) {
      // Reduce-scatter: CTA sp adds, in split order (deterministic), the partial sums of tokens
      // sp, sp + splits, ... -- its own from local, the others' from distributed shared memory --
      // and writes those tokens of y.
      const int row = (warp & 3) * 32 + lane;
      const int64_t mrow = static_cast<int64_t>(rt) * 128 + row;
      const uint32_t mine = smem_u32(smem) + row * 4;
      for (int t = sp; t < p.s; t += p.splits) {
        float part[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
          part[q] = q < p.splits ? ld_shared_cluster_f32(map_to_cta(mine + t * 512, q)) : 0.0f;
        float acc = part[0];
#pragma unroll
        for (int q = 1; q < 8; ++q) acc += part[q];
        if (mrow < p.m) {
          if (OUT_BF16)
            reinterpret_cast<__nv_bfloat16*>(p.y)[t * p.ldy + mrow] = __float2bfloat16_rn(acc);
          else
            reinterpret_cast<float*>(p.y)[t * p.ldy + mrow] = acc;
        }
      }
    }
    if (NTOK != 16) cluster_sync_all();  // pull mode: nobody leaves while its shared memory may still be read
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

}  // namespace batq
