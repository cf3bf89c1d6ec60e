// Measurement kernels: (1) the block-scaled FP4 tensor-core rate with operands resident in shared
// memory (the denominator of the GEMM's roofline fraction), (2) a wait that runs out on purpose,
// to show that the library's bounded waits report and return.
#pragma once
#include <cuda.h>

#include "gemm_mxfp4.cuh"
#include "gemm_w4a8_pair.cuh"
#include "ptx.cuh"

namespace batq {

constexpr int kPeakThreads = 128;
constexpr int kPeakBatch = 8;            // K-steps between two commits
constexpr int kPeakSfbAtoms = 2;         // 256 weight rows
constexpr int kPeakABytes = 128 * kBKBytes;
constexpr int kPeakBBytes = 256 * kBKBytes;
constexpr int kPeakSfBytes = 1024 + kPeakSfbAtoms * 1024;
constexpr int kPeakOperandBytes = kPeakABytes + kPeakBBytes + kPeakSfBytes;
constexpr int kPeakSmemBytes = kPeakOperandBytes + 1024;
constexpr int kPeakSfCols = 8 + 2 * 4 * kPeakSfbAtoms;
// The optional load stream: a ring of stages the size of a GEMM stage (two boxes of 128 rows x 128
// bytes), filled by TMA from a prepared weight and read by nobody.
constexpr int kPeakLoadStages = 5;   // at most; PeakParams::load_stages of them are used
constexpr int kPeakLoadBoxBytes = 128 * kBKBytes;
constexpr int kPeakLoadStageBytes = 2 * kPeakLoadBoxBytes;
constexpr int kPeakSmemBytesLoads = (kPeakOperandBytes + 1023) / 1024 * 1024 + kPeakLoadStages * kPeakLoadStageBytes + 1024;

struct PeakParams {
  int32_t iters;      // K-steps (four MMAs of K = 64 each); 0 = no MMAs
  int32_t bn;         // tile width
  int32_t sf_copies;  // 0: scale factors copied to tensor memory once; 1: again before every K-step, as a GEMM must
  int32_t load_iters; // stages (32 KiB) every CTA loads next to the MMAs, unsynchronised with them; 0 = none
  int32_t w_row_tiles;  // the weight the loads walk over: 128-row tiles and 128-byte K steps
  int32_t w_k_steps;
  int32_t load_stages;  // 1..kPeakLoadStages: copies in flight per CTA
  int32_t load_sharing; // >= 1: this many CTAs (blockIdx.x / load_sharing equal) load the same boxes at the same time
  int32_t load_from_peer;  // pairs only, != 0: the second box of every stage is not loaded from L2 but copied from
                           // the other CTA of the pair, shared memory to shared memory
  int32_t sf_col;       // tensor-memory column of the scale factors (behind the accumulators: 256, or 448 with bn2)
  int32_t bn2;          // KIND 1: width of the second MMA (into columns 256.. on the same operands: the issue
                        // pattern of the wide-tile GEMM)
  int32_t store_iters;  // stages (32 KiB) warps 2-3 of every CTA write into the ring with ordinary stores; 0 = none
};

// PAIR = false: every CTA issues tcgen05.mma.cta_group::1 on a 128 x bn tile.
// PAIR = true:  clusters of two; the leader issues cta_group::2 on a 256 x bn tile whose A rows and
//               B rows are split over the two CTAs' shared memories, as in the CTA-pair GEMM.
// With load_iters > 0 warp 0 of every CTA streams boxes of a prepared weight into a ring of its own
// while warp 1 issues the MMAs on the resident operands: the two share the shared memory and the
// path from L2 but never wait for one another, which separates what the hardware sustains from what
// a GEMM's barrier hand-shakes cost.
// Shared memory of this CTA -> shared memory of another CTA of the cluster; the bytes are counted
// on a barrier of the destination CTA.  Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_s2s_cluster(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes,
                                                 uint32_t bar_cluster) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   dst_cluster),
               "r"(src_cta), "r"(bytes), "r"(bar_cluster)
               : "memory");
}

// KIND 0: kind::mxf4 on one accumulator; 1: kind::mxf4, every MMA followed by one of width bn2 into
// a second accumulator; 2: kind::mxf8f6f4; 3: kind::mxf4 issued by the CTA-pair GEMM's own loop
// (a wait, a fence, eight scale copies into alternating slots, four MMAs from stage-dependent
// descriptors and a commit per K-step, the whole warp around one elected lane).  A template parameter, not a field of PeakParams: the
// issue loop must stay free of run-time branches (with two of them per MMA the same loop measured
// 6.4 instead of 8.1 PFLOP/s: the rate at which one thread can issue is part of what is measured).
template <bool PAIR, int KIND>
__global__ void __launch_bounds__(kPeakThreads, 1)
mma_peak_kernel(const __grid_constant__ CUtensorMap tmap_w, const PeakParams p) {
  extern __shared__ uint8_t peak_smem_raw[];
  __shared__ __align__(8) uint64_t batch_bar[2];
  __shared__ __align__(8) uint64_t load_bar[kPeakLoadStages];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(peak_smem_raw) + 1023) & ~uintptr_t(1023));

  // Operands: every byte pattern is a pair of valid E2M1 codes; scale bytes 125..129 (2^-2..2^2).
  uint32_t h = 0x9E3779B9u * (blockIdx.x * kPeakThreads + tid + 1u);
  for (int i = tid; i < (kPeakABytes + kPeakBBytes) / 4; i += kPeakThreads) {
    h = h * 1664525u + 1013904223u;
    // (8-bit containers: the top two bits of every byte clear, so that no E4M3 code is a NaN)
    reinterpret_cast<uint32_t*>(smem)[i] = KIND == 2 ? ((h ^ (h >> 15)) & 0x3F3F3F3Fu) : (h ^ (h >> 15));
  }
  for (int i = tid; i < kPeakSfBytes; i += kPeakThreads) {
    h = h * 1664525u + 1013904223u;
    smem[kPeakABytes + kPeakBBytes + i] = static_cast<uint8_t>(125u + (h >> 24) % 5u);
  }
  if (tid == 0) {
    mbar_init(smem_u32(&batch_bar[0]), 1);
    mbar_init(smem_u32(&batch_bar[1]), 1);
    for (int i = 0; i < kPeakLoadStages; ++i) mbar_init(smem_u32(&load_bar[i]), 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    if (PAIR) { tmem_alloc_pair(smem_u32(&tmem_base_slot), 512); tmem_relinquish_pair(); }
    else      { tmem_alloc(smem_u32(&tmem_base_slot), 512); tmem_relinquish(); }
  }
  fence_proxy_async_smem();   // the generic-proxy writes above are read by the tensor cores
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0 && p.load_iters > 0) {
    // ------------------------------------------------------------ load stream (every CTA its own)
    const uint32_t ring = smem_u32(smem) + (kPeakOperandBytes + 1023) / 1024 * 1024;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    int issued = 0;
    for (int i = 0; i < p.load_iters; ++i) {
      // a stage is refilled as soon as the copy that filled it last has landed
      if (i >= p.load_stages) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&load_bar[stage]), phase ^ 1u, &abort_flag));
        if (!ok) break;
      }
      if (elect_one()) {
        const int rt = static_cast<int>((static_cast<int64_t>(blockIdx.x / p.load_sharing) * 13 + i / p.w_k_steps) % p.w_row_tiles);
        const int rt2 = (rt + p.w_row_tiles / 2) % p.w_row_tiles;
        const int kt = i % p.w_k_steps;
        const uint32_t dst = ring + stage * kPeakLoadStageBytes;
        const uint32_t bar = smem_u32(&load_bar[stage]);
        mbar_arrive_expect_tx(bar, kPeakLoadStageBytes);
        tma_load_2d(dst, &tmap_w, kt * kBKBytes, rt * 128, bar);
        if (PAIR && p.load_from_peer) {
          // this CTA fills the second half of the PEER's stage (from its own resident operands) and
          // the peer fills this CTA's: 16 KiB of every stage arrive over the cluster's network
          const uint32_t peer = rank ^ 1u;
          bulk_s2s_cluster(map_to_cta(dst + kPeakLoadBoxBytes, peer), smem_u32(smem), kPeakLoadBoxBytes,
                           map_to_cta(bar, peer));
        } else {
          tma_load_2d(dst + kPeakLoadBoxBytes, &tmap_w, kt * kBKBytes, rt2 * 128, bar);
        }
      }
      ++issued;
      if (++stage == p.load_stages) { stage = 0; phase ^= 1u; }
    }
    // drain: every copy issued has landed before the CTA exits (also after a wait that gave up)
    if ((tid & 31) == 0) {
      const int pending = min(issued, p.load_stages);
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = p.load_stages - 1; phase ^= 1u; }
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&load_bar[stage]), phase) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
    __syncwarp();
  }

  if (warp >= 2 && p.store_iters > 0) {
    // ------------------------------------------------------------ ordinary shared-memory stores
    // 64 threads x 16 bytes = 1 KiB per instruction, 32 instructions per stage; the ring is only
    // written (with load_iters > 0 as well, both write the same bytes: nobody reads them).
    uint8_t* ring = smem + (kPeakOperandBytes + 1023) / 1024 * 1024;
    const int t64 = tid - 64;
    uint4 val = make_uint4(tid, 2u, 3u, 4u);
    for (int i = 0; i < p.store_iters; ++i) {
      uint8_t* st = ring + (i % p.load_stages) * kPeakLoadStageBytes + t64 * 16;
#pragma unroll 8
      for (int j = 0; j < kPeakLoadStageBytes / 1024; ++j) {
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(st + j * 1024)), "r"(val.x), "r"(val.y),
                     "r"(val.z), "r"(val.w)
                     : "memory");
      }
      val.x += 1u;
    }
  }

  if (warp == 1 && rank == 0 && p.iters > 0) {
    const uint32_t smem_base = smem_u32(smem);
    const uint64_t adesc = make_smem_desc(smem_base, 16, 1024, 2);
    const uint64_t bdesc = adesc + (kPeakABytes >> 4);
    const uint64_t sfd = make_smem_desc(smem_base + kPeakABytes + kPeakBBytes, 0, 128, 0);
    const uint32_t sfa_col = tmem_base + static_cast<uint32_t>(p.sf_col);
    const uint32_t sfb_col = sfa_col + 8;
    const uint32_t idesc0 = mxf4_idesc(PAIR ? 256 : 128, p.bn);
    const uint32_t idesc1 = idesc0 | (2u << 29) | (2u << 4);
    const uint32_t idesc8 = mxf8f6f4_idesc_e4m3_e2m1(PAIR ? 256 : 128, p.bn);
    const uint32_t idesc2 = mxf4_idesc(PAIR ? 256 : 128, p.bn2 > 0 ? p.bn2 : 64);
    bool ok = true;
    if (elect_one()) {
      // scale factors once: shared -> tensor memory, the layout of the GEMM kernels
      if (PAIR) {
        tc_cp_32x128b_warpx4_pair(sfa_col, sfd);
        tc_cp_32x128b_warpx4_pair(sfa_col + 4, sfd + 32);
      } else {
        tc_cp_32x128b_warpx4(sfa_col, sfd);
        tc_cp_32x128b_warpx4(sfa_col + 4, sfd + 32);
      }
#pragma unroll
      for (int rt = 0; rt < kPeakSfbAtoms; ++rt)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const uint32_t col = sfa_col + 8 + c * 4 * kPeakSfbAtoms + 4 * rt;
          const uint64_t src = sfd + ((1024 + rt * 1024 + c * 512) >> 4);
          if (PAIR) tc_cp_32x128b_warpx4_pair(col, src); else tc_cp_32x128b_warpx4(col, src);
        }
    }
    __syncwarp();
    if (KIND == 3) {
      // The issue loop of the CTA-pair GEMM, statement for statement: the whole warp waits for a stage
      // (here a barrier phase that is complete from the start), one elected lane copies the scales of
      // the K-step into one of two slots and issues its four MMAs from descriptors that depend on the
      // run-time stage index, then commits.  All five "stages" are the same resident operands.
      const uint32_t zero = static_cast<uint32_t>(p.w_k_steps - 1);   // 0 at run time (no load stream)
      const uint64_t ab_desc0 = adesc;
      const uint32_t sf_tmem0 = sfa_col;
      const uint32_t full0 = smem_u32(&load_bar[0]);
      int stage = 0;
      uint32_t phase = 1;
      uint32_t g = 0;
      for (int kt = 0; kt < p.iters && ok; ++kt, ++g) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(full0 + 8u * stage * zero, phase, &abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t soff = static_cast<uint32_t>(stage * (36864 >> 4)) * zero;
        const uint64_t a_k = ab_desc0 + soff;
        const uint64_t b_k = a_k + (kPeakABytes >> 4);
        const uint64_t sfd_k = sfd + soff;
        const uint32_t sfa_k = sf_tmem0 + (g & 1u) * 24u;
        const uint32_t sfb_k = sfa_k + 8;
        if (elect_one()) {
          if (PAIR) { tc_cp_32x128b_warpx4_pair(sfa_k, sfd_k); tc_cp_32x128b_warpx4_pair(sfa_k + 4, sfd_k + 32); }
          else      { tc_cp_32x128b_warpx4(sfa_k, sfd_k); tc_cp_32x128b_warpx4(sfa_k + 4, sfd_k + 32); }
#pragma unroll
          for (int rt = 0; rt < kPeakSfbAtoms; ++rt)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              const uint32_t col = sfa_k + 8 + c * 4 * kPeakSfbAtoms + 4 * rt;
              const uint64_t src = sfd_k + ((1024 + rt * 1024 + c * 512) >> 4);
              if (PAIR) tc_cp_32x128b_warpx4_pair(col, src); else tc_cp_32x128b_warpx4(col, src);
            }
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint32_t c = kb >> 1;
            const uint32_t sfid = (kb & 1) * 2;
            const uint32_t sa = (sfa_k + 4 * c) | (sfid << 30);
            const uint32_t sb = (sfb_k + c * 4 * kPeakSfbAtoms) | (sfid << 30);
            const uint32_t acc = (kt | kb) != 0 ? 1u : 0u;
            if (PAIR) tc_mma_mxf4_pair(tmem_base, a_k + 2 * kb, b_k + 2 * kb, (kb & 1) ? idesc1 : idesc0, sa, sb, acc);
            else      tc_mma_mxf4(tmem_base, a_k + 2 * kb, b_k + 2 * kb, (kb & 1) ? idesc1 : idesc0, sa, sb, acc);
          }
          if (PAIR) tc_commit_pair_local(smem_u32(&load_bar[1])); else tc_commit(smem_u32(&load_bar[1]));
        }
        if (++stage == 5) { stage = 0; phase ^= zero; }
      }
      if (elect_one()) {
        if (PAIR) tc_commit_pair_local(smem_u32(&batch_bar[0])); else tc_commit(smem_u32(&batch_bar[0]));
      }
      __syncwarp();
      mbar_wait(smem_u32(&batch_bar[0]), 0, &abort_flag);
      __syncwarp();
    }
    const int n_batches = KIND == 3 ? 0 : (p.iters + kPeakBatch - 1) / kPeakBatch;
    for (int b = 0; b < n_batches && ok; ++b) {
      // at most two batches in flight, like a ring of stages
      if (b >= 2) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&batch_bar[b & 1]), ((b >> 1) - 1) & 1u, &abort_flag));
        if (!ok) break;
      }
      if (elect_one()) {
        const int k1 = min(p.iters, (b + 1) * kPeakBatch);
        for (int kt = b * kPeakBatch; kt < k1; ++kt) {
          if (p.sf_copies) {
            if (PAIR) {
              tc_cp_32x128b_warpx4_pair(sfa_col, sfd);
              tc_cp_32x128b_warpx4_pair(sfa_col + 4, sfd + 32);
            } else {
              tc_cp_32x128b_warpx4(sfa_col, sfd);
              tc_cp_32x128b_warpx4(sfa_col + 4, sfd + 32);
            }
#pragma unroll
            for (int rt = 0; rt < kPeakSfbAtoms; ++rt)
#pragma unroll
              for (int c = 0; c < 2; ++c) {
                const uint32_t col = sfa_col + 8 + c * 4 * kPeakSfbAtoms + 4 * rt;
                const uint64_t src = sfd + ((1024 + rt * 1024 + c * 512) >> 4);
                if (PAIR) tc_cp_32x128b_warpx4_pair(col, src); else tc_cp_32x128b_warpx4(col, src);
              }
          }
          if (KIND == 2) {
#pragma unroll
            for (uint32_t kb = 0; kb < 4; ++kb) {   // byte kb of one scale column per 32 rows
              const uint32_t id = idesc8 | (kb << 29) | (kb << 4);
              const uint32_t acc = (kt | static_cast<int>(kb)) != 0 ? 1u : 0u;
              if (PAIR) tc_mma_mxf8f6f4_pair(tmem_base, adesc + 2 * kb, bdesc + 2 * kb, id, sfa_col | (kb << 30), sfb_col | (kb << 30), acc);
              else      tc_mma_mxf8f6f4(tmem_base, adesc + 2 * kb, bdesc + 2 * kb, id, sfa_col | (kb << 30), sfb_col | (kb << 30), acc);
            }
          } else {
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
              const uint32_t c = kb >> 1;
              const uint32_t sfid = (kb & 1) * 2;
              const uint32_t sa = (sfa_col + 4 * c) | (sfid << 30);
              const uint32_t sb = (sfb_col + c * 4 * kPeakSfbAtoms) | (sfid << 30);
              const uint32_t acc = (kt | kb) != 0 ? 1u : 0u;
              if (PAIR) tc_mma_mxf4_pair(tmem_base, adesc + 2 * kb, bdesc + 2 * kb, (kb & 1) ? idesc1 : idesc0, sa, sb, acc);
              else      tc_mma_mxf4(tmem_base, adesc + 2 * kb, bdesc + 2 * kb, (kb & 1) ? idesc1 : idesc0, sa, sb, acc);
              if (KIND == 1) {
                const uint32_t i2 = idesc2 | ((kb & 1) ? ((2u << 29) | (2u << 4)) : 0u);
                if (PAIR) tc_mma_mxf4_pair(tmem_base + 256, adesc + 2 * kb, bdesc + 2 * kb, i2, sa, sb, acc);
                else      tc_mma_mxf4(tmem_base + 256, adesc + 2 * kb, bdesc + 2 * kb, i2, sa, sb, acc);
              }
            }
          }
        }
        if (PAIR) tc_commit_pair_local(smem_u32(&batch_bar[b & 1])); else tc_commit(smem_u32(&batch_bar[b & 1]));
      }
      __syncwarp();
    }
    // drain: the last two batches (fewer if there were fewer)
    for (int b = max(0, n_batches - 2); b < n_batches; ++b)
      if (!mbar_wait(smem_u32(&batch_bar[b & 1]), (b >> 1) & 1u, &abort_flag)) break;
    __syncwarp();
  }

  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) cluster_sync_all();   // the peer's shared memory is read until the leader has drained
  if (warp == 1) {
    tc_fence_after_sync();
    if (PAIR) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512);
  }
}

// One warp waits on a barrier nothing signals; the bounded wait gives up after limit_ns, records
// the time-out for the host and the kernel returns normally.
__global__ void wait_timeout_kernel(uint64_t limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_ns);
}

}  // namespace batq
