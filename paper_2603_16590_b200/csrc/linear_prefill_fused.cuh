// The whole layer for prefill shapes in ONE kernel: activation transform + block clip + MXFP4
// quantisation (stages 1+2; Eq. 1-4, Sec. 2) followed by the MXFP4 x MXFP4 GEMM (stage 3,
// Sec. 3.2) on the same persistent grid of CTA pairs -- the "quantiser in the GEMM prologue" form
// of the path for s > 128.  No output tile requantises anything: X is quantised exactly once.
//
// Phase 1 (quantise).  The grid's CTA pairs share the 256-token x 4-block units of X (a pair's
// leader owns the first 128 token rows of a unit, its peer the other 128).  Per unit: TMA loads
// the bf16 tile, tcgen05.mma.cta_group::2 (kind::f16, M = 256 over the pair, N = 32) multiplies
// each 32-channel block by the dense block matrix P_j^T (three bf16 terms, see
// quantize_act_tc.cuh; each CTA stages the 16 output channels of P_j^T that its half of the B
// operand holds), sixteen quantiser warps clip, scale and round their token rows out of tensor
// memory, and a store warp writes the unit's codes (one TMA store) and scale atom (one bulk
// copy) to the workspace.  When all stores of a CTA have completed it publishes that in its own
// flag word in the workspace (no atomics: one release store per CTA).
//
// Phase 2 (GEMM).  Exactly the CTA-pair GEMM of gemm_mxfp4_pair.cuh (same schedule, same
// barriers, same tensor-memory plan); instead of waiting for a preceding grid, the TMA producer
// of a CTA first waits -- bounded -- until every CTA's flag says that its share of X is in the
// workspace.
//
// Flag words.  The workspace holds a run counter and one flag per CTA.  Every CTA reads the run
// counter once the grid before it has completed (griddepcontrol.wait); counter + 1 is the number
// of this run, and a CTA that has finished phase 1 stores that number, mixed with a tag unique to
// the call (host counter), in its flag.  Flags of earlier runs -- of this launch or of any other
// that shares the workspace, replays of a CUDA graph included -- hold smaller numbers and never
// read as done, and neither does whatever an uninitialised workspace holds.  CTA 0 writes the new
// run number back after it has seen every flag, i.e. after every CTA has read the old one.
//
// All tcgen05 instructions of the kernel use cta_group::2.  Every wait is bounded; a wait that
// gives up raises the CTA's abort flag, records the time-out for the host and falls through to
// the common exit, where tensor memory is released.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_mxfp4_pair.cuh"
#include "ptx.cuh"
#include "quantize_act_tc.cuh"

namespace batq {

constexpr int kPfThreads = kQtThreads;        // 19 warps: producer, MMA issuer, 16 quantiser warps, store warp
constexpr int kPfXStages = 3;
constexpr int kPfOutBufs = 3;
constexpr int kPfHalfTermBytes = kQtTermBytes / 2;                       // 16 of the 32 rows of one term of P_j^T
constexpr int kPfStripImageBytes = kQtGroups * 3 * kPfHalfTermBytes;     // 12 KiB per CTA and strip
constexpr int kPfOutBufBytes = kQtCodeTileBytes + 512;                   // 128 rows x 64 bytes of codes + one scale atom
constexpr int kPfPhase1Bytes = kPfXStages * kQtStageBytes + 2 * kPfStripImageBytes + kPfOutBufs * kPfOutBufBytes;
constexpr int kPfSmemBytes = PairCfg::kSmemBytes;
static_assert(kPfPhase1Bytes + 1024 <= kPfSmemBytes, "phase 1 fits the GEMM's shared memory");
static_assert((kPfXStages * kQtStageBytes) % 1024 == 0 && kPfStripImageBytes % 1024 == 0 && kPfOutBufBytes % 512 == 0,
              "alignment of the phase-1 regions");
constexpr int kPfTagShift = 24;               // flag word: run number ^ (tag << 24)

struct PrefillFusedParams {
  PairParams g;            // the GEMM: shapes, schedule, y
  int32_t n;               // channels
  int32_t k;               // n / 32
  int32_t n_strips;        // k / 4 (the host takes this path only when the scale atoms come in pairs)
  int32_t n_row_tiles;     // ceil(s / 128)
  int32_t n_units;         // m_pairs * n_strips
  const float* clip_lo;    // [k] or NULL
  const float* clip_hi;
  uint8_t* scales;         // activation scale atoms (BATQ_SF_MMA layout) in the workspace
  unsigned long long* sync;    // in the workspace: [0] run counter, [1 + i] flag of CTA i
  unsigned long long tag;      // this call's tag (40 bits)
};

__device__ __forceinline__ void tc_mma_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 4-D tiled tensor-map load whose completion is counted on a barrier of either CTA of the pair.
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst_smem, const void* tmap, int32_t c0, int32_t c1, int32_t c2,
                                                 int32_t c3, uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, "
      "{%2, %3, %4, %5}], [%6];" ::"r"(dst_smem),
      "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(cluster_bar)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned long long ld_acquire_gpu_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ void st_release_gpu_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// Bounded wait of a whole warp until all n flag words equal `want` (lane l polls words l, l + 32, ...).
__device__ __forceinline__ bool flags_wait_all(const unsigned long long* flags, int n, unsigned long long want,
                                               volatile int* abort_flag) {
  const int lane = threadIdx.x & 31;
  uint64_t t0 = 0;
  for (;;) {
    bool mine = true;
    for (int i = lane; i < n; i += 32) mine = mine && (ld_acquire_gpu_u64(flags + i) == want);
    if (__all_sync(0xFFFFFFFFu, mine)) return true;
    if (__any_sync(0xFFFFFFFFu, *abort_flag != 0)) return false;
    const uint64_t now = global_timer_ns();
    if (t0 == 0) t0 = now;
    if (__any_sync(0xFFFFFFFFu, now - t0 > kWaitLimitNs)) {
      if (lane == 0) {
        *abort_flag = 1;
        atomicExch(&g_device_error, 1);
      }
      return false;
    }
    __nanosleep(200);
  }
}

template <bool CLIP, bool OUT_BF16>
__global__ void __launch_bounds__(kPfThreads, 1)
linear_prefill_fused_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_pimg,
                            const __grid_constant__ CUtensorMap tmap_codes, const __grid_constant__ CUtensorMap tmap_a,
                            const __grid_constant__ CUtensorMap tmap_b32, const __grid_constant__ CUtensorMap tmap_sfa,
                            const __grid_constant__ CUtensorMap tmap_sfb, const __grid_constant__ CUtensorMap tmap_y,
                            const __grid_constant__ PrefillFusedParams q) {
  using Cfg = PairCfg;
  const PairParams& p = q.g;
  extern __shared__ uint8_t pf_smem_raw[];
  // phase 1
  __shared__ __align__(8) uint64_t x_full[kPfXStages];    // leader: both CTAs' X tiles of a unit have landed
  __shared__ __align__(8) uint64_t x_empty[kPfXStages];   // both CTAs: the MMAs have read the stage
  __shared__ __align__(8) uint64_t p_full[2];             // leader: both CTAs' halves of a strip's block matrices
  __shared__ __align__(8) uint64_t p_empty[2];            // both CTAs
  __shared__ __align__(8) uint64_t d_full[kQtDBufs];      // both CTAs: accumulators of a unit complete
  __shared__ __align__(8) uint64_t d_empty[kQtDBufs];     // leader: read out by the quantiser warps of both CTAs
  __shared__ __align__(8) uint64_t t_full[kPfOutBufs];    // per CTA: staging tile complete
  __shared__ __align__(8) uint64_t t_empty[kPfOutBufs];   // per CTA: staging tile read out by its stores
  __shared__ __align__(8) uint64_t q_drain;               // leader: all phase-1 MMAs done
  // phase 2
  __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];   // leader
  __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];  // both CTAs
  __shared__ __align__(8) uint64_t acc_full_bar[2];          // both CTAs
  __shared__ __align__(8) uint64_t acc_empty_bar[2];         // leader
  __shared__ __align__(8) uint64_t drain_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ unsigned long long run_number;                  // this run's number
  __shared__ unsigned long long flag_value;                  // what a finished CTA's flag holds in this run

  grid_launch_dependents();
  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const int lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(pf_smem_raw) + 1023) & ~uintptr_t(1023));
  // phase-1 view of the shared memory
  uint8_t* const x_smem = smem;
  uint8_t* const img_smem = smem + kPfXStages * kQtStageBytes;
  uint8_t* const out_smem = img_smem + 2 * kPfStripImageBytes;
  // phase-2 view: the GEMM's ring and epilogue staging
  uint8_t* const staging = smem + Cfg::kStages * Cfg::kStageBytes;

  if (tid == 0) {
    for (int i = 0; i < kPfXStages; ++i) { mbar_init(smem_u32(&x_full[i]), 1); mbar_init(smem_u32(&x_empty[i]), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&p_full[i]), 1); mbar_init(smem_u32(&p_empty[i]), 1); }
    for (int i = 0; i < kQtDBufs; ++i) {
      mbar_init(smem_u32(&d_full[i]), 1);
      mbar_init(smem_u32(&d_empty[i]), kQtQuantWarps);     // 8 warps of a group in each CTA
    }
    for (int i = 0; i < kPfOutBufs; ++i) {
      mbar_init(smem_u32(&t_full[i]), kQtQuantWarps / 2);
      mbar_init(smem_u32(&t_empty[i]), 1);
    }
    mbar_init(smem_u32(&q_drain), 1);
    for (int i = 0; i < Cfg::kStages; ++i) { mbar_init(smem_u32(&full_bar[i]), 1); mbar_init(smem_u32(&empty_bar[i]), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full_bar[i]), 1); mbar_init(smem_u32(&acc_empty_bar[i]), 8); }
    mbar_init(smem_u32(&drain_bar), 1);
    abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_x);
    tma_prefetch_desc(&tmap_pimg);
    tma_prefetch_desc(&tmap_codes);
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
  cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  // ================================================================================ phase 1
  // Units of this pair: a contiguous range; unit u = strip * m_pairs + row block.
  const int u0 = static_cast<int>(static_cast<int64_t>(q.n_units) * pair / n_pairs);
  const int u1 = static_cast<int>(static_cast<int64_t>(q.n_units) * (pair + 1) / n_pairs);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    // X may come from the grid before this one (programmatic dependent launch): wait for it here.
    // Nothing of this grid is written to global memory before data has flowed through this wait
    // in some CTA, and no counter reaches its target before every CTA's share has.
    grid_dependency_wait();
    const uint32_t x_full0_leader = map_to_cta(smem_u32(&x_full[0]), 0);
    const uint32_t p_full0_leader = map_to_cta(smem_u32(&p_full[0]), 0);
    int stage = 0;
    uint32_t phase = 0;
    int cur_strip = -1, n_img = 0;
    bool ok = true;
    for (int u = u0; u < u1 && ok; ++u) {
      const int strip = u / p.m_pairs;
      const int rb = u - strip * p.m_pairs;
      if (strip != cur_strip) {
        cur_strip = strip;
        const int pb = n_img & 1;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&p_empty[pb]), ((n_img >> 1) & 1) ^ 1u, &abort_flag));
        if (!ok) break;
        if (elect_one()) {
          if (rank == 0) mbar_arrive_expect_tx(smem_u32(&p_full[pb]), 2u * kPfStripImageBytes);
          // [4 blocks][3 terms][this CTA's 16 rows] of P^T, blocks past k read as zero
          tma_load_4d_pair(smem_u32(img_smem + pb * kPfStripImageBytes), &tmap_pimg, 0, static_cast<int>(rank), 0,
                           strip * kQtGroups, p_full0_leader + 8u * pb);
        }
        ++n_img;
      }
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&x_empty[stage]), phase ^ 1u, &abort_flag));
      if (!ok) break;
      if (elect_one()) {
        const uint32_t bar = x_full0_leader + 8u * stage;
        const uint32_t dst = smem_u32(x_smem + stage * kQtStageBytes);
        const int col0 = strip * (kQtGroups * 32);
        const int row0 = rb * 256 + static_cast<int>(rank) * kQtRows;
        if (rank == 0) mbar_arrive_expect_tx(smem_u32(&x_full[stage]), 2u * kQtStageBytes);
        tma_load_2d_pair(dst, &tmap_x, col0, row0, bar);
        tma_load_2d_pair(dst + kQtBoxBytes, &tmap_x, col0 + 64, row0, bar);
      }
      if (++stage == kPfXStages) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader only)
    if (rank == 0) {
      constexpr uint32_t idesc = f16_idesc_bf16(256, 32);
      const uint64_t a_desc0 = make_smem_desc(smem_u32(x_smem), 16, 1024, 2);    // 128-byte swizzle, K-major
      const uint64_t b_desc0 = make_smem_desc(smem_u32(img_smem), 128, 512, 0);  // no swizzle: LBO 128 (K), SBO 512 (N)
      int stage = 0;
      uint32_t phase = 0;
      int cur_strip = -1, n_img = 0, it = 0;
      bool ok = true;
      for (int u = u0; u < u1 && ok; ++u, ++it) {
        const int strip = u / p.m_pairs;
        if (strip != cur_strip) {
          if (cur_strip >= 0 && elect_one()) tc_commit_pair(smem_u32(&p_empty[(n_img - 1) & 1]), 3);
          cur_strip = strip;
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&p_full[n_img & 1]), (n_img >> 1) & 1u, &abort_flag));
          if (!ok) break;
          ++n_img;
        }
        const int pb = (n_img - 1) & 1;
        const int buf = it & (kQtDBufs - 1);
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&d_empty[buf]), ((it >> 2) & 1u) ^ 1u, &abort_flag));
        if (!ok) break;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&x_full[stage]), phase, &abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t a_stage = a_desc0 + static_cast<uint32_t>((stage * kQtStageBytes) >> 4);
        const uint64_t b_img = b_desc0 + static_cast<uint32_t>((pb * kPfStripImageBytes) >> 4);
        const uint32_t d0 = tmem_base + buf * (kQtGroups * 32);
        if (elect_one()) {
#pragma unroll
          for (int g = 0; g < kQtGroups; ++g) {
            // block g lives in box g / 2 at byte offset (g % 2) * 64 of each 128-byte row
            const uint64_t a_g = a_stage + static_cast<uint32_t>(((g >> 1) * kQtBoxBytes + (g & 1) * 64) >> 4);
            const uint64_t b_g = b_img + static_cast<uint32_t>((g * 3 * kPfHalfTermBytes) >> 4);
#pragma unroll
            for (int t = 2; t >= 0; --t)  // smallest term first
#pragma unroll
              for (int kk = 0; kk < 2; ++kk)
                tc_mma_f16_pair(d0 + g * 32, a_g + 2 * kk, b_g + static_cast<uint32_t>((t * kPfHalfTermBytes + kk * 256) >> 4),
                                idesc, (t == 2 && kk == 0) ? 0u : 1u);
          }
          tc_commit_pair(smem_u32(&x_empty[stage]), 3);
          tc_commit_pair(smem_u32(&d_full[buf]), 3);
        }
        if (++stage == kPfXStages) { stage = 0; phase ^= 1u; }
      }
      // every MMA of phase 1 has completed before either CTA reuses shared or tensor memory
      if (lane == 0) {
        tc_commit_pair_local(smem_u32(&q_drain));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&q_drain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
      __syncwarp();
    }
  } else if (warp == 2 + kQtQuantWarps) {
    // ------------------------------------------------------------ store warp (both CTAs)
    if (lane == 0) {
      // The grid before this one (possibly an earlier run of this very launch) has completed once
      // this returns: only then is the run counter final.
      grid_dependency_wait();
      run_number = *reinterpret_cast<volatile unsigned long long*>(q.sync) + 1ull;
      flag_value = run_number ^ (q.tag << kPfTagShift);
      int it = 0;
      bool ok = true;
      for (int u = u0; u < u1; ++u, ++it) {
        const int strip = u / p.m_pairs;
        const int rb = u - strip * p.m_pairs;
        const int row_tile = rb * 2 + static_cast<int>(rank);
        const int sb = it % kPfOutBufs;
        if (!mbar_wait(smem_u32(&t_full[sb]), static_cast<uint32_t>(it / kPfOutBufs) & 1u, &abort_flag)) { ok = false; break; }
        uint8_t* const ob = out_smem + sb * kPfOutBufBytes;
        tma_store_2d(&tmap_codes, strip * (kQtGroups * 16), row_tile * kQtRows, smem_u32(ob));   // rows past s are clipped
        if (row_tile < q.n_row_tiles)
          bulk_s2g(q.scales + (static_cast<int64_t>(row_tile) * p.katoms + strip) * 512, smem_u32(ob + kQtCodeTileBytes), 512);
        bulk_commit_group();
        if (it > 0) {  // the stores of the unit before this one have read their buffer: hand it back
          bulk_wait_group_read<1>();
          mbar_arrive(smem_u32(&t_empty[(it - 1) % kPfOutBufs]));
        }
      }
      // All stores of this CTA are in global memory: publish it (also with no units at all).
      bulk_wait_group<0>();
      if (ok) {
        fence_proxy_async_all();
        __threadfence();
        st_release_gpu_u64(q.sync + 1 + blockIdx.x, flag_value);
      }
    }
  } else {
    // ------------------------------------------------------------ quantiser warps (both CTAs)
    const int qw = warp - 2;            // 0..15
    const int quad = warp & 3;          // tensor-memory lanes [32 quad, 32 quad + 32)
    const int grp = qw >> 3;            // takes the units with it % 2 == grp
    const int half = (qw & 7) >> 2;     // blocks 2 half and 2 half + 1 of the unit
    const uint32_t d_empty0_leader = map_to_cta(smem_u32(&d_empty[0]), 0);
    for (int it = grp; u0 + it < u1; it += 2) {
      const int u = u0 + it;
      const int strip = u / p.m_pairs;
      const int buf = it & (kQtDBufs - 1);
      bool ok = mbar_wait(smem_u32(&d_full[buf]), (it >> 2) & 1u, &abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const int sb = it % kPfOutBufs;
      if (it >= kPfOutBufs) {
        ok = mbar_wait(smem_u32(&t_empty[sb]), static_cast<uint32_t>(it / kPfOutBufs - 1) & 1u, &abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
      }
      uint8_t* const ob = out_smem + sb * kPfOutBufBytes;
#pragma unroll 1
      for (int e = 0; e < 2; ++e) {
        const int g = 2 * half + e;
        const int j = strip * kQtGroups + g;
        const uint32_t taddr = tmem_base + buf * (kQtGroups * 32) + g * 32 + (static_cast<uint32_t>(quad * 32) << 16);
        uint32_t v[32];
        tmem_ld_32x32b_x32(taddr, v);
        tmem_ld_wait();
        if (e == 1) {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(d_empty0_leader + 8u * buf);  // both accumulator rows have been read
        }
        float o[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(v[i]);
        float mn0 = fmin3(o[0], o[1], o[2]), mn1 = fmin3(o[3], o[4], o[5]), mn2 = fmin3(o[6], o[7], o[8]),
              mn3 = fmin3(o[9], o[10], o[11]);
        float mx0 = fmax3(o[0], o[1], o[2]), mx1 = fmax3(o[3], o[4], o[5]), mx2 = fmax3(o[6], o[7], o[8]),
              mx3 = fmax3(o[9], o[10], o[11]);
#pragma unroll
        for (int i = 12; i < 28; i += 8) {
          mn0 = fmin3(mn0, o[i], o[i + 1]); mn1 = fmin3(mn1, o[i + 2], o[i + 3]);
          mn2 = fmin3(mn2, o[i + 4], o[i + 5]); mn3 = fmin3(mn3, o[i + 6], o[i + 7]);
          mx0 = fmax3(mx0, o[i], o[i + 1]); mx1 = fmax3(mx1, o[i + 2], o[i + 3]);
          mx2 = fmax3(mx2, o[i + 4], o[i + 5]); mx3 = fmax3(mx3, o[i + 6], o[i + 7]);
        }
        mn0 = fmin3(mn0, o[28], o[29]); mn1 = fmin3(mn1, o[30], o[31]);
        mx0 = fmax3(mx0, o[28], o[29]); mx1 = fmax3(mx1, o[30], o[31]);
        const float mn = fminf(fmin3(mn0, mn1, mn2), mn3);
        const float mx = fmaxf(fmax3(mx0, mx1, mx2), mx3);
        float amax;
        if (CLIP) {
          const int jc = min(j, q.k - 1);
          const float lo = __ldg(q.clip_lo + jc) * mn;
          const float hi = __ldg(q.clip_hi + jc) * mx;
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = fminf(fmaxf(o[i], lo), hi);
          amax = fmaxf(fabsf(fminf(fmaxf(mn, lo), hi)), fabsf(fminf(fmaxf(mx, lo), hi)));
        } else {
          amax = fmaxf(fabsf(mn), fabsf(mx));
        }
        // shared scale: byte = max(biased_exponent(amax) - 2, 0)
        const int ef = static_cast<int>(__float_as_uint(amax) >> 23);
        const int sbyte = max(ef - 2, 0);
        const float inv = __uint_as_float(static_cast<uint32_t>(254 - sbyte) << 23);
        const int trow = quad * 32 + lane;
        uint32_t cw[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          float uu[8];
#pragma unroll
          for (int c = 0; c < 8; c += 2) mul2(o[8 * r + c], o[8 * r + c + 1], inv, uu[c], uu[c + 1]);
          cw[r] = e2m1x8_pack(uu);
        }
        // 64-byte swizzle: 16-byte chunk index XOR ((row / 2) & 3)
        *reinterpret_cast<uint4*>(ob + trow * 64 + ((g ^ ((trow >> 1) & 3)) << 4)) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
        ob[kQtCodeTileBytes + lane * 16 + quad * 4 + g] = static_cast<uint8_t>(j < q.k ? sbyte : 0);
      }
      fence_proxy_async_smem();   // the staging writes become visible to the TMA store
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&t_full[sb]));
    }
  }

  // ---------------------------------------------------------------- phase switch
  // Both CTAs: phase-1 MMAs drained (leader's warp 1), tensor-memory reads done, staging read out
  // by completed stores.  After this barrier shared and tensor memory belong to the GEMM.
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after_sync();
  const bool phase1_ok = *static_cast<volatile int*>(&abort_flag) == 0;

  // ================================================================================ phase 2
  const PairWalk walk0(p, pair, n_pairs);
  if (!phase1_ok) {
    // Given up in phase 1: no GEMM.  The loads of both CTAs are counted on the leader's barriers, so
    // neither CTA can wait for its own; give the copies already in flight ample time to land.
    if (tid == 0) {
      const uint64_t t0 = global_timer_ns();
      while (global_timer_ns() - t0 < 1000000ull) {}
    }
  } else if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (both CTAs)
    bool ok = true;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0_leader = map_to_cta(smem_u32(&full_bar[0]), 0);
    auto issue = [&](const PairTile& t, int kt, int stage) {
      const int m0 = t.mp * 256 + static_cast<int>(rank) * kBM;
      const int half = t.bn >> 1;
      const uint32_t st = smem_base + stage * Cfg::kStageBytes;
      const uint32_t bar = full0_leader + 8u * stage;
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
      tma_load_2d_pair(st, &tmap_a, kt * kBKBytes, m0, bar);
      tma_load_2d_pair(st + Cfg::kABytes + Cfg::kBBytes, &tmap_sfa, 0, (m0 >> 7) * p.katoms + 2 * kt, bar);
    };
    int stage = 0;
    uint32_t phase = 0;
    PairWalk w = walk0;
    PairTile t;
    // Every CTA's share of X quantised and in global memory?  (Every lane takes the acquire
    // itself, so whichever lane is elected to issue the copies below has observed the flags.)
    ok = flags_wait_all(q.sync + 1, static_cast<int>(gridDim.x), flag_value, &abort_flag);
    fence_proxy_async_all();   // the TMA loads below read what other SMs wrote
    // every CTA has read the run counter (it publishes its flag after that): CTA 0 moves it on
    if (ok && blockIdx.x == 0 && lane == 0) *reinterpret_cast<volatile unsigned long long*>(q.sync) = run_number;
    while (ok && w.next(t)) {
      for (int kt = 0; kt < p.k_steps; ++kt) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, &abort_flag));
        if (!ok) break;
        if (elect_one()) issue(t, kt, stage);
        if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) {
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
      uint32_t g = 0;
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
            tc_commit_pair(empty0 + 8u * stage, 3);
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
  } else if (warp < 6) {
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
#pragma unroll 1
      for (int c0 = 0; c0 < t.bn; c0 += kChunkCols) {
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
        const int col0 = t.n0 + c0;
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
        for (int qq = 0; qq < 8; ++qq)
          *reinterpret_cast<uint4*>(sb + ((qq ^ (lane & 7)) << 4)) = make_uint4(w[4 * qq], w[4 * qq + 1], w[4 * qq + 2], w[4 * qq + 3]);
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
      if (lane == 0) mbar_arrive_cluster(acc_empty0_leader + 8u * acc);
    }
    if (lane == 0) bulk_wait_group<0>();
  }

  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, Cfg::kTmemCols);
  }
}

}  // namespace batq
