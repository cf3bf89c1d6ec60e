// The whole layer in ONE kernel for a handful of tokens (decode, s <= 16): activation transform
// + block clip + MXFP4 quantisation fused into the prologue of the small-s GEMM.
//
//   x~ = x P (Eq. 1-2, Kronecker form V~ = L^T V R of Algorithm 1), block clip (Eq. 3-4), MXFP4
//   (Sec. 2), then Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} qx[s,j,i] * qw[m,j,i]
//   (the low-bit matrix multiplication of Sec. 3.2).
//
// At these sizes a call is a chain of latencies, not of bandwidths: two kernels (quantiser, GEMM)
// cost two launches, two prologues and a round trip of the codes through global memory.  Here a
// CTA owns 128 weight rows and a slice of at most 8 K-steps (2048 channels); while its TMA
// producer streams the weight slice, the four warps that will later run the epilogue quantise
// the matching slice of the s activation rows straight into shared memory, in the operand
// layout the MMA reads (the activations are tiny: every CTA of a K split redoes the same few
// blocks).  The K splits of a row tile form a thread-block cluster; their partial tiles are
// reduce-scattered through distributed shared memory (CTA q adds, in rank order, and writes tokens
// q, q + splits, ...: deterministic; no scratch in global memory, no atomics).
//
// Warp roles: warp 0 = TMA producer (weights), warp 1 = MMA issuer and tensor-memory owner,
// warps 2..5 = activation quantisers (four lanes per (token, block)), then epilogue.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_small_s.cuh"
#include "ptx.cuh"
#include "quantize_act.cuh"

namespace batq {

constexpr int kFusedThreads = 192;
constexpr int kFusedTok = 16;        // MMA N: tokens padded to 16
constexpr int kFusedMaxSteps = 8;    // K-steps per CTA (the slice of X it quantises)
constexpr int kFusedMaxSplits = 8;   // cluster size (portable limit)

struct FusedCfg {
  static constexpr int kWBytes = 128 * kBKBytes;            // 16 KiB of weight codes per K-step
  static constexpr int kSfBytes = 1024;                     // two 512-byte scale atoms (8 blocks)
  static constexpr int kStageBytes = kWBytes + kSfBytes;    // ring stage: weights only
  static constexpr int kStages = 5;
  static constexpr int kXStepBytes = kFusedTok * kBKBytes;  // 2 KiB of activation codes per K-step
  static constexpr int kXBytes = kFusedMaxSteps * kXStepBytes;
  static constexpr int kXSfBytes = kFusedMaxSteps * kSfBytes;
  static constexpr int kSfColsPerStage = 16;                // W: 2 atoms x 4 columns, X: 2 atoms x 4 columns
  static constexpr int kTmemCols = 128;
  static constexpr int kSmemBytes = kStages * kStageBytes + kXBytes + kXSfBytes + 1024;
  static_assert(kFusedTok + kStages * kSfColsPerStage <= kTmemCols, "tensor memory budget");
  static_assert(2 * (kSmemBytes + 2048) <= 232448, "two CTAs per SM");
  static_assert(kStageBytes % 1024 == 0, "stage alignment");
  static_assert(kXBytes >= kFusedTok * 128 * 4, "the partial tile reuses the activation-code region");
};

struct FusedParams {
  const uint16_t* x;     // bf16 bits [s x n], row stride ld
  int64_t ld;
  int32_t s;             // tokens (<= 16)
  int32_t n;
  int32_t k;             // n / 32
  const float* left;     // [.][gr x gr], left_stride floats apart (0 = shared); NULL = identity transform
  const float* right;    // [.][gc x gc]
  int32_t left_stride;
  int32_t right_stride;
  const float* clip_lo;  // [k] or NULL
  const float* clip_hi;
  const uint8_t* sfw;    // weight scales, BATQ_SF_MMA layout
  int32_t m;             // weight rows = output features
  int32_t katoms;        // 2*ceil(k/8)
  int32_t k_steps;       // ceil(n / 256)
  int32_t splits;        // gridDim.y = cluster size along y
  void* y;               // [s x m] fp32 or bf16, row stride ldy
  int64_t ldy;
};

// One (token, block) is worked on by FOUR lanes of a warp.  The block is a gr x gc matrix V
// (row-major, gr * gc = 32) and lane q of the group holds its elements 8 q .. 8 q + 7, i.e.
// 8 / GC whole rows when gc = GC is 8, 4 or 2; it produces the same elements of V~ = L^T V R
// (Algorithm 1) and one 32-bit word of codes.  Same arithmetic, in the same order, for every GC:
// fp32 fused multiply-adds, V R first (ascending inner index), then L^T (ascending row index).
// At this size a kernel is a chain of latencies: a short instruction stream per lane (the code is
// executed once, from a cold instruction cache) counts for more than the number of lanes.
//
// The constants of the layer; requested before the wait for the previous grid.
template <int GC>
struct QuadFactors {
  static constexpr int kGR = 32 / GC;   // rows of V = size of the left factor
  static constexpr int kRows = 8 / GC;  // rows of V held by one lane
  float R[GC * GC];        // right factor, [cc][c]
  float Lc[kRows * kGR];   // [rr][i] = L[i][q * kRows + rr]: the columns of L this lane's rows need
  float c_lo, c_hi;
};

// Lanes without an item (valid = false) get zeros and read nothing.  q = lane within the group.
template <int GC>
__device__ __forceinline__ void quad_load_factors(bool valid, const float* L, const float* R, const float* clip_lo,
                                                  const float* clip_hi, int j, int q, QuadFactors<GC>& f) {
  using F = QuadFactors<GC>;
  const bool xf = valid && L != nullptr;
#pragma unroll
  for (int i = 0; i < GC * GC / 4; ++i) {
    const float4 t = xf ? __ldg(reinterpret_cast<const float4*>(R) + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    f.R[4 * i] = t.x; f.R[4 * i + 1] = t.y; f.R[4 * i + 2] = t.z; f.R[4 * i + 3] = t.w;
  }
#pragma unroll
  for (int rr = 0; rr < F::kRows; ++rr)
#pragma unroll
    for (int i = 0; i < F::kGR; ++i) f.Lc[rr * F::kGR + i] = xf ? __ldg(L + i * F::kGR + q * F::kRows + rr) : 0.0f;
  f.c_lo = (valid && clip_lo != nullptr) ? __ldg(clip_lo + j) : 1.0f;
  f.c_hi = (valid && clip_hi != nullptr) ? __ldg(clip_hi + j) : 1.0f;
}

// Elements 8 q .. 8 q + 7 of the block (8 bf16 at xrow) -> this lane's 8 transformed, clipped
// values and the block's amax (the same in the four lanes).  Every lane of the warp calls this
// (shuffles inside); lanes without an item pass valid = false and get zeros.  x is read after the
// wait for the previous grid.
template <int GC>
__device__ __forceinline__ void quad_transform_clip(const uint16_t* xrow, bool valid, bool xform, bool clip,
                                                    const QuadFactors<GC>& f, int lane, float (&o)[8], float& amax,
                                                    bool bf16_mid = false) {
  using F = QuadFactors<GC>;
  grid_dependency_wait();
  uint4 q = make_uint4(0u, 0u, 0u, 0u);
  if (valid) q = ld_global_ordered_v4(xrow);
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  float v[8];
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    v[2 * h] = __uint_as_float(w[h] << 16);
    v[2 * h + 1] = __uint_as_float(w[h] & 0xFFFF0000u);
  }
  if (xform) {
    float U[8];  // this lane's rows of V R
#pragma unroll
    for (int rr = 0; rr < F::kRows; ++rr)
#pragma unroll
      for (int c = 0; c < GC; ++c) {
        float acc = v[rr * GC] * f.R[c];
#pragma unroll
        for (int cc = 1; cc < GC; ++cc) acc = fmaf(v[rr * GC + cc], f.R[cc * GC + c], acc);
        U[rr * GC + c] = bf16_mid ? round_bf16(acc) : acc;   // a BF16 implementation stores V R as bf16
      }
    const int base = lane & ~3;
    // this lane's rows of L^T (V R): row i of V R sits in lane i / kRows of the group
#pragma unroll
    for (int i = 0; i < F::kGR; ++i)
#pragma unroll
      for (int c = 0; c < GC; ++c) {
        const float u = __shfl_sync(0xFFFFFFFFu, U[(i % F::kRows) * GC + c], base + i / F::kRows);
#pragma unroll
        for (int rr = 0; rr < F::kRows; ++rr)
          o[rr * GC + c] = i == 0 ? f.Lc[rr * F::kGR] * u : fmaf(f.Lc[rr * F::kGR + i], u, o[rr * GC + c]);
      }
    if (bf16_mid) {
#pragma unroll
      for (int c = 0; c < 8; ++c) o[c] = round_bf16(o[c]);
    }
  } else {
#pragma unroll
    for (int c = 0; c < 8; ++c) o[c] = v[c];
  }
  float mn = o[0], mx = o[0];
#pragma unroll
  for (int c = 1; c < 8; ++c) {
    mn = fminf(mn, o[c]);
    mx = fmaxf(mx, o[c]);
  }
#pragma unroll
  for (int d = 1; d < 4; d <<= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, d));
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, d));
  }
  if (clip) {
    const float lo = f.c_lo * mn, hi = f.c_hi * mx;
#pragma unroll
    for (int c = 0; c < 8; ++c) o[c] = fminf(fmaxf(o[c], lo), hi);
    amax = fmaxf(fabsf(fminf(fmaxf(mn, lo), hi)), fabsf(fminf(fmaxf(mx, lo), hi)));
  } else {
    amax = fmaxf(fabsf(mn), fabsf(mx));
  }
}

// This lane's 8 values -> one word of codes; the block's scale byte (MXFP4, Sec. 2).
__device__ __forceinline__ void quad_encode(const float (&o)[8], float amax, uint32_t& cw, uint32_t& sbyte) {
  // shared scale: byte = max(biased_exponent(amax) - 2, 0) = clamp(floor(log2 amax) - 2) + 127
  const int ef = static_cast<int>(__float_as_uint(amax) >> 23);
  const int sb = max(ef - 2, 0);
  const float inv = __uint_as_float(static_cast<uint32_t>(254 - sb) << 23);
  float uu[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) uu[c] = o[c] * inv;
  cw = e2m1x8_pack(uu);
  sbyte = static_cast<uint32_t>(sb);
}

// ---------------------------------------------------------------------------------------------
// Stages 1+2 alone for a handful of tokens: four lanes per (token, block), the factors requested
// before the wait for the previous grid and x right after it, no shared-memory ring -- a launch of
// a few microseconds in front of the small-s GEMM, whose weight stream it releases at once
// (programmatic dependent launch).  Also clears the GEMM's split-K tickets.
struct QuantSmallParams {
  const uint16_t* x;     // bf16 bits [s x n], row stride ld
  int64_t ld;
  int32_t s;
  int32_t n;
  int32_t k;             // n / 32
  const float* left;     // [.][gr x gr], left_stride floats apart (0 = shared); NULL = identity transform
  const float* right;    // [.][gc x gc]
  int32_t left_stride;
  int32_t right_stride;
  const float* clip_lo;  // [k] or NULL
  const float* clip_hi;
  uint8_t* codes;        // [s x n/2]
  uint8_t* scales;
  int32_t sf_layout;     // BATQ_SF_ROWMAJOR / BATQ_SF_MMA
  int32_t sf_katoms;
  float* debug_out;      // [s x n] fp32 (DEBUG_OUT builds)
  uint32_t* zero_words;  // optional: n_zero_words 32-bit words set to zero
  int32_t n_zero_words;
  int32_t bf16_mid;      // != 0: both contractions of the transform store their result as bf16
};

template <bool DEBUG_OUT, int GC>
__global__ void __launch_bounds__(128) quantize_act_small_kernel(const QuantSmallParams p) {
  grid_launch_dependents();
  const int lane = threadIdx.x & 31;
  const int64_t gt = static_cast<int64_t>(blockIdx.x) * 128 + threadIdx.x;
  const int r = static_cast<int>(gt & 3);
  const int64_t item = gt >> 2;
  const bool valid = item < static_cast<int64_t>(p.s) * p.k;
  const int64_t row = valid ? item / p.k : 0;
  const int j = valid ? static_cast<int>(item - row * p.k) : 0;
  const bool xform = p.left != nullptr, clip = p.clip_lo != nullptr;
  QuadFactors<GC> f;
  quad_load_factors<GC>(valid, xform ? p.left + static_cast<int64_t>(j) * p.left_stride : nullptr,
                        xform ? p.right + static_cast<int64_t>(j) * p.right_stride : nullptr, p.clip_lo, p.clip_hi, j, r, f);
  float o[8];
  float amax;
  quad_transform_clip<GC>(p.x + row * p.ld + static_cast<int64_t>(j) * 32 + r * 8, valid, xform, clip, f, lane, o, amax,
                      p.bf16_mid != 0);
  // Past the wait inside quad_transform_clip: the grid in front of this one has finished and no
  // longer reads the codes, scales and tickets of its own call.
  if (blockIdx.x == 0)
    for (int i = threadIdx.x; i < p.n_zero_words; i += 128) p.zero_words[i] = 0u;
  if (!valid) return;
  if (DEBUG_OUT) {
    float4* dst = reinterpret_cast<float4*>(p.debug_out + row * p.n + static_cast<int64_t>(j) * 32 + r * 8);
    dst[0] = make_float4(o[0], o[1], o[2], o[3]);
    dst[1] = make_float4(o[4], o[5], o[6], o[7]);
    return;
  }
  uint32_t cw, sbyte;
  quad_encode(o, amax, cw, sbyte);
  *reinterpret_cast<uint32_t*>(p.codes + row * (p.n / 2) + static_cast<int64_t>(j) * 16 + r * 4) = cw;
  if (r != 0) return;
  if (p.sf_layout == 0) {
    p.scales[row * p.k + j] = static_cast<uint8_t>(sbyte);
  } else {
    p.scales[sf_mma_offset(row, j, p.sf_katoms)] = static_cast<uint8_t>(sbyte);
    if (j == p.k - 1)  // keep the padded blocks of this row finite
      for (int jj = p.k; jj < p.sf_katoms * 4; ++jj) p.scales[sf_mma_offset(row, jj, p.sf_katoms)] = 0;
  }
}

template <bool OUT_BF16, int GC>
__global__ void __launch_bounds__(kFusedThreads, 2)
linear_small_s_fused_kernel(const __grid_constant__ CUtensorMap tmap_w, const FusedParams p) {
  using Cfg = FusedCfg;
  extern __shared__ uint8_t fused_smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];
  __shared__ __align__(8) uint64_t x_ready_bar;
  __shared__ __align__(8) uint64_t acc_full_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  // The next grid on the stream may be scheduled at once: a kernel of this library touches nothing
  // the grid before it reads or writes until its own grid_dependency_wait().
  grid_launch_dependents();
  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const int lane = tid & 31;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(fused_smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* const x_codes = smem + Cfg::kStages * Cfg::kStageBytes;  // [step][16 rows x 128 B], 128-byte swizzle
  uint8_t* const x_sf = x_codes + Cfg::kXBytes;                     // [step][2 atoms x 512 B]

  if (tid == 0) {
    for (int i = 0; i < Cfg::kStages; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), 1);
    }
    mbar_init(smem_u32(&x_ready_bar), 4);
    mbar_init(smem_u32(&acc_full_bar), 1);
    abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_w);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  const int rt = blockIdx.x;   // 128-row tile of W
  const int sp = blockIdx.y;   // K split = rank in the cluster
  const int kt0 = static_cast<int>(static_cast<int64_t>(p.k_steps) * sp / p.splits);
  const int kt1 = static_cast<int>(static_cast<int64_t>(p.k_steps) * (sp + 1) / p.splits);
  const int n_steps = kt1 - kt0;  // 1..kFusedMaxSteps: the host chooses the splits accordingly
  bool epi_ok = false;
  uint32_t v[kFusedTok];

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (weights)
    const uint32_t smem_base = smem_u32(smem);
    const uint8_t* sfw_src = p.sfw + static_cast<int64_t>(rt) * p.katoms * 512;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    int issued = 0;
    for (int i = 0; i < n_steps; ++i) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, &abort_flag));
      if (!ok) break;
      if (elect_one()) {
        const uint32_t st = smem_base + stage * Cfg::kStageBytes;
        const uint32_t bar = smem_u32(&full_bar[stage]);
        mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
        tma_load_2d(st, &tmap_w, (kt0 + i) * kBKBytes, rt * 128, bar);
        bulk_g2s(st + Cfg::kWBytes, sfw_src + static_cast<int64_t>(kt0 + i) * 1024, 1024, bar);
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
    constexpr uint32_t idesc0 = mxf4_idesc(128, kFusedTok);
    constexpr uint32_t idesc1 = idesc0 | (2u << 29) | (2u << 4);  // scale byte pair 2 instead of 0
    const uint32_t smem_base = smem_u32(smem);
    const uint64_t w_desc0 = make_smem_desc(smem_base, 16, 1024, 2);
    const uint64_t wsf_desc0 = make_smem_desc(smem_base + Cfg::kWBytes, 0, 128, 0);
    const uint64_t x_desc0 = make_smem_desc(smem_u32(x_codes), 16, 1024, 2);
    const uint64_t xsf_desc0 = make_smem_desc(smem_u32(x_sf), 0, 128, 0);
    const uint32_t sf_tmem0 = tmem_base + kFusedTok;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&x_ready_bar), 0, &abort_flag));
    for (int i = 0; i < n_steps && ok; ++i) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&full_bar[stage]), phase, &abort_flag));
      if (!ok) break;
      tc_fence_after_sync();
      const uint64_t wdesc = w_desc0 + static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
      const uint64_t wsfd = wsf_desc0 + static_cast<uint32_t>(stage * (Cfg::kStageBytes >> 4));
      const uint64_t xdesc = x_desc0 + static_cast<uint32_t>(i * (Cfg::kXStepBytes >> 4));
      const uint64_t xsfd = xsf_desc0 + static_cast<uint32_t>(i * (Cfg::kSfBytes >> 4));
      const uint32_t sfw_col = sf_tmem0 + stage * Cfg::kSfColsPerStage;
      const uint32_t sfx_col = sfw_col + 8;
      if (elect_one()) {
        tc_cp_32x128b_warpx4(sfw_col, wsfd);
        tc_cp_32x128b_warpx4(sfw_col + 4, wsfd + 32);
        tc_cp_32x128b_warpx4(sfx_col, xsfd);
        tc_cp_32x128b_warpx4(sfx_col + 4, xsfd + 32);
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
    // ---------------------------------------------------------------- activation quantisers, then epilogue
    const int qt = tid - 64;                 // 0..127: four lanes per (token, block), 32 items per pass
    const int r = qt & 3;
    const int nb = n_steps * 8;              // blocks of this CTA's K slice
    const int total = p.s * nb;
    const bool xform = p.left != nullptr, clip = p.clip_lo != nullptr;
    for (int it0 = 0; it0 < total; it0 += 32) {  // the same trip count in every lane (shuffles inside)
      const int item = it0 + (qt >> 2);
      const bool valid = item < total;
      const int t = valid ? item / nb : 0;
      const int jj = valid ? item - t * nb : 0;
      const int j = kt0 * 8 + jj;
      const bool real = valid && j < p.k;    // blocks past the last channel: zero codes, finite scale
      QuadFactors<GC> f;
      quad_load_factors<GC>(real, xform ? p.left + static_cast<int64_t>(j) * p.left_stride : nullptr,
                            xform ? p.right + static_cast<int64_t>(j) * p.right_stride : nullptr, p.clip_lo, p.clip_hi, j, r, f);
      float o[8];
      float amax;
      quad_transform_clip<GC>(p.x + t * p.ld + static_cast<int64_t>(j) * 32 + r * 8, real, xform, clip, f, lane, o, amax);
      uint32_t cw = 0u, sbyte = 0u;
      if (real) quad_encode(o, amax, cw, sbyte);
      if (valid) {
        const int step = jj >> 3, c = jj & 7;
        *reinterpret_cast<uint32_t*>(x_codes + step * Cfg::kXStepBytes + t * 128 + ((c ^ (t & 7)) << 4) + r * 4) = cw;
        if (r == 0) x_sf[step * Cfg::kSfBytes + (c >> 2) * 512 + t * 16 + (c & 3)] = static_cast<uint8_t>(sbyte);
      }
    }
    grid_dependency_wait();  // threads without an item: these warps write y below
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&x_ready_bar));

    mbar_wait(smem_u32(&acc_full_bar), 0, &abort_flag);
    // A wait that gave up has raised abort_flag before this barrier, so the four warps agree.
    named_barrier_sync(1, 128);
    epi_ok = *static_cast<volatile int*>(&abort_flag) == 0;
    if (epi_ok) {
      tc_fence_after_sync();
      const int quad = warp & 3;  // tensor-memory lanes [32*quad, 32*quad + 32)
      tmem_ld_32x32b_x16(tmem_base + (static_cast<uint32_t>(quad * 32) << 16), v);
      tmem_ld_wait();
      tc_fence_before_sync();
      if (p.splits > 1) {
        // every MMA has completed: the activation-code region is free and takes the partial tile
        float* part = reinterpret_cast<float*>(x_codes);
        const int row = quad * 32 + lane;
#pragma unroll
        for (int t = 0; t < kFusedTok; ++t)
          if (t < p.s) part[t * 128 + row] = __uint_as_float(v[t]);
      }
    }
  }

  // The K splits of this row tile (one cluster) exchange their partial tiles.  Every thread of
  // every CTA takes both barriers, whatever happened above, so none can wait for ever.
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp >= 2 && epi_ok) {
    const int row = (warp & 3) * 32 + lane;
    const int64_t mrow = static_cast<int64_t>(rt) * 128 + row;
    if (p.splits > 1) {
      // Reduce-scatter: CTA sp adds, in rank order (deterministic), the partial sums of tokens sp,
      // sp + splits, ... -- its own from local, the others' from distributed shared memory -- and
      // writes those tokens of y.
      const uint32_t mine = smem_u32(x_codes) + row * 4;
      for (int t = sp; t < p.s; t += p.splits) {
        float part[kFusedMaxSplits];
#pragma unroll
        for (int q = 0; q < kFusedMaxSplits; ++q)
          part[q] = q < p.splits ? ld_shared_cluster_f32(map_to_cta(mine + t * 512, q)) : 0.0f;
        float acc = part[0];
#pragma unroll
        for (int q = 1; q < kFusedMaxSplits; ++q) acc += part[q];
        if (mrow < p.m) {
          if (OUT_BF16)
            reinterpret_cast<__nv_bfloat16*>(p.y)[t * p.ldy + mrow] = __float2bfloat16_rn(acc);
          else
            reinterpret_cast<float*>(p.y)[t * p.ldy + mrow] = acc;
        }
      }
    } else if (mrow < p.m) {
#pragma unroll
      for (int t = 0; t < kFusedTok; ++t) {
        if (t < p.s) {
          if (OUT_BF16)
            reinterpret_cast<__nv_bfloat16*>(p.y)[t * p.ldy + mrow] = __float2bfloat16_rn(__uint_as_float(v[t]));
          else
            reinterpret_cast<float*>(p.y)[t * p.ldy + mrow] = __uint_as_float(v[t]);
        }
      }
    }
  }
  cluster_sync_all();  // nobody leaves while its shared memory may still be read
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

}  // namespace batq
