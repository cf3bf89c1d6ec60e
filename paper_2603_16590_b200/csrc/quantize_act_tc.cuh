// Activation transform + block clip + MXFP4 quantiser with the block transform on
// the tensor cores (stages 1+2 of the path).
//
// x~ = x P_j (Eq. 1) is a dense 32 x 32 contraction per block.  The ALU version of
// this kernel (quantize_act.cuh, the Kronecker-factored form of Eq. 2) is bound by
// instruction issue, not by HBM, so here the contraction runs as tcgen05.mma
// (kind::f16, bf16 x bf16 -> fp32): A = a 128-token x 32-channel tile of X exactly
// as TMA lands it in shared memory, B = P_j^T split into three bf16 terms
// (hi + mid + lo reproduce the fp32 entries), D = 128 x 32 fp32 in tensor memory.
// The accumulator row of a token is then read by one thread, which clips (Eq. 3-4),
// derives the shared scale, rounds to E2M1 and stores 16 code bytes + 1 scale byte.
//
// Work unit: 128 tokens x 4 blocks (one 512-byte scale atom).  Warp 0 = TMA
// producer (X tiles, block-matrix images), warp 1 = MMA issuer and tensor-memory
// owner, warps 2..17 = quantiser warps (4 lane quadrants x 4 blocks), one
// (token, block) per thread; warp 18 = store warp: once the pieces of a unit have arrived in
// the staging buffer it issues the unit's TMA store and scale-atom copy.  The quantiser warps
// form two groups of eight (4 lane quadrants x 2, two blocks per thread) that take alternate
// units: the MMA issuer finishes their units half a period apart, so one group's tensor-memory
// loads and stores fall into the other group's ALU phase.
#pragma once
#include <cuda.h>

#include "ptx.cuh"
#include "quantize_act.cuh"

namespace batq {

constexpr int kQtGroups = 4;                  // blocks per unit
constexpr int kQtRows = 128;                  // tokens per unit
constexpr int kQtStages = 3;
constexpr int kQtBoxBytes = kQtRows * 128;    // one TMA box: 128 rows x 64 bf16
constexpr int kQtStageBytes = 2 * kQtBoxBytes;
constexpr int kQtTermBytes = 2048;            // one bf16 term of one 32 x 32 block matrix
constexpr int kQtImageBytes = 3 * kQtTermBytes;            // per block
constexpr int kQtStripImageBytes = kQtGroups * kQtImageBytes;  // 24 KiB
constexpr int kQtQuantWarps = 16;
constexpr int kQtThreads = (3 + kQtQuantWarps) * 32;  // + TMA producer, MMA issuer, store warp
constexpr int kQtCodeTileBytes = kQtRows * kQtGroups * 16;  // 4-bit codes of one unit: 128 rows x 64 bytes
constexpr int kQtCodeTileBytes8 = 2 * kQtCodeTileBytes;     // 8-bit codes: 128 rows x 128 bytes
constexpr int kQtOutBufs = 4;   // staging buffers between the quantiser warps and the store warp
constexpr int kQtDBufs = 4;     // accumulator buffers in tensor memory: two per group of quantiser warps
constexpr int kQtStagingBytes = kQtOutBufs * (kQtCodeTileBytes8 + 512);  // code tiles (sized for 8-bit), scale atoms
constexpr int kQtSmemBytes = kQtStages * kQtStageBytes + 2 * kQtStripImageBytes + kQtStagingBytes + 1024;
constexpr int kQtTmemCols = kQtDBufs * kQtGroups * 32;  // 4 buffers x 4 blocks x 32 columns = all 512

struct QuantTcParams {
  int64_t s;
  int32_t n;
  int32_t k;             // n / 32
  int32_t n_strips;      // ceil(k / 4)
  int64_t n_row_tiles;   // ceil(s / 128)
  int64_t n_units;       // n_strips * n_row_tiles
  const uint8_t* pimg;   // [k][3 terms][2048]: P_j^T as bf16 in the MMA's no-swizzle K-major layout
  const float* clip_lo;  // [k] or NULL
  const float* clip_hi;
  uint8_t* scales;
  int32_t sf_layout;
  int32_t sf_katoms;
  float* debug_out;      // [s x n] fp32 (DEBUG_OUT builds)
};

// Instruction descriptor of tcgen05.mma kind::f16: [4,6) D format (1 = F32), [7,10) A format
// (1 = BF16), [10,13) B format, [15]/[16] A/B major (0 = K), [17,23) N >> 3, [24,29) M >> 4.
__host__ __device__ constexpr uint32_t f16_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ float fmin3(float a, float b, float c) {
  float d;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// (a, b) * s with one packed instruction (the products are the same fp32 values as two scalar
// multiplications give: s is a power of two here).
__device__ __forceinline__ void mul2(float a, float b, float s, float& ra, float& rb) {
  asm("{\n\t.reg .b64 v, w, r;\n\t"
      "mov.b64 v, {%2, %3};\n\t"
      "mov.b64 w, {%4, %4};\n\t"
      "mul.rn.f32x2 r, v, w;\n\t"
      "mov.b64 {%0, %1}, r;\n\t}"
      : "=f"(ra), "=f"(rb)
      : "f"(a), "f"(b), "f"(s));
}

// Four floats -> four E4M3 bytes (round to nearest even, saturating at +-448), first value in byte 0.
__device__ __forceinline__ uint32_t e4m3x4_pack(float a, float b, float c, float d) {
  uint32_t w;
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
      "mov.b32 %0, {lo, hi};\n\t}"
      : "=r"(w)
      : "f"(a), "f"(b), "f"(c), "f"(d));
  return w;
}

// FP8 = false: MXFP4 (E2M1 codes, two per byte).  FP8 = true: MXFP8 (E4M3 codes, Sec. 2), one byte per
// element, shared scale e = floor(log2 amax) - 8.
template <bool CLIP, bool DEBUG_OUT, bool FP8 = false>
__global__ void __launch_bounds__(kQtThreads, 1)
quantize_act_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_codes,
                       const QuantTcParams p) {
  extern __shared__ uint8_t qt_smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * kQtStages + 4 + 2 * kQtDBufs + 2 * kQtOutBufs];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  uint64_t* const x_full = bars;                     // [kQtStages]
  uint64_t* const x_empty = bars + kQtStages;        // [kQtStages]
  uint64_t* const p_full = bars + 2 * kQtStages;     // [2]
  uint64_t* const p_empty = p_full + 2;              // [2]
  uint64_t* const d_full = p_full + 4;               // [kQtDBufs]
  uint64_t* const d_empty = d_full + kQtDBufs;       // [kQtDBufs]
  uint64_t* const t_full = d_empty + kQtDBufs;       // [kQtOutBufs] staging tile complete (the 8 warps of a group)
  uint64_t* const t_empty = t_full + kQtOutBufs;     // [kQtOutBufs] staging tile read out by its stores

  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const int lane = tid & 31;
  // A kernel launched as a programmatic dependent of this one (the GEMM of the same layer) may
  // take over each SM as soon as this grid's CTA there has finished; it still waits for the whole
  // grid before it reads the codes and scales written here.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(qt_smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* const x_smem = smem;                                             // kQtStages x 32 KiB
  uint8_t* const img_smem = smem + kQtStages * kQtStageBytes;               // 2 x 24 KiB
  uint8_t* const staging = img_smem + 2 * kQtStripImageBytes;               // 1024-aligned: code tiles, scale atoms

  if (tid == 0) {
    for (int i = 0; i < kQtStages; ++i) {
      mbar_init(smem_u32(&x_full[i]), 1);
      mbar_init(smem_u32(&x_empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&p_full[i]), 1);
      mbar_init(smem_u32(&p_empty[i]), 1);
    }
    for (int i = 0; i < kQtDBufs; ++i) {
      mbar_init(smem_u32(&d_full[i]), 1);
      mbar_init(smem_u32(&d_empty[i]), kQtQuantWarps / 2);
    }
    for (int i = 0; i < kQtOutBufs; ++i) {
      mbar_init(smem_u32(&t_full[i]), kQtQuantWarps / 2);
      mbar_init(smem_u32(&t_empty[i]), 1);
    }
    abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_x);
    tma_prefetch_desc(&tmap_codes);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), kQtTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  // contiguous range of units for this CTA; unit u = strip * n_row_tiles + row_tile
  const int64_t u0 = p.n_units * blockIdx.x / gridDim.x;
  const int64_t u1 = p.n_units * (blockIdx.x + 1) / gridDim.x;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    int stage = 0;
    uint32_t phase = 0;
    int64_t cur_strip = -1;
    int n_img = 0;  // block-matrix images loaded so far
    bool ok = true;
    int issued = 0;
    bool waited = false;
    for (int64_t u = u0; u < u1 && ok; ++u) {
      const int64_t strip = u / p.n_row_tiles;
      const int row0 = static_cast<int>(u - strip * p.n_row_tiles) * kQtRows;
      if (strip != cur_strip) {
        cur_strip = strip;
        const int pb = n_img & 1;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&p_empty[pb]), ((n_img >> 1) & 1) ^ 1u, &abort_flag));
        if (!ok) break;
        const int j0 = static_cast<int>(strip) * kQtGroups;
        const int ng = min(kQtGroups, p.k - j0);
        if (elect_one()) {
          mbar_arrive_expect_tx(smem_u32(&p_full[pb]), static_cast<uint32_t>(ng) * kQtImageBytes);
          bulk_g2s(smem_u32(img_smem + pb * kQtStripImageBytes), p.pimg + static_cast<int64_t>(j0) * kQtImageBytes,
                   static_cast<uint32_t>(ng) * kQtImageBytes, smem_u32(&p_full[pb]));
        }
        ++n_img;
      }
      if (!waited) {
        // The block-matrix image above is the transform's own constant data; X may come from the
        // kernel before this one, which this kernel may have been launched as a programmatic
        // dependent of: wait for it here (nothing is written before data has flowed through).
        grid_dependency_wait();
        waited = true;
      }
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&x_empty[stage]), phase ^ 1u, &abort_flag));
      if (!ok) break;
      if (elect_one()) {
        const uint32_t bar = smem_u32(&x_full[stage]);
        const uint32_t dst = smem_u32(x_smem + stage * kQtStageBytes);
        const int col0 = static_cast<int>(strip) * (kQtGroups * 32);
        mbar_arrive_expect_tx(bar, kQtStageBytes);
        tma_load_2d(dst, &tmap_x, col0, row0, bar);
        tma_load_2d(dst + kQtBoxBytes, &tmap_x, col0 + 64, row0, bar);
      }
      ++issued;
      if (++stage == kQtStages) { stage = 0; phase ^= 1u; }
    }
    if (!ok && lane == 0) {
      const int pending = min(issued, kQtStages);
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = kQtStages - 1; phase ^= 1u; }
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&x_full[stage]), phase) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    constexpr uint32_t idesc = f16_idesc_bf16(kQtRows, 32);
    const uint64_t a_desc0 = make_smem_desc(smem_u32(x_smem), 16, 1024, 2);   // 128-byte swizzle, K-major
    const uint64_t b_desc0 = make_smem_desc(smem_u32(img_smem), 128, 512, 0); // no swizzle: LBO 128 (K), SBO 512 (N)
    int stage = 0;
    uint32_t phase = 0;
    int64_t cur_strip = -1;
    int n_img = 0;
    int it = 0;
    bool ok = true;
    for (int64_t u = u0; u < u1 && ok; ++u, ++it) {
      const int64_t strip = u / p.n_row_tiles;
      if (strip != cur_strip) {
        if (cur_strip >= 0 && elect_one()) tc_commit(smem_u32(&p_empty[(n_img - 1) & 1]));  // old image no longer read
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
      const int ng = min(kQtGroups, p.k - static_cast<int>(strip) * kQtGroups);
      const uint64_t a_stage = a_desc0 + static_cast<uint32_t>((stage * kQtStageBytes) >> 4);
      const uint64_t b_img = b_desc0 + static_cast<uint32_t>((pb * kQtStripImageBytes) >> 4);
      const uint32_t d0 = tmem_base + buf * (kQtGroups * 32);
      if (elect_one()) {
#pragma unroll
        for (int g = 0; g < kQtGroups; ++g) {
          if (g < ng) {
            // block g lives in box g / 2 at byte offset (g % 2) * 64 of each 128-byte row
            const uint64_t a_g = a_stage + static_cast<uint32_t>(((g >> 1) * kQtBoxBytes + (g & 1) * 64) >> 4);
            const uint64_t b_g = b_img + static_cast<uint32_t>((g * kQtImageBytes) >> 4);
#pragma unroll
            for (int t = 2; t >= 0; --t)  // smallest term first
#pragma unroll
              for (int kk = 0; kk < 2; ++kk)
                tc_mma_f16(d0 + g * 32, a_g + 2 * kk, b_g + static_cast<uint32_t>((t * kQtTermBytes + kk * 256) >> 4),
                           idesc, (t == 2 && kk == 0) ? 0u : 1u);
          }
        }
        tc_commit(smem_u32(&x_empty[stage]));
        tc_commit(smem_u32(&d_full[buf]));
      }
      if (++stage == kQtStages) { stage = 0; phase ^= 1u; }
    }
    __syncwarp();
  } else if (warp == 2 + kQtQuantWarps) {
    // ---------------------------------------------------------------- store warp
    if (!DEBUG_OUT && lane == 0) {
      int it = 0;
      for (int64_t u = u0; u < u1; ++u, ++it) {
        const int64_t strip = u / p.n_row_tiles;
        const int64_t row_tile = u - strip * p.n_row_tiles;
        const int sb = it % kQtOutBufs;
        if (!mbar_wait(smem_u32(&t_full[sb]), static_cast<uint32_t>(it / kQtOutBufs) & 1u, &abort_flag)) break;
        tma_store_2d(&tmap_codes, static_cast<int>(strip) * (kQtGroups * (FP8 ? 32 : 16)),
                     static_cast<int>(row_tile) * kQtRows, smem_u32(staging + sb * kQtCodeTileBytes8));
        if (p.sf_layout != 0)
          bulk_s2g(p.scales + (row_tile * p.sf_katoms + strip) * 512,
                   smem_u32(staging + kQtOutBufs * kQtCodeTileBytes8 + sb * 512), 512);
        bulk_commit_group();
        if (it > 0) {  // the stores of the unit before this one have read their buffer: hand it back
          bulk_wait_group_read<1>();
          mbar_arrive(smem_u32(&t_empty[(it - 1) % kQtOutBufs]));
        }
      }
      bulk_wait_group<0>();  // all stores complete before the CTA exits
    }
  } else {
    // ---------------------------------------------------------------- quantiser warps
    const int qw = warp - 2;            // 0..15
    const int quad = warp & 3;          // tensor-memory lanes [32 quad, 32 quad + 32)
    const int grp = qw >> 3;            // takes the units of this CTA with it % 2 == grp
    const int half = (qw & 7) >> 2;     // blocks 2 half and 2 half + 1 of the unit
    for (int it = grp; u0 + it < u1; it += 2) {
      const int64_t u = u0 + it;
      const int64_t strip = u / p.n_row_tiles;
      const int64_t row_tile = u - strip * p.n_row_tiles;
      const int buf = it & (kQtDBufs - 1);
      bool ok = mbar_wait(smem_u32(&d_full[buf]), (it >> 2) & 1u, &abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      // Staging buffer sb was last used by unit it - kQtOutBufs; the store warp hands it back once
      // that unit's stores have read it.
      const int sb = it % kQtOutBufs;
      if (!DEBUG_OUT && it >= kQtOutBufs) {
        ok = mbar_wait(smem_u32(&t_empty[sb]), static_cast<uint32_t>(it / kQtOutBufs - 1) & 1u, &abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
      }
      const int64_t row = row_tile * kQtRows + quad * 32 + lane;
#pragma unroll 1
     for (int e = 0; e < 2; ++e) {
      const int g = 2 * half + e;
      const int j = static_cast<int>(strip) * kQtGroups + g;
      const uint32_t taddr = tmem_base + buf * (kQtGroups * 32) + g * 32 + (static_cast<uint32_t>(quad * 32) << 16);
      uint32_t v[32];
      tmem_ld_32x32b_x32(taddr, v);
      tmem_ld_wait();
      if (e == 1) {
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&d_empty[buf]));  // both accumulator rows have been read
      }

      float o[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(v[i]);
      // four independent reduction chains
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
        const int jc = min(j, p.k - 1);
        const float lo = __ldg(p.clip_lo + jc) * mn;
        const float hi = __ldg(p.clip_hi + jc) * mx;
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = fminf(fmaxf(o[i], lo), hi);
        amax = fmaxf(fabsf(fminf(fmaxf(mn, lo), hi)), fabsf(fminf(fmaxf(mx, lo), hi)));
      } else {
        amax = fmaxf(fabsf(mn), fabsf(mx));
      }
      if (DEBUG_OUT) {
        if (row < p.s && j < p.k) {
          float4* dst = reinterpret_cast<float4*>(p.debug_out + row * p.n + static_cast<int64_t>(j) * 32);
#pragma unroll
          for (int q = 0; q < 8; ++q) dst[q] = make_float4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
        continue;
      }
      // shared scale: byte = max(biased_exponent(amax) - emax, 0), emax = 2 (E2M1) or 8 (E4M3)
      const int ef = static_cast<int>(__float_as_uint(amax) >> 23);
      const int sbyte = max(ef - (FP8 ? 8 : 2), 0);
      const float inv = __uint_as_float(static_cast<uint32_t>(254 - sbyte) << 23);
      // Codes and scale bytes of the whole unit meet in shared memory (128 rows x 64 or 128 bytes of
      // codes, one 512-byte scale atom) and leave as one TMA store and one bulk copy: full 32-byte
      // sectors instead of 16-byte and 1-byte pieces.
      const int trow = quad * 32 + lane;
      if (FP8) {
        uint8_t* tile = staging + sb * kQtCodeTileBytes8 + trow * 128;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t cw[4];
#pragma unroll
          for (int r = 0; r < 4; ++r)
            cw[r] = e4m3x4_pack(o[16 * h + 4 * r] * inv, o[16 * h + 4 * r + 1] * inv, o[16 * h + 4 * r + 2] * inv,
                                o[16 * h + 4 * r + 3] * inv);
          // 128-byte swizzle: 16-byte chunk index XOR (row & 7)
          *reinterpret_cast<uint4*>(tile + (((2 * g + h) ^ (trow & 7)) << 4)) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
        }
      } else {
        uint32_t cw[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          float uu[8];
#pragma unroll
          for (int c = 0; c < 8; c += 2) mul2(o[8 * r + c], o[8 * r + c + 1], inv, uu[c], uu[c + 1]);
          cw[r] = e2m1x8_pack(uu);
        }
        // 64-byte swizzle: 16-byte chunk index XOR ((row / 2) & 3)
        *reinterpret_cast<uint4*>(staging + sb * kQtCodeTileBytes8 + trow * 64 + ((g ^ ((trow >> 1) & 3)) << 4)) =
            make_uint4(cw[0], cw[1], cw[2], cw[3]);
      }
      const uint8_t sbv = static_cast<uint8_t>(j < p.k ? sbyte : 0);
      if (p.sf_layout == 0) {
        if (row < p.s && j < p.k) p.scales[row * p.k + j] = sbv;
      } else {
        staging[kQtOutBufs * kQtCodeTileBytes8 + sb * 512 + lane * 16 + quad * 4 + g] = sbv;
      }
     }  // the two blocks of this thread
      if (!DEBUG_OUT) {
        fence_proxy_async_smem();   // the staging writes become visible to the TMA store
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&t_full[sb]));
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kQtTmemCols);
  }
}

}  // namespace batq
