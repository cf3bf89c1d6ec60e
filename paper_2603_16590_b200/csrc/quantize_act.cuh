// Fused activation transform + block clip + MXFP4 quantiser (stages 1+2).
//
// Per (row, 32-channel block): V~ = L^T V R (the factored form of x P_j,
// Eq. 1-2 and Algorithm 1), clip to [c_lo*min, c_hi*max] (Eq. 3-4), shared
// scale e = floor(log2 amax) - 2, E2M1 round-to-nearest-even (Sec. 2).
//
// Layout of the work.  One "item" is one block of one row: 64 bytes in, 16
// bytes of codes + 1 scale byte out.  A CTA owns a contiguous range of units;
// a unit is a tile of kItems items = (kItems / gs) rows x gs consecutive blocks
// (a "strip" of columns), so every consumer thread keeps the same block -- and
// its two factor matrices in registers -- while the CTA walks down the rows.
// A producer warp streams tiles into a shared-memory ring with 1-D bulk copies
// (one per row); eight consumer warps transform, clip and quantise them.
#pragma once
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace batq {

constexpr int kQaConsumers = 256;            // items per tile, one per consumer thread
constexpr int kQaThreads = kQaConsumers + 32;  // + producer warp
constexpr int kQaStages = 8;
constexpr int kQaStageBytes = kQaConsumers * 64;
constexpr int kQaSmemBytes = kQaStages * kQaStageBytes + 1024;

struct QuantActParams {
  const uint16_t* x;   // bf16 bits, [s x n], row stride ld
  int64_t ld;
  int64_t s;
  int32_t n;
  int32_t k;             // n / 32
  int32_t gs;            // blocks per strip: power of two <= 32 that divides k
  int32_t rows_per_tile; // kQaConsumers / gs
  int64_t n_row_tiles;
  int64_t n_units;       // (k / gs) * n_row_tiles
  const float* left;     // [.][16], left_stride floats apart (0 = shared)
  const float* right;    // [.][64]
  int32_t left_stride;
  int32_t right_stride;
  const float* clip_lo;  // [k], or [s x k] with clip_row_stride = k
  const float* clip_hi;
  int64_t clip_row_stride;
  uint8_t* codes;        // [s x n/2]
  uint8_t* scales;
  int32_t sf_layout;     // BATQ_SF_ROWMAJOR / BATQ_SF_MMA
  int32_t sf_katoms;     // KA = 2*ceil(k/8), atoms per 128-row tile
  float* debug_out;      // [s x n] fp32 when the kernel is built with DEBUG_OUT
  uint32_t* zero_words;  // optional: n_zero_words 32-bit words set to zero (tickets of the kernel that follows)
  int32_t n_zero_words;
  int32_t bf16_mid;      // != 0: V R and L^T (V R) are rounded to bf16, as a BF16 implementation of Algorithm 1 stores them
};

// fp32 -> nearest bf16 value (ties to even), as fp32.
__device__ __forceinline__ float round_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

// Two floats -> one byte holding two E2M1 codes (hi in bits 4-7, lo in bits 0-3),
// four such bytes -> one 32-bit word (byte 0 = first pair).
__device__ __forceinline__ uint32_t e2m1x8_pack(const float (&u)[8]) {
  uint32_t w;
  asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
      : "=r"(w)
      : "f"(u[0]), "f"(u[1]), "f"(u[2]), "f"(u[3]), "f"(u[4]), "f"(u[5]), "f"(u[6]), "f"(u[7]));
  return w;
}

__device__ __forceinline__ int64_t sf_mma_offset(int64_t row, int32_t j, int32_t katoms) {
  return ((row >> 7) * katoms + (j >> 2)) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (j & 3);
}

template <bool XFORM, bool CLIP, bool DEBUG_OUT>
__global__ void __launch_bounds__(kQaThreads, 1) quantize_act_kernel(const QuantActParams p) {
  extern __shared__ __align__(128) uint8_t qa_smem[];
  __shared__ __align__(8) uint64_t full_bar[kQaStages];
  __shared__ __align__(8) uint64_t empty_bar[kQaStages];
  __shared__ int abort_flag;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  // A kernel launched as a programmatic dependent of this one may start its own prologue now;
  // it still waits for this grid to finish before it reads anything written here.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (p.n_zero_words > 0 && blockIdx.x == 0)
    for (int i = tid; i < p.n_zero_words; i += kQaThreads) p.zero_words[i] = 0u;
  // 128-byte aligned base of the ring
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(qa_smem) + 127) & ~uintptr_t(127));

  if (tid == 0) {
    for (int i = 0; i < kQaStages; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), kQaConsumers / 32);
    }
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  const int64_t u0 = p.n_units * blockIdx.x / gridDim.x;
  const int64_t u1 = p.n_units * (blockIdx.x + 1) / gridDim.x;
  const uint32_t row_bytes = static_cast<uint32_t>(p.gs) * 64u;

  if (warp == kQaConsumers / 32) {
    // ------------------------------------------------------------ producer warp
    int stage = 0;
    uint32_t phase = 0;
    int64_t issued = 0;
    bool ok = true;
    for (int64_t u = u0; u < u1 && ok; ++u) {
      const int64_t strip = u / p.n_row_tiles;
      const int64_t row0 = (u - strip * p.n_row_tiles) * p.rows_per_tile;
      const int nrows = static_cast<int>(min(static_cast<int64_t>(p.rows_per_tile), p.s - row0));
      ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, &abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      const uint32_t bar = smem_u32(&full_bar[stage]);
      if (lane == 0) mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nrows) * row_bytes);
      __syncwarp();
      const uint32_t dst = smem_u32(ring + stage * kQaStageBytes);
      const uint16_t* src = p.x + row0 * p.ld + strip * (p.gs * 32);
      for (int r = lane; r < nrows; r += 32) bulk_g2s(dst + r * row_bytes, src + r * p.ld, row_bytes, bar);
      ++issued;
      if (++stage == kQaStages) { stage = 0; phase ^= 1u; }
    }
    if (!ok) {
      // Given up: let the copies already in flight land before the CTA exits.
      const int pending = issued < kQaStages ? static_cast<int>(issued) : kQaStages;
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = kQaStages - 1; phase ^= 1u; }
        const uint32_t bar = smem_u32(&full_bar[stage]);
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(bar, phase) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else {
    // ------------------------------------------------------------ consumer warps
    const int rot = XFORM ? ((lane >> 1) & 3) : 0;  // chunk read order, avoids bank conflicts
    const int g_in_strip = tid & (p.gs - 1);
    const int row_in_tile = tid / p.gs;
    float R[64];
    float Lr[16];  // Lr[i][r'] = L[(i + rot) & 3][r']: rows permuted like the chunks
    int64_t cur_strip = -1;
    int j = 0;
    int stage = 0;
    uint32_t phase = 0;
    for (int64_t u = u0; u < u1; ++u) {
      const int64_t strip = u / p.n_row_tiles;
      const int64_t row0 = (u - strip * p.n_row_tiles) * p.rows_per_tile;
      if (strip != cur_strip) {
        cur_strip = strip;
        j = static_cast<int>(strip) * p.gs + g_in_strip;
        if (XFORM) {
          const float4* rp = reinterpret_cast<const float4*>(p.right + static_cast<int64_t>(j) * p.right_stride);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float4 t = __ldg(rp + i);
            R[4 * i + 0] = t.x; R[4 * i + 1] = t.y; R[4 * i + 2] = t.z; R[4 * i + 3] = t.w;
          }
          const float* lp = p.left + static_cast<int64_t>(j) * p.left_stride;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(lp) + ((i + rot) & 3));
            Lr[4 * i + 0] = t.x; Lr[4 * i + 1] = t.y; Lr[4 * i + 2] = t.z; Lr[4 * i + 3] = t.w;
          }
        }
      }
      bool ok = mbar_wait(smem_u32(&full_bar[stage]), phase, &abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      const uint4* src = reinterpret_cast<const uint4*>(ring + stage * kQaStageBytes + tid * 64);
      uint4 q[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) q[i] = src[(i + rot) & 3];
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty_bar[stage]));
      if (++stage == kQaStages) { stage = 0; phase ^= 1u; }

      const int64_t row = row0 + row_in_tile;
      if (row >= p.s) continue;

      // bf16 -> fp32; v[i][c] is row (i + rot) & 3 of the block matrix V
      float v[4][8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t w[4] = {q[i].x, q[i].y, q[i].z, q[i].w};
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          v[i][2 * h] = __uint_as_float(w[h] << 16);
          v[i][2 * h + 1] = __uint_as_float(w[h] & 0xFFFF0000u);
        }
      }
      float o[4][8];  // XFORM: natural row order r'; else same (rot == 0)
      if (XFORM) {
        float U[4][8];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float acc = v[i][0] * R[c];
#pragma unroll
            for (int cc = 1; cc < 8; ++cc) acc = fmaf(v[i][cc], R[cc * 8 + c], acc);
            U[i][c] = p.bf16_mid ? round_bf16(acc) : acc;
          }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float acc = Lr[r] * U[0][c];
#pragma unroll
            for (int i = 1; i < 4; ++i) acc = fmaf(Lr[4 * i + r], U[i][c], acc);
            o[r][c] = p.bf16_mid ? round_bf16(acc) : acc;
          }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int c = 0; c < 8; ++c) o[i][c] = v[i][c];
      }

      float mn = o[0][0], mx = o[0][0];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          mn = fminf(mn, o[r][c]);
          mx = fmaxf(mx, o[r][c]);
        }
      float amax;
      if (CLIP) {
        const int64_t ci = row * p.clip_row_stride + j;
        const float lo = __ldg(p.clip_lo + ci) * mn;
        const float hi = __ldg(p.clip_hi + ci) * mx;
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 8; ++c) o[r][c] = fminf(fmaxf(o[r][c], lo), hi);
        // the clamp is monotone, so the extreme magnitudes come from the extreme values
        amax = fmaxf(fabsf(fminf(fmaxf(mn, lo), hi)), fabsf(fminf(fmaxf(mx, lo), hi)));
      } else {
        amax = fmaxf(fabsf(mn), fabsf(mx));
      }

      if (DEBUG_OUT) {
        float4* dst = reinterpret_cast<float4*>(p.debug_out + row * p.n + static_cast<int64_t>(j) * 32);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          dst[2 * r] = make_float4(o[r][0], o[r][1], o[r][2], o[r][3]);
          dst[2 * r + 1] = make_float4(o[r][4], o[r][5], o[r][6], o[r][7]);
        }
        continue;
      }

      // shared scale: byte = max(biased_exponent(amax) - 2, 0) = clamp(floor(log2 amax) - 2) + 127
      const int ef = static_cast<int>(__float_as_uint(amax) >> 23);
      const int sbyte = max(ef - 2, 0);
      const float inv = __uint_as_float(static_cast<uint32_t>(254 - sbyte) << 23);  // 2^-(e)
      uint32_t cw[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        float uu[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) uu[c] = o[r][c] * inv;
        cw[r] = e2m1x8_pack(uu);
      }
      *reinterpret_cast<uint4*>(p.codes + row * (p.n / 2) + static_cast<int64_t>(j) * 16) =
          make_uint4(cw[0], cw[1], cw[2], cw[3]);
      if (p.sf_layout == 0) {
        p.scales[row * p.k + j] = static_cast<uint8_t>(sbyte);
      } else {
        p.scales[sf_mma_offset(row, j, p.sf_katoms)] = static_cast<uint8_t>(sbyte);
        if (j == p.k - 1) {  // keep the padded blocks of this row finite
          for (int jj = p.k; jj < p.sf_katoms * 4; ++jj) p.scales[sf_mma_offset(row, jj, p.sf_katoms)] = 0;
        }
      }
    }
  }
}

}  // namespace batq
