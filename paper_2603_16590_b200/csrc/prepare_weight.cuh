// Offline weight fusion: W~ = W P^-T per 32-block of each weight row, optional
// block clip, MXFP4 quantisation, written as row-major packed codes plus scale
// bytes in the tensor-core layout.  fp64 throughout: this runs once per layer
// and is not on the timed path, so exactness beats speed.  One thread per
// (row, block).
#pragma once
#include "quantize_act.cuh"

namespace batq {

struct PrepWeightParams {
  const uint16_t* w;  // bf16 bits [m x n], row stride ld
  int64_t ld;
  int64_t m;
  int32_t n;
  int32_t k;
  const double* left;   // L' = L^-T per block: [.][16], left_stride doubles apart (0 = shared); NULL = identity
  const double* right;  // R' = R^-T: [.][64]
  int32_t left_stride;
  int32_t right_stride;
  int32_t gr, gc;        // factor sizes, gr * gc == 32 (set when left != NULL)
  const float* clip_lo;  // [m x k] or NULL
  const float* clip_hi;
  uint8_t* codes;   // [m x n/2]
  uint8_t* scales;  // BATQ_SF_MMA layout
  int32_t katoms;
};

__device__ __forceinline__ uint32_t e2m1_code_f64(double u) {
  const double a = fabs(u);
  uint32_t c;
  if (a <= 0.25) c = 0;          // tie 0 | 0.5 -> even code 0
  else if (a < 0.75) c = 1;
  else if (a <= 1.25) c = 2;     // ties 0.75 and 1.25 -> even code 2 (value 1)
  else if (a < 1.75) c = 3;
  else if (a <= 2.5) c = 4;      // ties 1.75 and 2.5 -> even code 4 (value 2)
  else if (a < 3.5) c = 5;
  else if (a <= 5.0) c = 6;      // ties 3.5 and 5 -> even code 6 (value 4)
  else c = 7;                    // saturates at 6
  return c | (signbit(u) ? 8u : 0u);
}

__global__ void __launch_bounds__(128) prepare_weight_kernel(const PrepWeightParams p) {
  const int64_t item = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (item >= p.m * p.k) return;
  const int64_t row = item / p.k;
  const int j = static_cast<int>(item - row * p.k);
  const uint16_t* src = p.w + row * p.ld + static_cast<int64_t>(j) * 32;
  // the block as V[r][c], element r*gc + c (flat arrays: the factor sizes are run-time values)
  double v[32], o[32];
  for (int e = 0; e < 32; ++e) v[e] = static_cast<double>(__uint_as_float(static_cast<uint32_t>(src[e]) << 16));
  if (p.left != nullptr) {
    const int gr = p.gr, gc = p.gc;
    const double* L = p.left + static_cast<int64_t>(j) * p.left_stride;
    const double* R = p.right + static_cast<int64_t>(j) * p.right_stride;
    double U[32];
    for (int r = 0; r < gr; ++r)
      for (int c = 0; c < gc; ++c) {
        double acc = 0.0;
        for (int cc = 0; cc < gc; ++cc) acc = fma(v[r * gc + cc], R[cc * gc + c], acc);
        U[r * gc + c] = acc;
      }
    for (int r = 0; r < gr; ++r)
      for (int c = 0; c < gc; ++c) {
        double acc = 0.0;
        for (int i = 0; i < gr; ++i) acc = fma(L[i * gr + r], U[i * gc + c], acc);
        o[r * gc + c] = acc;
      }
  } else {
    for (int e = 0; e < 32; ++e) o[e] = v[e];
  }
  double mn = o[0], mx = o[0];
  for (int e = 0; e < 32; ++e) {
    mn = fmin(mn, o[e]);
    mx = fmax(mx, o[e]);
  }
  if (p.clip_lo != nullptr) {
    const double lo = static_cast<double>(p.clip_lo[item]) * mn;
    const double hi = static_cast<double>(p.clip_hi[item]) * mx;
    for (int e = 0; e < 32; ++e) o[e] = fmin(fmax(o[e], lo), hi);
  }
  double amax = 0.0;
  for (int e = 0; e < 32; ++e) amax = fmax(amax, fabs(o[e]));
  int e = -127;
  if (amax > 0.0) {
    int ex;
    frexp(amax, &ex);  // amax = f * 2^ex, f in [0.5, 1)  =>  floor(log2 amax) = ex - 1
    e = min(max(ex - 1 - 2, -127), 127);
  }
  uint32_t cw[4];
  for (int r = 0; r < 4; ++r) {
    uint32_t w = 0;
    for (int c = 0; c < 8; ++c) w |= e2m1_code_f64(scalbn(o[r * 8 + c], -e)) << (4 * c);
    cw[r] = w;
  }
  *reinterpret_cast<uint4*>(p.codes + row * (p.n / 2) + static_cast<int64_t>(j) * 16) =
      make_uint4(cw[0], cw[1], cw[2], cw[3]);
  p.scales[sf_mma_offset(row, j, p.katoms)] = static_cast<uint8_t>(e + 127);
  if (j == p.k - 1)
    for (int jj = p.k; jj < p.katoms * 4; ++jj) p.scales[sf_mma_offset(row, jj, p.katoms)] = 0;
}

// Prepared weight -> row-major scale bytes (codes are already row-major).
__global__ void export_scales_kernel(const uint8_t* sf_mma, uint8_t* out, int64_t m, int32_t k, int32_t katoms) {
  const int64_t item = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (item >= m * k) return;
  const int64_t row = item / k;
  const int j = static_cast<int>(item - row * k);
  out[item] = sf_mma[sf_mma_offset(row, j, katoms)];
}

// Row-major scale bytes -> the layout of a prepared weight (the padding was zeroed before).
__global__ void import_scales_kernel(const uint8_t* in, uint8_t* sf_mma, int64_t m, int32_t k, int32_t katoms) {
  const int64_t item = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (item >= m * k) return;
  const int64_t row = item / k;
  const int j = static_cast<int>(item - row * k);
  sf_mma[sf_mma_offset(row, j, katoms)] = in[item];
}

}  // namespace batq
