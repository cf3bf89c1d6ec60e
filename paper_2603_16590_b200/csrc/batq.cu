// C-ABI of the batq library: host-side validation, handles and kernel launches.
// The whole library is this one translation unit.
#include "batq_debug.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <climits>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "gemm_mxfp4.cuh"
#include "gemm_mxfp4_pair.cuh"
#include "gemm_mxfp4_wide.cuh"
#include "gemm_small_s.cuh"
#include "gemm_w4a8.cuh"
#include "gemm_w4a8_pair.cuh"
#include "gemm_w4a8_wide.cuh"
#include "linear_prefill_fused.cuh"
#include "linear_small_s_fused.cuh"
#include "mma_peak.cuh"
#include "prepare_weight.cuh"
#include "quantize_act.cuh"
#include "quantize_act_tc.cuh"

using namespace batq;

// ------------------------------------------------------------------------------------
// handles
// ------------------------------------------------------------------------------------
struct batq_transform {
  int device;
  int32_t n, k, gr, gc;
  int32_t left_stride, right_stride;  // 0 = shared
  bool has_clip;
  bool bf16_mid;                      // the transform's two contractions store bf16 (emulation of a BF16 implementation)
  std::vector<float> left, right;     // host copies (for the inverse)
  float* d_left;                      // device copies (for the kernels)
  float* d_right;
  float* d_clip_lo;
  float* d_clip_hi;
  uint8_t* d_pimg;                    // [k][3][2048]: dense P_j^T as three bf16 terms, tensor-core operand layout
  CUtensorMap tmap_pimg;              // the same bytes as [k][3 terms][2 halves of 16 rows][1024]: boxes of 4 blocks x 3 terms x one half
};

struct batq_weight {
  int device;
  int64_t m, n;
  int32_t k, katoms;
  int32_t sm_count;  // of the device the weight lives on (sizes the small-s split-K scratch)
  uint8_t* codes;   // [m x n/2]
  uint8_t* scales;  // BATQ_SF_MMA
  CUtensorMap tmap_b256;  // boxes of 256 / 192 / 128 weight rows x 128 bytes
  CUtensorMap tmap_b192;
  CUtensorMap tmap_b128;
  CUtensorMap tmap_b64;
  CUtensorMap tmap_b32;   // boxes of 32 weight rows: the CTA-pair kernel composes its half tiles from them
  CUtensorMap tmap_sf;    // scale atoms: [row tiles x KA] rows of 512 bytes, boxes of two atoms
  // CTA-pair schedules already worked out for this weight, by token count (host only)
  struct SchedEntry { int64_t s; int force_bn; bool wide, a8; double cost; int32_t n_cols, n_segs, pairs; batq::PairSeg seg[batq::kPairMaxSegs]; };
  mutable std::mutex sched_mutex;
  mutable std::vector<SchedEntry> sched_cache;
  bool has_u4;            // n % 128 == 0: the maps below exist (W4A8 GEMM)
  CUtensorMap tmap_u4_128;  // packed 4-bit codes widened to 8-bit containers by the TMA unit: boxes of
  CUtensorMap tmap_u4_256;  // 128 elements x 128 / 256 weight rows
  CUtensorMap tmap_u4_32;   // 128 elements x 32 weight rows: the W4A8 CTA-pair kernel composes its half tiles from them
  CUtensorMap tmap_sf1;     // scale atoms, boxes of one atom = the 4 blocks of one 128-element K step
};

// Scratch for batq_linear_w4a4_noalloc: part of the library image, one copy per GPU.
// In host code this name is only a handle for cudaGetSymbolAddress, never a pointer
// a kernel may be given.
static __device__ __align__(256) uint8_t g_static_workspace[BATQ_STATIC_WORKSPACE_BYTES];

namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int32_t katoms_of(int64_t k) { return static_cast<int32_t>(2 * ((k + 7) / 8)); }

constexpr int kMaxDevices = 64;

struct DeviceInfo {
  bool ready = false;
  int sm_count = 0;
  int cc_major = 0;
  uint8_t* static_ws = nullptr;  // device address of g_static_workspace on this device, 1024-aligned
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_mutex;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;

template <typename K>
cudaError_t set_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

// Per-device one-time setup: properties, opt-in shared memory sizes, driver entry point.
batq_status device_setup(int* device_out, const DeviceInfo** info_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BATQ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceInfo& d = g_dev[dev];
  if (!d.ready) {
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return BATQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return BATQ_ERR_CUDA;
    if (d.cc_major != 10) return BATQ_ERR_UNSUPPORTED;
    cudaError_t e = cudaSuccess;
    e = e ? e : set_smem(quantize_act_kernel<true, true, false>, kQaSmemBytes);
    e = e ? e : set_smem(quantize_act_kernel<true, false, false>, kQaSmemBytes);
    e = e ? e : set_smem(quantize_act_kernel<false, false, false>, kQaSmemBytes);
    e = e ? e : set_smem(quantize_act_kernel<true, true, true>, kQaSmemBytes);
    e = e ? e : set_smem(quantize_act_kernel<true, false, true>, kQaSmemBytes);
    e = e ? e : set_smem(quantize_act_kernel<false, false, true>, kQaSmemBytes);
    e = e ? e : set_smem(quantize_act_tc_kernel<true, false>, kQtSmemBytes);
    e = e ? e : set_smem(quantize_act_tc_kernel<false, false>, kQtSmemBytes);
    e = e ? e : set_smem(quantize_act_tc_kernel<true, true>, kQtSmemBytes);
    e = e ? e : set_smem(quantize_act_tc_kernel<false, true>, kQtSmemBytes);
    e = e ? e : set_smem(quantize_act_tc_kernel<true, false, true>, kQtSmemBytes);
    e = e ? e : set_smem(quantize_act_tc_kernel<false, false, true>, kQtSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<256, false>, GemmCfg<256>::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<256, true>, GemmCfg<256>::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<192, false>, GemmCfg<192>::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<192, true>, GemmCfg<192>::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<128, false>, GemmCfg<128>::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<128, true>, GemmCfg<128>::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<64, false>, GemmCfg<64>::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_kernel<64, true>, GemmCfg<64>::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_kernel<128, false>, W4A8Cfg<128>::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_kernel<128, true>, W4A8Cfg<128>::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_kernel<256, false>, W4A8Cfg<256>::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_kernel<256, true>, W4A8Cfg<256>::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_pair_kernel<false>, A8PairCfg::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_pair_kernel<true>, A8PairCfg::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_wide_kernel<false>, A8WideCfg::kSmemBytes);
    e = e ? e : set_smem(gemm_w4a8_wide_kernel<true>, A8WideCfg::kSmemBytes);
    e = e ? e : set_smem(mma_peak_kernel<false, 0>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(mma_peak_kernel<true, 0>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(mma_peak_kernel<false, 1>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(mma_peak_kernel<true, 1>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(mma_peak_kernel<false, 2>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(mma_peak_kernel<true, 2>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(mma_peak_kernel<false, 3>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(mma_peak_kernel<true, 3>, kPeakSmemBytesLoads);
    e = e ? e : set_smem(gemm_mxfp4_pair_kernel<false>, PairCfg::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_pair_kernel<true>, PairCfg::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_wide_kernel<false>, WideCfg::kSmemBytes);
    e = e ? e : set_smem(gemm_mxfp4_wide_kernel<true>, WideCfg::kSmemBytes);
    e = e ? e : set_smem(linear_prefill_fused_kernel<false, false>, kPfSmemBytes);
    e = e ? e : set_smem(linear_prefill_fused_kernel<false, true>, kPfSmemBytes);
    e = e ? e : set_smem(linear_prefill_fused_kernel<true, false>, kPfSmemBytes);
    e = e ? e : set_smem(linear_prefill_fused_kernel<true, true>, kPfSmemBytes);
    e = e ? e : set_smem(linear_small_s_fused_kernel<false, 8>, FusedCfg::kSmemBytes);
    e = e ? e : set_smem(linear_small_s_fused_kernel<true, 8>, FusedCfg::kSmemBytes);
    e = e ? e : set_smem(linear_small_s_fused_kernel<false, 4>, FusedCfg::kSmemBytes);
    e = e ? e : set_smem(linear_small_s_fused_kernel<true, 4>, FusedCfg::kSmemBytes);
    e = e ? e : set_smem(linear_small_s_fused_kernel<false, 2>, FusedCfg::kSmemBytes);
    e = e ? e : set_smem(linear_small_s_fused_kernel<true, 2>, FusedCfg::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<16, false>, SmallCfg<16>::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<16, true>, SmallCfg<16>::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<32, false>, SmallCfg<32>::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<32, true>, SmallCfg<32>::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<64, false>, SmallCfg<64>::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<64, true>, SmallCfg<64>::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<128, false>, SmallCfg<128>::kSmemBytes);
    e = e ? e : set_smem(gemm_small_s_kernel<128, true>, SmallCfg<128>::kSmemBytes);
    if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
    if (g_encode_tiled == nullptr) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
          qres != cudaDriverEntryPointSuccess || fn == nullptr) {
        cudaGetLastError();
        return BATQ_ERR_CUDA;
      }
      g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    }
    d.ready = true;
  }
  if (device_out) *device_out = dev;
  if (info_out) *info_out = &d;
  return BATQ_OK;
}

// Tensor map over packed codes [rows x row_bytes] (uint8), box = 128 bytes x box_rows, 128-byte swizzle.
batq_status make_codes_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t row_bytes, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(row_bytes), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(row_bytes)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBKBytes), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides,
                                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BATQ_OK : BATQ_ERR_CUDA;
}

// Tensor map over packed 4-bit codes [rows x n] (n elements per row, n % 128 == 0) whose loads widen
// every 16 codes (8 bytes) into a 16-byte slot of shared memory: box = 128 elements x box_rows.
batq_status make_u4_unpack_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t n, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(n), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(n / 2)};
  const cuuint32_t box[2] = {128, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 2, const_cast<void*>(base), dims, strides,
                                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BATQ_OK : BATQ_ERR_CUDA;
}

batq_status make_tmap_2d(CUtensorMap* map, CUtensorMapDataType dt, int esz, const void* base, int64_t cols,
                         int64_t rows, int64_t ld_bytes, int box_cols, int box_rows, CUtensorMapSwizzle sw) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld_bytes)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  (void)esz;
  const CUresult r = g_encode_tiled(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BATQ_OK : BATQ_ERR_CUDA;
}

// Tensor map over scale bytes in the BATQ_SF_MMA layout: one row per 512-byte atom (128 uint32),
// boxes of two consecutive atoms = the 8 blocks of one K step; rows past the buffer read as zero.
batq_status make_sf_tmap(CUtensorMap* map, const void* base, int64_t row_tiles, int64_t katoms, int box_atoms = 2) {
  return make_tmap_2d(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, base, 128, row_tiles * katoms, 512, 128, box_atoms,
                      CU_TENSOR_MAP_SWIZZLE_NONE);
}

// fp32 -> bf16 bits, round to nearest even (finite inputs).
inline uint16_t bf16_rn(float f) {
  uint32_t b;
  std::memcpy(&b, &f, 4);
  b += 0x7FFFu + ((b >> 16) & 1u);
  return static_cast<uint16_t>(b >> 16);
}
inline float bf16_to_f32(uint16_t h) {
  const uint32_t b = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &b, 4);
  return f;
}

// Dense block matrices P_j = L_j (x) R_j (Eq. 2), P[(r,c),(r',c')] = L[r][r'] R[c][c'], rounded to
// fp32 and split into three bf16 terms, laid out as the tensor-core B operand (rows = output
// channel f, K = input channel e, no-swizzle K-major: 8 x 16-byte core matrices, K chunks 128
// bytes apart, 8-row groups 512 bytes apart).
void build_block_images(const batq_transform* t, std::vector<uint8_t>* out) {
  out->assign(static_cast<size_t>(t->k) * kQtImageBytes, 0);
  for (int j = 0; j < t->k; ++j) {
    const int gr = t->gr, gc = t->gc;
    const float* L = t->left.data() + (t->left_stride ? static_cast<size_t>(j) * gr * gr : 0);
    const float* R = t->right.data() + (t->right_stride ? static_cast<size_t>(j) * gc * gc : 0);
    uint8_t* img = out->data() + static_cast<size_t>(j) * kQtImageBytes;
    for (int e = 0; e < 32; ++e)
      for (int f = 0; f < 32; ++f) {
        const float pv = static_cast<float>(static_cast<double>(L[(e / gc) * gr + (f / gc)]) *
                                            static_cast<double>(R[(e % gc) * gc + (f % gc)]));
        const uint16_t hi = bf16_rn(pv);
        const float r1 = pv - bf16_to_f32(hi);
        const uint16_t mid = bf16_rn(r1);
        const float r2 = r1 - bf16_to_f32(mid);
        const uint16_t lo = bf16_rn(r2);
        const size_t off = static_cast<size_t>(((f >> 3) * 4 + (e >> 3)) * 128 + (f & 7) * 16 + (e & 7) * 2);
        const uint16_t terms[3] = {hi, mid, lo};
        for (int term = 0; term < 3; ++term) std::memcpy(img + term * kQtTermBytes + off, &terms[term], 2);
      }
  }
}

// Gauss-Jordan inverse with partial pivoting of a small dense matrix, fp64.
bool invert_small(const double* a, int n, double* inv) {
  std::vector<double> w(static_cast<size_t>(n) * 2 * n);
  for (int r = 0; r < n; ++r)
    for (int c = 0; c < n; ++c) {
      w[r * 2 * n + c] = a[r * n + c];
      w[r * 2 * n + n + c] = (r == c) ? 1.0 : 0.0;
    }
  for (int col = 0; col < n; ++col) {
    int piv = col;
    for (int r = col + 1; r < n; ++r)
      if (std::fabs(w[r * 2 * n + col]) > std::fabs(w[piv * 2 * n + col])) piv = r;
    const double pv = w[piv * 2 * n + col];
    if (!(std::fabs(pv) > 1e-300) || !std::isfinite(pv)) return false;
    if (piv != col)
      for (int c = 0; c < 2 * n; ++c) std::swap(w[col * 2 * n + c], w[piv * 2 * n + c]);
    for (int c = 0; c < 2 * n; ++c) w[col * 2 * n + c] /= pv;
    for (int r = 0; r < n; ++r) {
      if (r == col) continue;
      const double f = w[r * 2 * n + col];
      if (f == 0.0) continue;
      for (int c = 0; c < 2 * n; ++c) w[r * 2 * n + c] -= f * w[col * 2 * n + c];
    }
  }
  for (int r = 0; r < n; ++r)
    for (int c = 0; c < n; ++c) inv[r * n + c] = w[r * 2 * n + n + c];
  return true;
}

batq_status check_x(const void* x, int64_t s, int64_t n, int64_t ld) {
  if (s < 0 || n <= 0 || n % 32 != 0 || ld < n || n > (int64_t(1) << 24) || s > (int64_t(1) << 30)) return BATQ_ERR_SHAPE;
  if (s > 0 && x == nullptr) return BATQ_ERR_NULL;
  if (ld % 8 != 0 || !aligned(x, 16)) return BATQ_ERR_ALIGN;
  return BATQ_OK;
}

constexpr int64_t kSmallSMax = 128;       // the swapped-operand split-K GEMM takes up to this many tokens
constexpr int64_t kSmallQuantAuto = 128;  // per-block ALU quantiser up to here, tensor cores above (4.0 us against 1.7-3.0 us back to back at n = 4096)
std::atomic<int> g_force_quantizer{0};  // tuning hook: 0 = automatic, 1 = ALU (Kronecker form), 2 = tensor cores (dense form)

// Tensor-core version: 128-token x 4-block units.
batq_status launch_quantize_tc(const batq_transform* t, const void* x, int64_t s, int64_t n, int64_t ld, void* codes,
                               void* scales, int32_t layout, float* debug_out, cudaStream_t stream, int sm_count,
                               bool fp8 = false) {
  QuantTcParams p{};
  p.s = s;
  p.n = static_cast<int32_t>(n);
  p.k = static_cast<int32_t>(n / 32);
  p.n_strips = (p.k + kQtGroups - 1) / kQtGroups;
  p.n_row_tiles = (s + kQtRows - 1) / kQtRows;
  p.n_units = p.n_strips * p.n_row_tiles;
  p.pimg = t->d_pimg;
  p.clip_lo = t->d_clip_lo;
  p.clip_hi = t->d_clip_hi;
  p.scales = static_cast<uint8_t*>(scales);
  p.sf_layout = layout;
  p.sf_katoms = katoms_of(p.k);
  p.debug_out = debug_out;
  CUtensorMap tmap_x, tmap_codes;
  std::memset(&tmap_codes, 0, sizeof(tmap_codes));
  batq_status st = make_tmap_2d(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x, n, s, ld * 2, 64, kQtRows,
                                CU_TENSOR_MAP_SWIZZLE_128B);
  if (st == BATQ_OK && debug_out == nullptr)
    st = fp8 ? make_tmap_2d(&tmap_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes, n, s, n, 128, kQtRows,
                            CU_TENSOR_MAP_SWIZZLE_128B)
             : make_tmap_2d(&tmap_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes, n / 2, s, n / 2, 64, kQtRows,
                            CU_TENSOR_MAP_SWIZZLE_64B);
  if (st != BATQ_OK) return st;
  if (debug_out == nullptr && layout == BATQ_SF_MMA && p.sf_katoms > p.n_strips) {
    // an odd number of 4-block atoms: keep the padding atom finite
    if (cudaMemsetAsync(scales, 0, batq_sf_bytes(s, n, BATQ_SF_MMA), stream) != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  }
  const int grid = static_cast<int>(std::min<int64_t>(sm_count, p.n_units));
  const bool cl = t->has_clip, dbg = debug_out != nullptr;
  // Launched as a programmatic dependent: if the kernel before it on the stream releases its
  // dependents early (the GEMMs of this library do), the quantiser's CTAs take over the SMs that
  // kernel has left and wait there; otherwise this is an ordinary launch.
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(kQtThreads);
  cfg.dynamicSmemBytes = kQtSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
#define BATQ_QT(CL, DB, F8) cudaLaunchKernelEx(&cfg, quantize_act_tc_kernel<CL, DB, F8>, tmap_x, tmap_codes, p)
  if (fp8 && !dbg) e = cl ? BATQ_QT(true, false, true) : BATQ_QT(false, false, true);
  else if (!dbg) e = cl ? BATQ_QT(true, false, false) : BATQ_QT(false, false, false);
  else e = cl ? BATQ_QT(true, true, false) : BATQ_QT(false, true, false);
#undef BATQ_QT
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

// Factor sizes the four-lanes-per-block ALU code (small quantiser, fused small-s layer) is built for.
bool alu_small_geometry(const batq_transform* t) {
  return t == nullptr || t->gc == 8 || t->gc == 4 || t->gc == 2;
}

batq_status launch_quantize(const batq_transform* t, const void* x, int64_t s, int64_t n, int64_t ld, void* codes,
                            void* scales, int32_t layout, float* debug_out, cudaStream_t stream,
                            uint32_t* zero_words = nullptr, int32_t n_zero_words = 0) {
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (t != nullptr && t->device != dev) return BATQ_ERR_CUDA;
  // The dense-block tensor-core kernel works on 128-token tiles; tiny batches (decode) and the
  // identity transform stay on the ALU kernel.
  // The per-block ALU kernel takes right factors of 8, 4 or 2 columns (4 x 8, 8 x 4, 16 x 2), the
  // streaming ALU kernel 4 x 8 only; every other case goes through the tensor-core kernel, which
  // only sees the dense block matrices.
  const bool small_ok = alu_small_geometry(t);
  const bool stream_ok = t == nullptr || (t->gr == 4 && t->gc == 8);
  const bool mid = t != nullptr && t->bf16_mid;   // needs the factored form: the ALU kernels (4 x 8 only, checked when it is set)
  const bool small_path = n_zero_words > 0;  // in front of the small-s GEMM (its tickets to clear)
  const int force_q = g_force_quantizer.load(std::memory_order_relaxed);
  // Narrower right factors cost the four lanes more work per block (8 x 4: 2.0 us at 16 tokens and
  // 4.5 us at 128 for n = 4096; 16 x 2: 2.9 and 7.8 us; the tensor-core kernel 4.0-4.2 us throughout).
  const int64_t small_limit = stream_ok ? kSmallQuantAuto : (t->gc == 4 ? 64 : 32);
  const bool want_small = force_q == 3 || (force_q == 0 && (s <= small_limit || (stream_ok && small_path && s <= kSmallSMax)));
  const bool use_tc = !small_ok || (!stream_ok && !want_small) ||
                      (!mid && !small_path && t != nullptr && (force_q == 2 || (force_q == 0 && s > kSmallQuantAuto)));
  if (use_tc) {
    if (n_zero_words > 0 &&
        cudaMemsetAsync(zero_words, 0, static_cast<size_t>(n_zero_words) * 4, stream) != cudaSuccess) {
      cudaGetLastError();
      return BATQ_ERR_CUDA;
    }
    return launch_quantize_tc(t, x, s, n, ld, codes, scales, layout, debug_out, stream, info->sm_count);
  }
  // A handful of tokens: the ring of the streaming kernel below is all latency there; one thread
  // per (token, block) with everything loaded up front is quicker.
  if (want_small) {
    QuantSmallParams q{};
    q.x = static_cast<const uint16_t*>(x);
    q.ld = ld;
    q.s = static_cast<int32_t>(s);
    q.n = static_cast<int32_t>(n);
    q.k = static_cast<int32_t>(n / 32);
    if (t != nullptr) {
      q.left = t->d_left; q.right = t->d_right;
      q.left_stride = t->left_stride; q.right_stride = t->right_stride;
      q.clip_lo = t->d_clip_lo; q.clip_hi = t->d_clip_hi;
    }
    q.codes = static_cast<uint8_t*>(codes);
    q.scales = static_cast<uint8_t*>(scales);
    q.sf_layout = layout;
    q.sf_katoms = katoms_of(q.k);
    q.debug_out = debug_out;
    q.zero_words = zero_words;
    q.n_zero_words = n_zero_words;
    q.bf16_mid = mid ? 1 : 0;
    // Launched as a programmatic dependent of whatever precedes it on the stream (in a decode loop
    // the GEMM of the layer before): it is scheduled early and waits inside the kernel.
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>((s * q.k + 31) / 32));  // four lanes per (token, block)
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int gc = t != nullptr ? t->gc : 8;
    const bool dbg = debug_out != nullptr;
    cudaError_t e;
    if (gc == 8)      e = dbg ? cudaLaunchKernelEx(&cfg, quantize_act_small_kernel<true, 8>, q)
                              : cudaLaunchKernelEx(&cfg, quantize_act_small_kernel<false, 8>, q);
    else if (gc == 4) e = dbg ? cudaLaunchKernelEx(&cfg, quantize_act_small_kernel<true, 4>, q)
                              : cudaLaunchKernelEx(&cfg, quantize_act_small_kernel<false, 4>, q);
    else              e = dbg ? cudaLaunchKernelEx(&cfg, quantize_act_small_kernel<true, 2>, q)
                              : cudaLaunchKernelEx(&cfg, quantize_act_small_kernel<false, 2>, q);
    if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
    return BATQ_OK;
  }
  QuantActParams p{};
  p.x = static_cast<const uint16_t*>(x);
  p.ld = ld;
  p.s = s;
  p.n = static_cast<int32_t>(n);
  p.k = static_cast<int32_t>(n / 32);
  int gs = 32;
  while (p.k % gs != 0) gs >>= 1;
  p.gs = gs;
  p.rows_per_tile = kQaConsumers / gs;
  p.n_row_tiles = (s + p.rows_per_tile - 1) / p.rows_per_tile;
  p.n_units = (p.k / gs) * p.n_row_tiles;
  if (t != nullptr) {
    p.left = t->d_left; p.right = t->d_right;
    p.left_stride = t->left_stride; p.right_stride = t->right_stride;
    p.clip_lo = t->d_clip_lo; p.clip_hi = t->d_clip_hi;
  }
  p.clip_row_stride = 0;
  p.codes = static_cast<uint8_t*>(codes);
  p.scales = static_cast<uint8_t*>(scales);
  p.sf_layout = layout;
  p.sf_katoms = katoms_of(p.k);
  p.debug_out = debug_out;
  p.zero_words = zero_words;
  p.n_zero_words = n_zero_words;
  p.bf16_mid = mid ? 1 : 0;
  const int grid = static_cast<int>(std::min<int64_t>(info->sm_count, p.n_units));
  const bool xf = t != nullptr, cl = t != nullptr && t->has_clip, dbg = debug_out != nullptr;
#define BATQ_QA(XF, CL, DB) quantize_act_kernel<XF, CL, DB><<<grid, kQaThreads, kQaSmemBytes, stream>>>(p)
  if (xf && cl && !dbg) BATQ_QA(true, true, false);
  else if (xf && !cl && !dbg) BATQ_QA(true, false, false);
  else if (!xf && !dbg) BATQ_QA(false, false, false);
  else if (xf && cl && dbg) BATQ_QA(true, true, true);
  else if (xf && !cl && dbg) BATQ_QA(true, false, true);
  else BATQ_QA(false, false, true);
#undef BATQ_QA
  return cudaGetLastError() == cudaSuccess ? BATQ_OK : BATQ_ERR_CUDA;
}

// Tensor map over a row-major output [rows x cols], box = 128 (or 64) bytes x 32 rows with the
// swizzle of that width.
batq_status make_y_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                        int row_bytes = 128) {
  const int esz = bf16 ? 2 : 4;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld * esz)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(row_bytes / esz), 32};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode_tiled(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                                    const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BATQ_OK : BATQ_ERR_CUDA;
}

// Tile width.  192 and 128 keep two accumulators in tensor memory (the epilogue of a tile
// overlaps the main loop of the next); 256 has the highest flop per byte staged but a single
// accumulator.  Pick by modelled time: waves x (main loop + exposed epilogue), with the main
// loop proportional to the tile width.
std::atomic<int> g_force_bn{0};  // test hook: 0 = automatic
int pick_bn(int64_t s, int64_t m, int64_t n, int sm_count) {
  const int force_bn = g_force_bn.load(std::memory_order_relaxed);
  if (force_bn == 64 || force_bn == 128 || force_bn == 192 || force_bn == 256) return force_bn;
  const int64_t mt = (s + kBM - 1) / kBM;
  // A few dozen tiles cannot pull the weights fast enough (a CTA streams what its ring keeps in
  // flight): below half a wave of 128-wide tiles, twice as many 64-wide ones.
  if (mt * ((m + 127) / 128) * 2 <= sm_count && m > 64) return 64;
  const double k_steps = static_cast<double>((n + 255) / 256);
  auto cost = [&](int bn, double exposed_epilogue) {
    const int64_t tiles = mt * ((m + bn - 1) / bn);
    const int64_t waves = (tiles + sm_count - 1) / sm_count;
    return static_cast<double>(waves) * (k_steps * bn / 256.0 + exposed_epilogue * bn / 256.0);
  };
  const double c256 = cost(256, 3.0), c192 = cost(192, 0.3), c128 = cost(128, 0.3) * 1.08;
  if (m <= 128) return 128;
  if (c192 <= c256 && c192 <= c128) return 192;
  return c256 <= c128 ? 256 : 128;
}

std::atomic<int> g_force_gemm_kernel{0};  // tuning hook: 0 = automatic, 1 = one CTA per tile, 2 = CTA pairs (two accumulators), 3 = CTA pairs (wide tiles)

// The schedule of the CTA-pair kernel for an s x m output with k_steps K-steps: the segments of
// column widths and the number of pairs.  Candidates: columns all 128, 192 or 256 wide; 256 and
// 192 alternating; and every split of the features into a columns of 256 and b of 192, arranged as
// 256s-192s-256s or 192s-256s-192s with the outer group cut at several places.  Each candidate is
// walked exactly as the kernel walks it, and the pair that finishes last decides.
// Model, in units of one K-step of a 192-wide tile (about 0.36 us): a K-step of a W-wide tile
// moves 32 KiB of activations and W / 8 KiB of weights through L2, which is what its time follows;
// a tile adds a small fixed cost, and about 2 us when it has to wait for the accumulator slot of
// the tile just before it (that tile's epilogue, less what the filled ring wins back afterwards;
// fitted to measured layers); the epilogue of a pair's last tile (about 3 us at 256 columns) is
// always exposed.
struct PairSched {
  int32_t n_cols, n_segs, pairs;
  PairSeg seg[kPairMaxSegs];
};

inline int64_t seg_span(int wa, int wb, int64_t cols) { return (cols / 2) * (wa + wb) + (cols & 1) * wa; }

// Appends columns to a candidate; false if it does not fit the segment table.
bool sched_add(PairSched* c, int wa, int wb, int64_t cols) {
  if (cols <= 0) return true;
  if (c->n_segs > 0) {
    PairSeg& l = c->seg[c->n_segs - 1];
    if (l.wa == l.wb && wa == wb && l.wa == wa) { l.cols += static_cast<int32_t>(cols); c->n_cols += static_cast<int32_t>(cols); return true; }
  }
  if (c->n_segs == kPairMaxSegs) return false;
  PairSeg& g = c->seg[c->n_segs];
  g.col0 = c->n_cols;
  g.n0 = c->n_segs == 0 ? 0 : static_cast<int32_t>(c->seg[c->n_segs - 1].n0 +
                                                   seg_span(c->seg[c->n_segs - 1].wa, c->seg[c->n_segs - 1].wb, c->seg[c->n_segs - 1].cols));
  g.cols = static_cast<int32_t>(cols);
  g.wa = static_cast<int16_t>(wa);
  g.wb = static_cast<int16_t>(wb);
  ++c->n_segs;
  c->n_cols += static_cast<int32_t>(cols);
  return true;
}

double sched_cost(const PairSched& c, PairParams* p, int64_t k_steps, int max_pairs, int* pairs_out) {
  p->n_cols = c.n_cols;
  p->n_segs = c.n_segs;
  for (int i = 0; i < kPairMaxSegs; ++i) p->seg[i] = c.seg[i];
  const int np = static_cast<int>(std::min<int64_t>(max_pairs, static_cast<int64_t>(p->m_pairs) * c.n_cols));
  *pairs_out = np;
  double worst = 0.0;
  for (int pr = 0; pr < np; ++pr) {
    PairWalk walk(*p, pr, np);
    PairSlots slots;
    PairTile t;
    int last = -1, last_bn = 0;
    double cost = 0.0;
    while (walk.next(t)) {
      int slot;
      uint32_t phase;
      slots.take(t.bn, slot, phase);
      cost += static_cast<double>(k_steps) * (32.0 + t.bn / 8.0) / 56.0 + (slot == last ? 5.0 : 1.0);
      last = slot;
      last_bn = t.bn;
    }
    cost += 8.0 * last_bn / 256.0;
    worst = std::max(worst, cost);
  }
  return worst;
}

bool pair_schedule(int64_t s, int64_t m, int64_t k_steps, int sm_count, PairParams* p, int* pairs) {
  const int64_t m_pairs = (s + 255) / 256;
  const int max_pairs = std::max(1, sm_count / 2);
  if (m_pairs * ((m + 63) / 64) > INT32_MAX) return false;
  p->s = static_cast<int32_t>(s);
  p->m = static_cast<int32_t>(m);
  p->m_pairs = static_cast<int32_t>(m_pairs);
  const int force_bn = g_force_bn.load(std::memory_order_relaxed);
  const bool forced = force_bn == 64 || force_bn == 128 || force_bn == 192 || force_bn == 256 || force_bn == 448;
  PairSched best{};
  double best_cost = 1e30;
  auto consider = [&](const PairSched& c) {
    // every column must start inside the layer and the columns must reach its edge
    const PairSeg& l = c.seg[c.n_segs - 1];
    const int64_t end = l.n0 + seg_span(l.wa, l.wb, l.cols);
    const int64_t last_w = (l.cols & 1) ? l.wa : l.wb;
    if (end < m || end - last_w >= m) return;
    int np;
    const double cost = sched_cost(c, p, k_steps, max_pairs, &np);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = c; best.pairs = np; }
  };
  // columns all equally wide, or 256 and 192 alternating
  const int uniform[5] = {0, 256, 192, 128, 64};
  for (int ci = 0; ci < 5; ++ci) {
    const int w = uniform[ci];
    if (forced ? (force_bn == 448 ? w != 0 : w != force_bn) : w == 64) continue;  // 64: only when forced
    PairSched c{};
    if (w != 0) {
      sched_add(&c, w, w, (m + w - 1) / w);
    } else {
      const int64_t full = m / 448, rem = m % 448;
      sched_add(&c, 256, 192, 2 * full + (rem == 0 ? 0 : (rem <= 256 ? 1 : 2)));
    }
    consider(c);
  }
  if (!forced && force_bn != 1) {   // 1: only the uniform and alternating candidates above
    // a columns of 256 and b of 192 (the last one as narrow as the edge allows), in three groups;
    // with many tiles per pair the balance matters less and fewer splits are tried
    const int64_t a_max = (m + 255) / 256;
    const int64_t a_step = std::max<int64_t>(1, a_max * m_pairs / (24 * max_pairs));
    for (int64_t a = 1; a < a_max; a += a_step) {
      const int64_t rest = m - 256 * a;
      if (rest <= 0) break;
      const int64_t b = (rest + 191) / 192;
      const int64_t cuts[7] = {0, 1, 2, 3, 4, 5, 6};
      for (int ci = 0; ci < 7; ++ci) {
        const int64_t a1 = a * cuts[ci] / 6, b1 = b * cuts[ci] / 6;
        {
          PairSched c{};
          if (sched_add(&c, 256, 256, a1) && sched_add(&c, 192, 192, b) && sched_add(&c, 256, 256, a - a1)) consider(c);
        }
        if (ci > 0 && ci < 6) {
          PairSched c{};
          if (sched_add(&c, 192, 192, b1) && sched_add(&c, 256, 256, a) && sched_add(&c, 192, 192, b - b1)) consider(c);
        }
      }
    }
    // 256 and 192 alternating for the first 2c columns, then all 192 or all 256 to the edge
    const int64_t c_max = m / 448;
    const int64_t c_step = std::max<int64_t>(1, c_max * m_pairs / (24 * max_pairs));
    for (int64_t cp = 1; cp <= c_max; cp += c_step) {
      const int64_t rest = m - 448 * cp;
      if (rest <= 0) break;
      for (int w = 192; w <= 256; w += 64) {
        PairSched c{};
        if (sched_add(&c, 256, 192, 2 * cp) && sched_add(&c, w, w, (rest + w - 1) / w)) consider(c);
        PairSched d{};
        if (sched_add(&d, w, w, rest / w) && rest % w == 0 && sched_add(&d, 256, 192, 2 * cp)) consider(d);
      }
    }
  }
  if (best_cost >= 1e30) return false;
  p->n_cols = best.n_cols;
  p->n_segs = best.n_segs;
  for (int i = 0; i < kPairMaxSegs; ++i) p->seg[i] = best.seg[i];
  *pairs = best.pairs;
  return true;
}

// ---- the wide-tile pair kernel: one accumulator of up to 448 columns per tile ---------------------
// Cost of a pair's tiles in microseconds, fitted to measured layers (2048 tokens, K = 4096 and
// 14336, every column 256 / 320 / 384 / 448 wide): a K-step of a tile up to 384 wide takes
// 0.17 + 0.0009 bn us (0.40 at 256, 0.52 at 384: the bytes the SM pulls from L2), one of a 448-wide
// tile 0.66 us (four stages of 49 KiB turn over at the latency of a load from L2); about 1.4 us
// per tile pass between the last MMA of one tile and the first of the next.
// With MXFP8 activations (a8) the tensor cores run at half the rate and are the only limit:
// 0.60 us per 256 elements of K at 256 columns, in proportion to the width.
double wide_tile_us(int bn, int64_t k_steps, bool a8 = false) {
  const double step = a8 ? 0.60 * bn / 256.0 : (bn > 384 ? 0.66 : 0.17 + 0.0009 * bn);
  return static_cast<double>(k_steps) * step + 1.4;
}
// The same for the two-accumulator kernel: bound by its loads (36 KiB per K-step at 256 columns),
// the epilogue hidden unless two tiles in a row need the same accumulator.
double pair_tile_us(int bn, int64_t k_steps, bool same_slot) {
  return static_cast<double>(k_steps) * 0.383 * (32.0 + bn / 8.0) / 64.0 + (same_slot ? 1.7 : 1.1);
}

double wide_cost(const PairSched& c, PairParams* p, int64_t k_steps, int max_pairs, bool a8, int* pairs_out) {
  p->n_cols = c.n_cols;
  p->n_segs = c.n_segs;
  for (int i = 0; i < kPairMaxSegs; ++i) p->seg[i] = c.seg[i];
  const int np = static_cast<int>(std::min<int64_t>(max_pairs, static_cast<int64_t>(p->m_pairs) * c.n_cols));
  *pairs_out = np;
  double worst = 0.0;
  for (int pr = 0; pr < np; ++pr) {
    PairWalk walk(*p, pr, np);
    PairTile t;
    double cost = 0.0;
    while (walk.next(t)) cost += wide_tile_us(t.bn, k_steps, a8);
    worst = std::max(worst, cost);
  }
  return worst + 5.5;   // launch, first loads, the last tile's stores
}

// The two-accumulator schedule's cost in the same unit, for the choice between the kernels.
double pair_cost_us(PairParams* p, int64_t k_steps, int np) {
  double worst = 0.0;
  for (int pr = 0; pr < np; ++pr) {
    PairWalk walk(*p, pr, np);
    PairSlots slots;
    PairTile t;
    int last = -1;
    double cost = 0.0;
    while (walk.next(t)) {
      int slot;
      uint32_t phase;
      slots.take(t.bn, slot, phase);
      cost += pair_tile_us(t.bn, k_steps, slot == last);
      last = slot;
    }
    worst = std::max(worst, cost);
  }
  return worst + 1.5;   // the last tile's epilogue
}

bool wide_schedule(int64_t s, int64_t m, int64_t k_steps, int sm_count, int force_w, bool a8, PairParams* p, int* pairs,
                   double* cost_us) {
  const int64_t m_pairs = (s + 255) / 256;
  const int max_pairs = std::max(1, sm_count / 2);
  if (m_pairs * ((m + 63) / 64) > INT32_MAX) return false;
  p->s = static_cast<int32_t>(s);
  p->m = static_cast<int32_t>(m);
  p->m_pairs = static_cast<int32_t>(m_pairs);
  PairSched best{};
  double best_cost = 1e30;
  auto consider = [&](const PairSched& c) {
    const PairSeg& l = c.seg[c.n_segs - 1];
    const int64_t end = l.n0 + seg_span(l.wa, l.wb, l.cols);
    if (end < m || end - l.wb >= m) return;
    int np;
    const double cost = wide_cost(c, p, k_steps, max_pairs, a8, &np);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = c; best.pairs = np; }
  };
  const int widths[6] = {448, 384, 320, 256, 192, 128};
  if (force_w > 0) {   // tuning hook: every column this wide
    PairSched c{};
    sched_add(&c, force_w, force_w, (m + force_w - 1) / force_w);
    consider(c);
  }
  for (int i = 0; i < 6 && force_w <= 0; ++i) {
    const int w1 = widths[i];
    {
      PairSched c{};
      sched_add(&c, w1, w1, (m + w1 - 1) / w1);
      consider(c);
    }
    // x columns of w1, then columns of w2 to the edge, and the other way round
    const int64_t x_max = m / w1;
    const int64_t x_step = std::max<int64_t>(1, x_max * m_pairs / (32 * max_pairs));
    for (int j = 0; j < 6; ++j) {
      const int w2 = widths[j];
      if (w2 == w1) continue;
      for (int64_t x = 1; x <= x_max; x += x_step) {
        const int64_t rest = m - x * w1;
        if (rest <= 0) break;
        PairSched c{};
        if (sched_add(&c, w1, w1, x) && sched_add(&c, w2, w2, (rest + w2 - 1) / w2)) consider(c);
      }
    }
  }
  if (best_cost >= 1e30) return false;
  p->n_cols = best.n_cols;
  p->n_segs = best.n_segs;
  for (int i = 0; i < kPairMaxSegs; ++i) p->seg[i] = best.seg[i];
  *pairs = best.pairs;
  *cost_us = best_cost;
  return true;
}

// The same, remembered per prepared weight and token count (the search walks a few hundred
// candidates; a layer is called with few distinct token counts).
bool pair_schedule_cached(const batq_weight* w, int64_t s, int sm_count, bool wide, PairParams* p, int* pairs,
                          double* cost_us, bool a8 = false) {
  a8 = a8 && wide;   // the activations' format only enters the wide tiles' cost
  const int force_bn = g_force_bn.load(std::memory_order_relaxed);
  {
    std::lock_guard<std::mutex> lock(w->sched_mutex);
    for (const auto& e : w->sched_cache)
      if (e.s == s && e.force_bn == force_bn && e.wide == wide && e.a8 == a8) {
        p->s = static_cast<int32_t>(s);
        p->m = static_cast<int32_t>(w->m);
        p->m_pairs = static_cast<int32_t>((s + 255) / 256);
        p->n_cols = e.n_cols;
        p->n_segs = e.n_segs;
        for (int i = 0; i < kPairMaxSegs; ++i) p->seg[i] = e.seg[i];
        *pairs = e.pairs;
        *cost_us = e.cost;
        return true;
      }
  }
  const int64_t k_steps = (w->n + 255) / 256;
  if (wide) {
    const bool fw = force_bn >= 64 && force_bn <= kWideMaxBn && force_bn % 64 == 0;
    if (!wide_schedule(s, w->m, k_steps, sm_count, fw ? force_bn : 0, a8, p, pairs, cost_us)) return false;
  } else {
    if (!pair_schedule(s, w->m, k_steps, sm_count, p, pairs)) return false;
    *cost_us = pair_cost_us(p, k_steps, *pairs);
  }
  batq_weight::SchedEntry e{};
  e.s = s; e.force_bn = force_bn; e.wide = wide; e.a8 = a8; e.cost = *cost_us;
  e.n_cols = p->n_cols; e.n_segs = p->n_segs; e.pairs = *pairs;
  for (int i = 0; i < kPairMaxSegs; ++i) e.seg[i] = p->seg[i];
  std::lock_guard<std::mutex> lock(w->sched_mutex);
  if (w->sched_cache.size() >= 16) w->sched_cache.erase(w->sched_cache.begin());
  w->sched_cache.push_back(e);
  return true;
}

template <bool BF, bool WIDE>
cudaError_t launch_pair_kernel(int grid, cudaStream_t stream, bool dependent, const CUtensorMap& ta, const CUtensorMap& tb,
                               const CUtensorMap& tsfa, const CUtensorMap& tsfb, const CUtensorMap& ty,
                               const PairParams& p) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(WIDE ? kWideThreads : kPairThreads);
  cfg.dynamicSmemBytes = WIDE ? WideCfg::kSmemBytes : PairCfg::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 2 : 1;
  if (WIDE) return cudaLaunchKernelEx(&cfg, gemm_mxfp4_wide_kernel<BF>, ta, tb, tsfa, tsfb, ty, p);
  return cudaLaunchKernelEx(&cfg, gemm_mxfp4_pair_kernel<BF>, ta, tb, tsfa, tsfb, ty, p);
}

batq_status launch_gemm_pair(const void* x_codes, const void* x_sf, const batq_weight* w, int64_t s, void* y,
                             bool bf, int64_t ldy, cudaStream_t stream, int sm_count, const CUtensorMap& tmap_a,
                             const CUtensorMap& tmap_y, int64_t m16, bool dependent) {
  (void)x_codes;
  CUtensorMap tmap_sfa;
  batq_status st = make_sf_tmap(&tmap_sfa, x_sf, (s + 127) / 128, w->katoms);
  if (st != BATQ_OK) return st;
  // Two kernels share this launcher: tiles of up to 256 features with two accumulators, or tiles of
  // up to 448 with one; each comes with its own schedule and an estimate of its time.
  const int force_gemm = g_force_gemm_kernel.load(std::memory_order_relaxed);
  const int force_bn = g_force_bn.load(std::memory_order_relaxed);
  const bool may_wide = force_gemm == 3 ? (force_bn == 0 || (force_bn >= 64 && force_bn <= kWideMaxBn && force_bn % 64 == 0))
                                        : (w->m >= 320 && force_bn == 0);
  PairParams p{}, pw{};
  int pairs = 0, pairs_w = 0;
  double us = 0.0, us_w = 0.0;
  bool wide = false;
  if (force_gemm == 3 && may_wide) {
    if (!pair_schedule_cached(w, s, sm_count, true, &pw, &pairs_w, &us_w)) return BATQ_ERR_SHAPE;
    wide = true;
  } else {
    if (!pair_schedule_cached(w, s, sm_count, false, &p, &pairs, &us)) return BATQ_ERR_SHAPE;
    if (force_gemm == 0 && may_wide &&
        pair_schedule_cached(w, s, sm_count, true, &pw, &pairs_w, &us_w))
      wide = us_w < us;
  }
  CUtensorMap tmap_y64;
  std::memset(&tmap_y64, 0, sizeof(tmap_y64));
  if (wide) {
    p = pw;
    pairs = pairs_w;
    if (m16 > 0) {   // the wide kernel stages its output in boxes of 64-byte rows
      st = make_y_tmap(&tmap_y64, y, s, m16, ldy, bf, 64);
      if (st != BATQ_OK) return st;
    }
  }
  p.katoms = w->katoms;
  p.k_steps = static_cast<int32_t>((w->n + 255) / 256);
  p.m16 = static_cast<int32_t>(m16);
  p.y = y;
  p.ldy = ldy;
  const int grid = 2 * pairs;
  cudaError_t e;
  if (wide) e = bf ? launch_pair_kernel<true, true>(grid, stream, dependent, tmap_a, w->tmap_b32, tmap_sfa, w->tmap_sf, tmap_y64, p)
                   : launch_pair_kernel<false, true>(grid, stream, dependent, tmap_a, w->tmap_b32, tmap_sfa, w->tmap_sf, tmap_y64, p);
  else      e = bf ? launch_pair_kernel<true, false>(grid, stream, dependent, tmap_a, w->tmap_b32, tmap_sfa, w->tmap_sf, tmap_y, p)
                   : launch_pair_kernel<false, false>(grid, stream, dependent, tmap_a, w->tmap_b32, tmap_sfa, w->tmap_sf, tmap_y, p);
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

// `dependent`: the kernel directly before this one on the stream is the activation quantiser of
// the same layer; the GEMM is then launched as its programmatic dependent.
batq_status launch_gemm(const void* x_codes, const void* x_sf, const batq_weight* w, int64_t s, void* y,
                        int32_t y_dtype, int64_t ldy, cudaStream_t stream, bool dependent = false) {
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (w->device != dev) return BATQ_ERR_CUDA;
  const bool bf = y_dtype == BATQ_BF16;
  CUtensorMap tmap_a, tmap_y;
  std::memset(&tmap_y, 0, sizeof(tmap_y));
  st = make_codes_tmap(&tmap_a, x_codes, s, w->n / 2, kBM);
  const int64_t m16 = w->m / (bf ? 8 : 4) * (bf ? 8 : 4);
  if (st == BATQ_OK && m16 > 0) st = make_y_tmap(&tmap_y, y, s, m16, ldy, bf);
  if (st != BATQ_OK) return st;
  // CTA pairs need at least two 128-token tiles to pay, and wide enough a layer for their tiles.
  const int force_gemm = g_force_gemm_kernel.load(std::memory_order_relaxed);
  const bool use_pair = force_gemm == 2 || force_gemm == 3 || (force_gemm == 0 && s > 128 && w->m >= 192);
  if (use_pair) return launch_gemm_pair(x_codes, x_sf, w, s, y, bf, ldy, stream, info->sm_count, tmap_a, tmap_y, m16, dependent);
  const int bn = pick_bn(s, w->m, w->n, info->sm_count);
  GemmParams p{};
  p.sfa = static_cast<const uint8_t*>(x_sf);
  p.sfb = w->scales;
  p.s = static_cast<int32_t>(s);
  p.m = static_cast<int32_t>(w->m);
  p.katoms = w->katoms;
  p.k_steps = static_cast<int32_t>((w->n + 255) / 256);
  p.m_tiles = static_cast<int32_t>((s + kBM - 1) / kBM);
  p.n_tiles = static_cast<int32_t>((w->m + bn - 1) / bn);
  p.sfb_row_tiles = static_cast<int32_t>((w->m + 127) / 128);
  p.m16 = static_cast<int32_t>(m16);
  p.y = y;
  p.ldy = ldy;
  const int grid = std::min(info->sm_count, p.m_tiles * p.n_tiles);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(kGemmThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  cudaError_t e;
#define BATQ_GEMM(BN, BF, TB) \
  (cfg.dynamicSmemBytes = GemmCfg<BN>::kSmemBytes, cudaLaunchKernelEx(&cfg, gemm_mxfp4_kernel<BN, BF>, tmap_a, TB, tmap_y, p))
  if (bn == 256) e = bf ? BATQ_GEMM(256, true, w->tmap_b256) : BATQ_GEMM(256, false, w->tmap_b256);
  else if (bn == 192) e = bf ? BATQ_GEMM(192, true, w->tmap_b192) : BATQ_GEMM(192, false, w->tmap_b192);
  else if (bn == 128) e = bf ? BATQ_GEMM(128, true, w->tmap_b128) : BATQ_GEMM(128, false, w->tmap_b128);
  else e = bf ? BATQ_GEMM(64, true, w->tmap_b64) : BATQ_GEMM(64, false, w->tmap_b64);
#undef BATQ_GEMM
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

// ---- small-s (decode) GEMM: split choice, scratch layout, launch -------------------------------
std::atomic<int> g_force_splits{0};  // tuning hook: 0 = automatic
std::atomic<int> g_small_reduce{0};  // tuning hook: 0 = automatic, 1 = always tickets, 2 = cluster whenever splits <= 8
constexpr int kMaxSplits = 32;

inline int small_ntok(int64_t s) { return s <= 16 ? 16 : (s <= 32 ? 32 : (s <= 64 ? 64 : 128)); }


// The K splits of a row tile can meet as one thread-block cluster (reduction through distributed
// shared memory) when there are at most 8 of them and the grid leaves the gang scheduler of
// clusters some room: at most 90 % of the two-per-SM slots, 80 % above 4 tokens, where the CTAs
// of the quantiser in front (tokens x blocks / 32 of them, resident while they wait) take room
// too.  Measured: a fuller grid leaves a few clusters for a second wave, which costs a layer of
// the decode benchmark about 5 us.
bool cluster_reduce_ok(int64_t tiles, int sp, int64_t slots, int64_t s) {
  const int force_reduce = g_small_reduce.load(std::memory_order_relaxed);
  if (sp < 2 || sp > 8 || force_reduce == 1) return false;
  return force_reduce == 2 || tiles * sp * 10 <= slots * (s > 4 ? 8 : 9);
}

// Number of K splits: the grid is (row tiles) x (splits) CTAs, two resident per SM.  Modelled
// time = waves x (K-steps per CTA + fixed cost) + a reduction term that grows with the splits,
// plus the round trip through scratch and tickets where the cluster reduction does not apply
// (all in units of one K-step of streaming, about 0.5 us).
int pick_splits(int64_t m, int64_t n, int64_t s, int sm_count) {
  const int k_steps = static_cast<int>((n + 255) / 256);
  const int force_splits = g_force_splits.load(std::memory_order_relaxed);
  if (force_splits > 0) return std::min(std::min(force_splits, k_steps), kMaxSplits);
  const int64_t tiles = (m + 127) / 128;
  const int64_t slots = 2 * static_cast<int64_t>(sm_count > 0 ? sm_count : 148);
  int best = 1;
  double best_cost = 1e30;
  for (int sp = 1; sp <= std::min(k_steps, kMaxSplits); ++sp) {
    const int64_t waves = (tiles * sp + slots - 1) / slots;
    double cost = static_cast<double>(waves) * ((k_steps + sp - 1) / sp + 3.0) + 0.15 * sp;
    if (sp > 1 && !cluster_reduce_ok(tiles, sp, slots, s)) cost += 2.0;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = sp; }
  }
  return best;
}

// Scratch of the small-s GEMM: split-K partial tiles, then one ticket word per row tile.
struct SmallScratch {
  size_t partial_bytes, ticket_bytes;
  int splits, ntok;
  bool cluster;  // the splits of a row tile meet as a thread-block cluster (partials in shared memory)
  int64_t tiles;
  size_t total() const { return partial_bytes + ticket_bytes; }
};
SmallScratch small_scratch(const batq_weight* w, int64_t s) {
  SmallScratch sc{};
  sc.ntok = small_ntok(s);
  sc.splits = pick_splits(w->m, w->n, s, w->sm_count);
  sc.tiles = (w->m + 127) / 128;
  // the cluster reduction keeps its partial tiles in shared memory
  sc.cluster = cluster_reduce_ok(sc.tiles, sc.splits, 2 * static_cast<int64_t>(w->sm_count > 0 ? w->sm_count : 148), s);
  sc.partial_bytes = (sc.splits > 1 && !sc.cluster) ? round_up(static_cast<size_t>(sc.tiles) * sc.splits * sc.ntok * 128 * 4, 1024) : 0;
  sc.ticket_bytes = round_up(static_cast<size_t>(sc.tiles) * 4, 1024);
  return sc;
}

template <int NTOK, bool BF>
cudaError_t launch_small_kernel(dim3 grid, cudaStream_t stream, bool dependent, const CUtensorMap& tw,
                                const CUtensorMap& tx, const SmallParams& p) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kSmallThreads);
  cfg.dynamicSmemBytes = SmallCfg<NTOK>::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (p.cluster_reduce) {  // the K splits of a row tile as one cluster
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 1;
    attr[na].val.clusterDim.y = grid.y;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  if (dependent) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, gemm_small_s_kernel<NTOK, BF>, tw, tx, p);
}

// `dependent`: the kernel directly before this one on the stream is the activation quantiser
// (which releases its dependents early); the weight stream then starts while it still runs.
batq_status launch_gemm_small(const void* x_codes, const void* x_sf, const batq_weight* w, int64_t s, void* y,
                              int32_t y_dtype, int64_t ldy, uint8_t* scratch, const SmallScratch& sc,
                              cudaStream_t stream, bool dependent) {
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (w->device != dev) return BATQ_ERR_CUDA;
  CUtensorMap tmap_x;
  st = make_codes_tmap(&tmap_x, x_codes, s, w->n / 2, sc.ntok);
  if (st != BATQ_OK) return st;
  SmallParams p{};
  p.sfx = static_cast<const uint8_t*>(x_sf);
  p.sfw = w->scales;
  p.s = static_cast<int32_t>(s);
  p.m = static_cast<int32_t>(w->m);
  p.katoms = w->katoms;
  p.k_steps = static_cast<int32_t>((w->n + 255) / 256);
  p.splits = sc.splits;
  p.y = y;
  p.ldy = ldy;
  p.partial = reinterpret_cast<float*>(scratch);
  p.tickets = reinterpret_cast<uint32_t*>(scratch + sc.partial_bytes);
  p.cluster_reduce = sc.cluster ? 1 : 0;
  const dim3 grid(static_cast<unsigned>(sc.tiles), static_cast<unsigned>(sc.splits));
  const bool bf = y_dtype == BATQ_BF16;
  cudaError_t e;
#define BATQ_SMALL(NT) (bf ? launch_small_kernel<NT, true>(grid, stream, dependent, w->tmap_b128, tmap_x, p) \
                           : launch_small_kernel<NT, false>(grid, stream, dependent, w->tmap_b128, tmap_x, p))
  if (sc.ntok == 16) e = BATQ_SMALL(16);
  else if (sc.ntok == 32) e = BATQ_SMALL(32);
  else if (sc.ntok == 64) e = BATQ_SMALL(64);
  else e = BATQ_SMALL(128);
#undef BATQ_SMALL
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

// ---- fused small-s layer (quantiser inside the GEMM kernel) ------------------------------------
std::atomic<int> g_force_small_path{0};  // tuning hook: 0 = automatic, 1 = two kernels, 2 = fused whenever it applies
// K splits of the fused kernel: a power of two (the cluster size), at most 8, with at most
// kFusedMaxSteps K-steps per CTA; 0 if the shape does not fit.
int pick_fused_splits(int64_t m, int64_t n, int sm_count) {
  const int k_steps = static_cast<int>((n + 255) / 256);
  const int64_t tiles = (m + 127) / 128;
  const int64_t slots = 2 * static_cast<int64_t>(sm_count > 0 ? sm_count : 148);
  int best = 0;
  double best_cost = 1e30;
  const int force_splits = g_force_splits.load(std::memory_order_relaxed);
  for (int sp = 1; sp <= kFusedMaxSplits; sp *= 2) {
    if (sp > k_steps) break;
    const int per = (k_steps + sp - 1) / sp;
    if (per > kFusedMaxSteps) continue;
    if (force_splits > 0 && sp != force_splits) continue;
    const int64_t waves = (tiles * sp + slots - 1) / slots;
    const double cost = static_cast<double>(waves) * (per + 3.0) + 0.15 * sp;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = sp; }
  }
  return best;
}

// Automatic choice: every CTA of a K split requantises its slice of the activations, which is only
// hidden behind the weight stream while that is a few items per thread (tokens x K-steps <= 4) and
// the grid fits the SMs in one wave; measured, the fused kernel then saves about 5 % of a call.
bool use_fused_small(const batq_transform* t, const batq_weight* w, int64_t s) {
  const int force_path = g_force_small_path.load(std::memory_order_relaxed);
  if (force_path == 1 || s > kFusedTok) return false;
  if (!alu_small_geometry(t) || (t != nullptr && t->bf16_mid)) return false;  // its in-kernel quantiser: right factors of 8, 4, 2 columns, fp32
  const int sp = pick_fused_splits(w->m, w->n, w->sm_count);
  if (sp == 0) return false;
  if (force_path == 2) return true;
  const int64_t k_steps = (w->n + 255) / 256;
  const int64_t per = (k_steps + sp - 1) / sp;
  const int64_t slots = 2 * static_cast<int64_t>(w->sm_count > 0 ? w->sm_count : 148);
  return s * per <= 4 && ((w->m + 127) / 128) * sp <= slots;
}

batq_status launch_linear_fused(const batq_transform* t, const batq_weight* w, const void* x, int64_t s, int64_t ld,
                                void* y, int32_t y_dtype, int64_t ldy, cudaStream_t stream) {
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (w->device != dev || (t != nullptr && t->device != dev)) return BATQ_ERR_CUDA;
  FusedParams p{};
  p.x = static_cast<const uint16_t*>(x);
  p.ld = ld;
  p.s = static_cast<int32_t>(s);
  p.n = static_cast<int32_t>(w->n);
  p.k = w->k;
  if (t != nullptr) {
    p.left = t->d_left; p.right = t->d_right;
    p.left_stride = t->left_stride; p.right_stride = t->right_stride;
    p.clip_lo = t->d_clip_lo; p.clip_hi = t->d_clip_hi;
  }
  p.sfw = w->scales;
  p.m = static_cast<int32_t>(w->m);
  p.katoms = w->katoms;
  p.k_steps = static_cast<int32_t>((w->n + 255) / 256);
  p.splits = pick_fused_splits(w->m, w->n, w->sm_count);
  p.y = y;
  p.ldy = ldy;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>((w->m + 127) / 128), static_cast<unsigned>(p.splits));
  cfg.blockDim = dim3(kFusedThreads);
  cfg.dynamicSmemBytes = FusedCfg::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = static_cast<unsigned>(p.splits);
  attr[0].val.clusterDim.z = 1;
  // A programmatic dependent of whatever precedes it on the stream: its weight stream starts
  // while that still runs; x is read, and y written, after the wait inside the kernel.
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const int gc = t != nullptr ? t->gc : 8;
  const bool bf = y_dtype == BATQ_BF16;
  cudaError_t e;
  if (gc == 8)      e = bf ? cudaLaunchKernelEx(&cfg, linear_small_s_fused_kernel<true, 8>, w->tmap_b128, p)
                           : cudaLaunchKernelEx(&cfg, linear_small_s_fused_kernel<false, 8>, w->tmap_b128, p);
  else if (gc == 4) e = bf ? cudaLaunchKernelEx(&cfg, linear_small_s_fused_kernel<true, 4>, w->tmap_b128, p)
                           : cudaLaunchKernelEx(&cfg, linear_small_s_fused_kernel<false, 4>, w->tmap_b128, p);
  else              e = bf ? cudaLaunchKernelEx(&cfg, linear_small_s_fused_kernel<true, 2>, w->tmap_b128, p)
                           : cudaLaunchKernelEx(&cfg, linear_small_s_fused_kernel<false, 2>, w->tmap_b128, p);
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

// ---- prefill layer in one kernel (quantise phase + GEMM phase on one grid of CTA pairs) --------
std::atomic<int> g_force_prefill_path{0};  // tuning hook: 0 = automatic, 1 = two kernels, 2 = one kernel wherever it applies
std::atomic<unsigned long long> g_call_tag{1};  // tags the readiness counters of one call; never reused within a process

// a run counter and one flag word per CTA of the grid (at most one CTA per SM)
inline size_t prefill_flag_bytes(const batq_weight* w) { return round_up(static_cast<size_t>(std::max(w->sm_count, 148) + 1) * 8, 1024); }

// Applies to what the CTA-pair GEMM takes (s > 128, m >= 192) with a transform whose scale atoms
// come in pairs (k % 8 == 0: no padding atom to keep finite).
bool fused_prefill_applies(const batq_transform* t, const batq_weight* w, int64_t s) {
  return t != nullptr && !t->bf16_mid && s > 128 && w->m >= 192 && w->k % 8 == 0 &&
         g_force_gemm_kernel.load(std::memory_order_relaxed) != 1 && g_force_quantizer.load(std::memory_order_relaxed) == 0;
}
bool use_fused_prefill(const batq_transform* t, const batq_weight* w, int64_t s) {
  const int f = g_force_prefill_path.load(std::memory_order_relaxed);
  if (f == 1 || !fused_prefill_applies(t, w, s)) return false;
  return f == 2;
}

batq_status launch_linear_prefill_fused(const batq_transform* t, const batq_weight* w, const void* x, int64_t s, int64_t ld,
                                        void* y, int32_t y_dtype, int64_t ldy, uint8_t* codes, uint8_t* sf, uint8_t* ready,
                                        cudaStream_t stream) {
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (w->device != dev || t->device != dev) return BATQ_ERR_CUDA;
  const bool bf = y_dtype == BATQ_BF16;
  const int64_t n = w->n;
  CUtensorMap tmap_x, tmap_codes, tmap_a, tmap_sfa, tmap_y;
  std::memset(&tmap_y, 0, sizeof(tmap_y));
  st = make_tmap_2d(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x, n, s, ld * 2, 64, kQtRows, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st == BATQ_OK)
    st = make_tmap_2d(&tmap_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes, n / 2, s, n / 2, 64, kQtRows, CU_TENSOR_MAP_SWIZZLE_64B);
  if (st == BATQ_OK) st = make_codes_tmap(&tmap_a, codes, s, n / 2, kBM);
  if (st == BATQ_OK) st = make_sf_tmap(&tmap_sfa, sf, (s + 127) / 128, w->katoms);
  const int64_t m16 = w->m / (bf ? 8 : 4) * (bf ? 8 : 4);
  if (st == BATQ_OK && m16 > 0) st = make_y_tmap(&tmap_y, y, s, m16, ldy, bf);
  if (st != BATQ_OK) return st;
  PrefillFusedParams q{};
  int pairs = 0;
  double sched_us = 0.0;
  if (!pair_schedule_cached(w, s, info->sm_count, false, &q.g, &pairs, &sched_us)) return BATQ_ERR_SHAPE;
  q.g.katoms = w->katoms;
  q.g.k_steps = static_cast<int32_t>((n + 255) / 256);
  q.g.m16 = static_cast<int32_t>(m16);
  q.g.y = y;
  q.g.ldy = ldy;
  q.n = static_cast<int32_t>(n);
  q.k = w->k;
  q.n_strips = w->k / kQtGroups;
  q.n_row_tiles = static_cast<int32_t>((s + 127) / 128);
  q.n_units = q.g.m_pairs * q.n_strips;
  q.clip_lo = t->d_clip_lo;
  q.clip_hi = t->d_clip_hi;
  q.scales = sf;
  q.sync = reinterpret_cast<unsigned long long*>(ready);
  q.tag = g_call_tag.fetch_add(1, std::memory_order_relaxed) & ((1ull << 40) - 1ull);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs));
  cfg.blockDim = dim3(kPfThreads);
  cfg.dynamicSmemBytes = kPfSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // A programmatic dependent of whatever precedes it on the stream: its CTAs take over the SMs that
  // kernel has left and wait, inside the kernel, before they read x.
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaError_t e;
#define BATQ_PF(CL, BF) cudaLaunchKernelEx(&cfg, linear_prefill_fused_kernel<CL, BF>, tmap_x, t->tmap_pimg, tmap_codes, tmap_a, \
                                           w->tmap_b32, tmap_sfa, w->tmap_sf, tmap_y, q)
  if (t->has_clip) e = bf ? BATQ_PF(true, true) : BATQ_PF(true, false);
  else e = bf ? BATQ_PF(false, true) : BATQ_PF(false, false);
#undef BATQ_PF
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

// ---- W4A8: MXFP8 activations x MXFP4 weights --------------------------------------------------
// Bytes one weight row of a K-step adds to the mbarrier's transaction count: 128 four-bit codes
// are 64 bytes in global memory and land in 128 bytes of shared memory (8 data bytes at the start
// of every 16-byte slot, the other 8 left untouched); the copy reports the 64 bytes it moved.
constexpr int kU4RowTxBytes = 64;

batq_status launch_gemm_w4a8(const void* x_codes8, const void* x_sf, const batq_weight* w, int64_t s, void* y,
                             int32_t y_dtype, int64_t ldy, cudaStream_t stream, bool dependent) {
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (w->device != dev) return BATQ_ERR_CUDA;
  if (!w->has_u4) return BATQ_ERR_UNSUPPORTED;
  const bool bf = y_dtype == BATQ_BF16;
  CUtensorMap tmap_a, tmap_y;
  std::memset(&tmap_y, 0, sizeof(tmap_y));
  st = make_tmap_2d(&tmap_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, x_codes8, w->n, s, w->n, 128, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
  const int64_t m16 = w->m / (bf ? 8 : 4) * (bf ? 8 : 4);
  if (st == BATQ_OK && m16 > 0) st = make_y_tmap(&tmap_y, y, s, m16, ldy, bf);
  if (st != BATQ_OK) return st;
  // CTA pairs above 128 tokens (two 128-token tiles to share a weight tile), as in the W4A4 GEMM:
  // tiles of up to 256 features on two accumulators, or tiles of up to 448 on one.  kind::mxf8f6f4
  // runs at half the rate of kind::mxf4, so the wide tile (fewer bytes per flop, tensor-bound) is
  // the rule here; the two-accumulator kernel keeps the layers where a pair has at most two tiles
  // whichever way the features are cut.
  const int force_gemm = g_force_gemm_kernel.load(std::memory_order_relaxed);
  if (force_gemm == 2 || force_gemm == 3 || (force_gemm == 0 && s > 128 && w->m >= 192)) {
    CUtensorMap tmap_sfa, tmap_y64;
    std::memset(&tmap_y64, 0, sizeof(tmap_y64));
    st = make_sf_tmap(&tmap_sfa, x_sf, (s + 127) / 128, w->katoms, 1);
    if (st != BATQ_OK) return st;
    const int force_bn = g_force_bn.load(std::memory_order_relaxed);
    const bool forced_w = force_bn >= 64 && force_bn <= kWideMaxBn && force_bn % 64 == 0;
    PairParams p{}, pw{};
    int pairs = 0, pairs_w = 0;
    double us = 0.0, us_w = 0.0;
    bool wide = false;
    if (force_gemm == 3) {
      if (force_bn != 0 && !forced_w) return BATQ_ERR_SHAPE;
      if (!pair_schedule_cached(w, s, info->sm_count, true, &pw, &pairs_w, &us_w, true)) return BATQ_ERR_SHAPE;
      wide = true;
    } else {
      if (!pair_schedule_cached(w, s, info->sm_count, false, &p, &pairs, &us)) return BATQ_ERR_SHAPE;
      if (force_gemm == 0 && force_bn == 0 && w->m >= 320 &&
          pair_schedule_cached(w, s, info->sm_count, true, &pw, &pairs_w, &us_w, true)) {
        // four or more tiles for some pair in the two-accumulator schedule: take the wide tiles
        // (measured at 2048 tokens: gate/up, 14 tiles, 158 against 172 us; qkv, 3 tiles, 39.5 against 37.3)
        int max_tiles = 0;
        for (int pr = 0; pr < pairs; ++pr) {
          PairWalk walk(p, pr, pairs);
          PairTile t;
          int cnt = 0;
          while (walk.next(t)) ++cnt;
          max_tiles = std::max(max_tiles, cnt);
        }
        wide = max_tiles >= 4;
      }
    }
    if (wide) {
      p = pw;
      pairs = pairs_w;
      if (m16 > 0) {
        st = make_y_tmap(&tmap_y64, y, s, m16, ldy, bf, 64);
        if (st != BATQ_OK) return st;
      }
    }
    p.katoms = w->katoms;
    p.k_steps = static_cast<int32_t>(w->n / kW4A8KElems);
    p.m16 = static_cast<int32_t>(m16);
    p.y = y;
    p.ldy = ldy;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs));
    cfg.blockDim = dim3(wide ? kWideThreads : kPairThreads);
    cfg.dynamicSmemBytes = wide ? A8WideCfg::kSmemBytes : A8PairCfg::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    cudaError_t e;
    if (wide)
      e = bf ? cudaLaunchKernelEx(&cfg, gemm_w4a8_wide_kernel<true>, tmap_a, w->tmap_u4_32, tmap_sfa, w->tmap_sf1, tmap_y64, p)
             : cudaLaunchKernelEx(&cfg, gemm_w4a8_wide_kernel<false>, tmap_a, w->tmap_u4_32, tmap_sfa, w->tmap_sf1, tmap_y64, p);
    else
      e = bf ? cudaLaunchKernelEx(&cfg, gemm_w4a8_pair_kernel<true>, tmap_a, w->tmap_u4_32, tmap_sfa, w->tmap_sf1, tmap_y, p)
             : cudaLaunchKernelEx(&cfg, gemm_w4a8_pair_kernel<false>, tmap_a, w->tmap_u4_32, tmap_sfa, w->tmap_sf1, tmap_y, p);
    if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
    return BATQ_OK;
  }
  // One CTA per tile.  Tile width: 256 (half the operand bytes per flop of a 128-wide tile; measured 16 % faster on
  // the config-1 shapes at equal wave counts) unless 128-wide tiles need clearly fewer waves' worth
  // of time (a layer too small to fill the SMs with 256-wide tiles).
  const int64_t mt = (s + kBM - 1) / kBM;
  auto waves = [&](int bn) { return ((mt * ((w->m + bn - 1) / bn)) + info->sm_count - 1) / info->sm_count; };
  const int force_bn = g_force_bn.load(std::memory_order_relaxed);
  int bn = (w->m <= 128 || waves(128) * 128 * 1.2 < waves(256) * 256) ? 128 : 256;
  if (force_bn == 128 || force_bn == 256) bn = force_bn;
  W4A8Params p{};
  p.sfa = static_cast<const uint8_t*>(x_sf);
  p.sfb = w->scales;
  p.s = static_cast<int32_t>(s);
  p.m = static_cast<int32_t>(w->m);
  p.katoms = w->katoms;
  p.k_steps = static_cast<int32_t>(w->n / kW4A8KElems);
  p.m_tiles = static_cast<int32_t>(mt);
  p.n_tiles = static_cast<int32_t>((w->m + bn - 1) / bn);
  p.sfb_row_tiles = static_cast<int32_t>((w->m + 127) / 128);
  p.m16 = static_cast<int32_t>(m16);
  p.b_row_tx = kU4RowTxBytes;
  p.y = y;
  p.ldy = ldy;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(std::min<int64_t>(info->sm_count, static_cast<int64_t>(p.m_tiles) * p.n_tiles)));
  cfg.blockDim = dim3(kGemmThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  cudaError_t e;
  if (bn == 256) {
    cfg.dynamicSmemBytes = W4A8Cfg<256>::kSmemBytes;
    e = bf ? cudaLaunchKernelEx(&cfg, gemm_w4a8_kernel<256, true>, tmap_a, w->tmap_u4_256, tmap_y, p)
           : cudaLaunchKernelEx(&cfg, gemm_w4a8_kernel<256, false>, tmap_a, w->tmap_u4_256, tmap_y, p);
  } else {
    cfg.dynamicSmemBytes = W4A8Cfg<128>::kSmemBytes;
    e = bf ? cudaLaunchKernelEx(&cfg, gemm_w4a8_kernel<128, true>, tmap_a, w->tmap_u4_128, tmap_y, p)
           : cudaLaunchKernelEx(&cfg, gemm_w4a8_kernel<128, false>, tmap_a, w->tmap_u4_128, tmap_y, p);
  }
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

batq_status check_y(const void* y, int32_t y_dtype, int64_t ldy, int64_t m) {
  if (y_dtype != BATQ_F32 && y_dtype != BATQ_BF16) return BATQ_ERR_UNSUPPORTED;
  if (ldy < m) return BATQ_ERR_SHAPE;
  if (!aligned(y, 16) || ldy % (y_dtype == BATQ_F32 ? 4 : 8) != 0) return BATQ_ERR_ALIGN;
  return BATQ_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------
// exported functions
// ------------------------------------------------------------------------------------
extern "C" {

const char* batq_status_string(batq_status s) {
  switch (s) {
    case BATQ_OK: return "ok";
    case BATQ_ERR_NULL: return "null pointer";
    case BATQ_ERR_SHAPE: return "bad shape";
    case BATQ_ERR_ALIGN: return "bad alignment";
    case BATQ_ERR_UNSUPPORTED: return "unsupported";
    case BATQ_ERR_WORKSPACE: return "workspace too small";
    case BATQ_ERR_SINGULAR: return "singular transform factor";
    case BATQ_ERR_CUDA: return "CUDA error";
    case BATQ_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

int batq_version(void) { return 100; }

batq_status batq_transform_create(batq_transform** out, int32_t n, int32_t gr, int32_t gc, const float* left,
                                  int64_t left_stride, const float* right, int64_t right_stride,
                                  const float* clip_lo, const float* clip_hi) {
  if (out == nullptr) return BATQ_ERR_NULL;
  *out = nullptr;
  if (left == nullptr || right == nullptr) return BATQ_ERR_NULL;
  if ((clip_lo == nullptr) != (clip_hi == nullptr)) return BATQ_ERR_NULL;
  if (n <= 0 || n % 32 != 0 || gr <= 0 || gc <= 0 || gr * gc != 32) return BATQ_ERR_SHAPE;
  if ((left_stride != 0 && left_stride != gr * gr) || (right_stride != 0 && right_stride != gc * gc)) return BATQ_ERR_SHAPE;
  int dev;
  batq_status st = device_setup(&dev, nullptr);
  if (st != BATQ_OK) return st;
  batq_transform* t = new (std::nothrow) batq_transform();
  if (t == nullptr) return BATQ_ERR_CUDA;
  t->device = dev;
  t->n = n; t->k = n / 32; t->gr = gr; t->gc = gc;
  t->left_stride = static_cast<int32_t>(left_stride);
  t->right_stride = static_cast<int32_t>(right_stride);
  t->has_clip = clip_lo != nullptr;
  t->bf16_mid = false;
  const size_t nl = static_cast<size_t>(left_stride ? t->k : 1) * gr * gr;
  const size_t nr = static_cast<size_t>(right_stride ? t->k : 1) * gc * gc;
  t->left.assign(left, left + nl);
  t->right.assign(right, right + nr);
  t->d_left = t->d_right = t->d_clip_lo = t->d_clip_hi = nullptr;
  t->d_pimg = nullptr;
  std::vector<uint8_t> pimg;
  build_block_images(t, &pimg);
  cudaError_t e = cudaMalloc(&t->d_left, nl * sizeof(float));
  e = e ? e : cudaMalloc(&t->d_pimg, pimg.size());
  e = e ? e : cudaMemcpy(t->d_pimg, pimg.data(), pimg.size(), cudaMemcpyHostToDevice);
  e = e ? e : cudaMalloc(&t->d_right, nr * sizeof(float));
  e = e ? e : cudaMemcpy(t->d_left, left, nl * sizeof(float), cudaMemcpyHostToDevice);
  e = e ? e : cudaMemcpy(t->d_right, right, nr * sizeof(float), cudaMemcpyHostToDevice);
  if (t->has_clip) {
    e = e ? e : cudaMalloc(&t->d_clip_lo, t->k * sizeof(float));
    e = e ? e : cudaMalloc(&t->d_clip_hi, t->k * sizeof(float));
    e = e ? e : cudaMemcpy(t->d_clip_lo, clip_lo, t->k * sizeof(float), cudaMemcpyHostToDevice);
    e = e ? e : cudaMemcpy(t->d_clip_hi, clip_hi, t->k * sizeof(float), cudaMemcpyHostToDevice);
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    batq_transform_destroy(t);
    return BATQ_ERR_CUDA;
  }
  {
    // the block-matrix images seen as [k blocks][3 terms][2 halves][256 words]
    const cuuint64_t dims[4] = {256, 2, 3, static_cast<cuuint64_t>(t->k)};
    const cuuint64_t strides[3] = {1024, 2048, static_cast<cuuint64_t>(kQtImageBytes)};
    const cuuint32_t box[4] = {256, 1, 3, static_cast<cuuint32_t>(kQtGroups)};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (g_encode_tiled(&t->tmap_pimg, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, t->d_pimg, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      batq_transform_destroy(t);
      return BATQ_ERR_CUDA;
    }
  }
  *out = t;
  return BATQ_OK;
}

batq_status batq_transform_set_bf16_intermediates(batq_transform* t, int32_t on) {
  if (t == nullptr) return BATQ_ERR_NULL;
  if (on != 0 && (t->gr != 4 || t->gc != 8)) return BATQ_ERR_UNSUPPORTED;
  t->bf16_mid = on != 0;
  return BATQ_OK;
}

batq_status batq_transform_destroy(batq_transform* t) {
  if (t == nullptr) return BATQ_OK;
  cudaFree(t->d_left);
  cudaFree(t->d_right);
  cudaFree(t->d_clip_lo);
  cudaFree(t->d_clip_hi);
  cudaFree(t->d_pimg);
  delete t;
  return BATQ_OK;
}

size_t batq_sf_bytes(int64_t rows, int64_t n, int32_t layout) {
  if (rows < 0 || n <= 0 || n % 32 != 0) return 0;
  const int64_t k = n / 32;
  if (layout == BATQ_SF_ROWMAJOR) return static_cast<size_t>(rows * k);
  if (layout == BATQ_SF_MMA) return static_cast<size_t>((rows + 127) / 128) * katoms_of(k) * 512;
  return 0;
}

batq_status batq_quantize_act(const batq_transform* t, const void* x_bf16, int64_t s, int64_t n, int64_t ld,
                              void* codes, void* scales, int32_t scale_layout, void* stream) {
  batq_status st = check_x(x_bf16, s, n, ld);
  if (st != BATQ_OK) return st;
  if (t != nullptr && t->n != n) return BATQ_ERR_SHAPE;
  if (scale_layout != BATQ_SF_ROWMAJOR && scale_layout != BATQ_SF_MMA) return BATQ_ERR_UNSUPPORTED;
  if (s == 0) return BATQ_OK;
  if (codes == nullptr || scales == nullptr) return BATQ_ERR_NULL;
  if (!aligned(codes, 16) || (scale_layout == BATQ_SF_MMA && !aligned(scales, 16))) return BATQ_ERR_ALIGN;
  return launch_quantize(t, x_bf16, s, n, ld, codes, scales, scale_layout, nullptr, static_cast<cudaStream_t>(stream));
}

batq_status batq_quantize_act_mxfp8(const batq_transform* t, const void* x_bf16, int64_t s, int64_t n, int64_t ld,
                                    void* codes, void* scales, int32_t scale_layout, void* stream) {
  batq_status st = check_x(x_bf16, s, n, ld);
  if (st != BATQ_OK) return st;
  if (t == nullptr) return BATQ_ERR_NULL;
  if (t->n != n) return BATQ_ERR_SHAPE;
  if (t->bf16_mid) return BATQ_ERR_UNSUPPORTED;   // the 8-bit quantiser has the dense form only
  if (scale_layout != BATQ_SF_ROWMAJOR && scale_layout != BATQ_SF_MMA) return BATQ_ERR_UNSUPPORTED;
  if (s == 0) return BATQ_OK;
  if (codes == nullptr || scales == nullptr) return BATQ_ERR_NULL;
  if (!aligned(codes, 16) || (scale_layout == BATQ_SF_MMA && !aligned(scales, 16))) return BATQ_ERR_ALIGN;
  int dev;
  const DeviceInfo* info;
  st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (t->device != dev) return BATQ_ERR_CUDA;
  return launch_quantize_tc(t, x_bf16, s, n, ld, codes, scales, scale_layout, nullptr,
                            static_cast<cudaStream_t>(stream), info->sm_count, true);
}

batq_status batq_debug_transform_clip_f32(const batq_transform* t, const void* x_bf16, int64_t s, int64_t n,
                                          int64_t ld, float* out, void* stream) {
  batq_status st = check_x(x_bf16, s, n, ld);
  if (st != BATQ_OK) return st;
  if (t != nullptr && t->n != n) return BATQ_ERR_SHAPE;
  if (s == 0) return BATQ_OK;
  if (out == nullptr) return BATQ_ERR_NULL;
  if (!aligned(out, 16)) return BATQ_ERR_ALIGN;
  return launch_quantize(t, x_bf16, s, n, ld, nullptr, nullptr, BATQ_SF_ROWMAJOR, out, static_cast<cudaStream_t>(stream));
}

// The tensor maps every GEMM kernel takes over a prepared weight's codes and scales.
static batq_status weight_tensor_maps(batq_weight* w) {
  const int64_t m = w->m, n = w->n;
  batq_status st = make_codes_tmap(&w->tmap_b256, w->codes, m, n / 2, 256);
  if (st == BATQ_OK) st = make_codes_tmap(&w->tmap_b192, w->codes, m, n / 2, 192);
  if (st == BATQ_OK) st = make_codes_tmap(&w->tmap_b128, w->codes, m, n / 2, 128);
  if (st == BATQ_OK) st = make_codes_tmap(&w->tmap_b64, w->codes, m, n / 2, 64);
  if (st == BATQ_OK) st = make_codes_tmap(&w->tmap_b32, w->codes, m, n / 2, 32);
  if (st == BATQ_OK) st = make_sf_tmap(&w->tmap_sf, w->scales, (m + 127) / 128, w->katoms);
  w->has_u4 = n % 128 == 0;
  if (st == BATQ_OK && w->has_u4) st = make_u4_unpack_tmap(&w->tmap_u4_128, w->codes, m, n, 128);
  if (st == BATQ_OK && w->has_u4) st = make_u4_unpack_tmap(&w->tmap_u4_256, w->codes, m, n, 256);
  if (st == BATQ_OK && w->has_u4) st = make_u4_unpack_tmap(&w->tmap_u4_32, w->codes, m, n, 32);
  if (st == BATQ_OK && w->has_u4) st = make_sf_tmap(&w->tmap_sf1, w->scales, (m + 127) / 128, w->katoms, 1);
  return st;
}

size_t batq_weight_bytes(int64_t m, int64_t n) {
  if (m <= 0 || n <= 0 || n % 32 != 0) return 0;
  return round_up(static_cast<size_t>(m * (n / 2)), 1024) + batq_sf_bytes(m, n, BATQ_SF_MMA);
}

batq_status batq_prepare_weight(const batq_transform* t, const void* w_bf16, int64_t m, int64_t n, int64_t ld,
                                const float* w_clip_lo, const float* w_clip_hi, void* weight_buf, batq_weight** out,
                                void* stream) {
  if (out == nullptr) return BATQ_ERR_NULL;
  *out = nullptr;
  if (m <= 0 || m > (int64_t(1) << 24)) return BATQ_ERR_SHAPE;
  batq_status st = check_x(w_bf16, m, n, ld);
  if (st != BATQ_OK) return st;
  if (weight_buf == nullptr) return BATQ_ERR_NULL;
  if ((w_clip_lo == nullptr) != (w_clip_hi == nullptr)) return BATQ_ERR_NULL;
  if (!aligned(weight_buf, 1024)) return BATQ_ERR_ALIGN;
  if (t != nullptr && t->n != n) return BATQ_ERR_SHAPE;
  int dev;
  const DeviceInfo* dinfo;
  st = device_setup(&dev, &dinfo);
  if (st != BATQ_OK) return st;
  if (t != nullptr && t->device != dev) return BATQ_ERR_CUDA;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int32_t k = static_cast<int32_t>(n / 32);

  // L' = L^-T and R' = R^-T in fp64: W~_blk = L^-1 Wv R^-T = L'^T Wv R'.
  double* d_fac = nullptr;
  size_t nl = 0, nr = 0;
  if (t != nullptr) {
    const size_t cl = t->left_stride ? k : 1, cr = t->right_stride ? k : 1;
    const int gr = t->gr, gc = t->gc;
    nl = cl * gr * gr; nr = cr * gc * gc;
    std::vector<double> fac(nl + nr);
    double a[1024], inv[1024];
    for (size_t i = 0; i < cl; ++i) {
      for (int e = 0; e < gr * gr; ++e) a[e] = t->left[i * gr * gr + e];
      if (!invert_small(a, gr, inv)) return BATQ_ERR_SINGULAR;
      for (int r = 0; r < gr; ++r)
        for (int c = 0; c < gr; ++c) fac[i * gr * gr + r * gr + c] = inv[c * gr + r];
    }
    for (size_t i = 0; i < cr; ++i) {
      for (int e = 0; e < gc * gc; ++e) a[e] = t->right[i * gc * gc + e];
      if (!invert_small(a, gc, inv)) return BATQ_ERR_SINGULAR;
      for (int r = 0; r < gc; ++r)
        for (int c = 0; c < gc; ++c) fac[nl + i * gc * gc + r * gc + c] = inv[c * gc + r];
    }
    if (cudaMalloc(&d_fac, fac.size() * sizeof(double)) != cudaSuccess ||
        cudaMemcpyAsync(d_fac, fac.data(), fac.size() * sizeof(double), cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaStreamSynchronize(cs) != cudaSuccess) {
      cudaGetLastError();
      cudaFree(d_fac);
      return BATQ_ERR_CUDA;
    }
  }
  batq_weight* w = new (std::nothrow) batq_weight();
  if (w == nullptr) { cudaFree(d_fac); return BATQ_ERR_CUDA; }
  w->device = dev;
  w->m = m; w->n = n; w->k = k; w->katoms = katoms_of(k);
  w->sm_count = dinfo->sm_count;
  w->codes = static_cast<uint8_t*>(weight_buf);
  w->scales = w->codes + round_up(static_cast<size_t>(m * (n / 2)), 1024);

  PrepWeightParams p{};
  p.w = static_cast<const uint16_t*>(w_bf16);
  p.ld = ld; p.m = m; p.n = static_cast<int32_t>(n); p.k = k;
  if (t != nullptr) {
    p.left = d_fac; p.right = d_fac + nl;
    p.left_stride = t->left_stride; p.right_stride = t->right_stride;
    p.gr = t->gr; p.gc = t->gc;
  }
  p.clip_lo = w_clip_lo; p.clip_hi = w_clip_hi;
  p.codes = w->codes; p.scales = w->scales; p.katoms = w->katoms;
  const int64_t items = m * k;
  prepare_weight_kernel<<<static_cast<unsigned>((items + 127) / 128), 128, 0, cs>>>(p);
  cudaError_t e = cudaGetLastError();
  e = e ? e : cudaStreamSynchronize(cs);
  cudaFree(d_fac);
  if (e != cudaSuccess) { cudaGetLastError(); delete w; return BATQ_ERR_CUDA; }
  st = weight_tensor_maps(w);
  if (st != BATQ_OK) { delete w; return st; }
  *out = w;
  return BATQ_OK;
}

batq_status batq_weight_import(const void* codes_rowmajor, const void* scales_rowmajor, int64_t m, int64_t n,
                               void* weight_buf, batq_weight** out, void* stream) {
  if (out == nullptr) return BATQ_ERR_NULL;
  *out = nullptr;
  if (m <= 0 || m > (int64_t(1) << 24) || n <= 0 || n % 32 != 0 || n > (int64_t(1) << 24)) return BATQ_ERR_SHAPE;
  if (codes_rowmajor == nullptr || scales_rowmajor == nullptr || weight_buf == nullptr) return BATQ_ERR_NULL;
  if (!aligned(weight_buf, 1024)) return BATQ_ERR_ALIGN;
  int dev;
  const DeviceInfo* dinfo;
  batq_status st = device_setup(&dev, &dinfo);
  if (st != BATQ_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  batq_weight* w = new (std::nothrow) batq_weight();
  if (w == nullptr) return BATQ_ERR_CUDA;
  w->device = dev;
  w->m = m; w->n = n; w->k = static_cast<int32_t>(n / 32); w->katoms = katoms_of(w->k);
  w->sm_count = dinfo->sm_count;
  w->codes = static_cast<uint8_t*>(weight_buf);
  const size_t code_bytes = static_cast<size_t>(m * (n / 2));
  w->scales = w->codes + round_up(code_bytes, 1024);
  const int64_t items = m * w->k;
  // padded rows and blocks of the scale layout must hold finite scales: zero everything first
  cudaError_t e = cudaMemsetAsync(w->codes + code_bytes, 0, batq_weight_bytes(m, n) - code_bytes, cs);
  e = e ? e : cudaMemcpyAsync(w->codes, codes_rowmajor, code_bytes, cudaMemcpyDeviceToDevice, cs);
  if (e == cudaSuccess) {
    import_scales_kernel<<<static_cast<unsigned>((items + 255) / 256), 256, 0, cs>>>(
        static_cast<const uint8_t*>(scales_rowmajor), w->scales, m, w->k, w->katoms);
    e = cudaGetLastError();
  }
  e = e ? e : cudaStreamSynchronize(cs);
  if (e != cudaSuccess) { cudaGetLastError(); delete w; return BATQ_ERR_CUDA; }
  st = weight_tensor_maps(w);
  if (st != BATQ_OK) { delete w; return st; }
  *out = w;
  return BATQ_OK;
}

batq_status batq_weight_destroy(batq_weight* w) {
  delete w;
  return BATQ_OK;
}

batq_status batq_weight_export(const batq_weight* w, void* codes_rowmajor, void* scales_rowmajor, void* stream) {
  if (w == nullptr || codes_rowmajor == nullptr || scales_rowmajor == nullptr) return BATQ_ERR_NULL;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(codes_rowmajor, w->codes, static_cast<size_t>(w->m * (w->n / 2)), cudaMemcpyDeviceToDevice, cs) !=
      cudaSuccess) {
    cudaGetLastError();
    return BATQ_ERR_CUDA;
  }
  const int64_t items = w->m * w->k;
  export_scales_kernel<<<static_cast<unsigned>((items + 255) / 256), 256, 0, cs>>>(
      w->scales, static_cast<uint8_t*>(scales_rowmajor), w->m, w->k, w->katoms);
  return cudaGetLastError() == cudaSuccess ? BATQ_OK : BATQ_ERR_CUDA;
}

batq_status batq_gemm_mxfp4(const void* x_codes, const void* x_scales_mma, const batq_weight* w, int64_t s, void* y,
                            int32_t y_dtype, int64_t ldy, void* stream) {
  if (w == nullptr) return BATQ_ERR_NULL;
  if (s < 0 || s > (int64_t(1) << 30)) return BATQ_ERR_SHAPE;
  if (s == 0) return BATQ_OK;
  if (x_codes == nullptr || x_scales_mma == nullptr || y == nullptr) return BATQ_ERR_NULL;
  if (!aligned(x_codes, 16) || !aligned(x_scales_mma, 16)) return BATQ_ERR_ALIGN;
  batq_status st = check_y(y, y_dtype, ldy, w->m);
  if (st != BATQ_OK) return st;
  return launch_gemm(x_codes, x_scales_mma, w, s, y, y_dtype, ldy, static_cast<cudaStream_t>(stream));
}

batq_status batq_gemm_mxfp8_mxfp4(const void* x_codes8, const void* x_scales_mma, const batq_weight* w, int64_t s, void* y,
                                  int32_t y_dtype, int64_t ldy, void* stream) {
  if (w == nullptr) return BATQ_ERR_NULL;
  if (s < 0 || s > (int64_t(1) << 30)) return BATQ_ERR_SHAPE;
  if (!w->has_u4) return BATQ_ERR_UNSUPPORTED;
  if (s == 0) return BATQ_OK;
  if (x_codes8 == nullptr || x_scales_mma == nullptr || y == nullptr) return BATQ_ERR_NULL;
  if (!aligned(x_codes8, 16) || !aligned(x_scales_mma, 16)) return BATQ_ERR_ALIGN;
  batq_status st = check_y(y, y_dtype, ldy, w->m);
  if (st != BATQ_OK) return st;
  return launch_gemm_w4a8(x_codes8, x_scales_mma, w, s, y, y_dtype, ldy, static_cast<cudaStream_t>(stream), false);
}

size_t batq_linear_w4a8_workspace_bytes(const batq_weight* w, int64_t s) {
  if (w == nullptr || s < 0) return 0;
  return round_up(static_cast<size_t>(s * w->n), 1024) + round_up(batq_sf_bytes(s, w->n, BATQ_SF_MMA), 1024);
}

batq_status batq_linear_w4a8(const batq_transform* t, const batq_weight* w, const void* x_bf16, int64_t s, int64_t ld,
                             void* y, int32_t y_dtype, int64_t ldy, void* workspace, size_t workspace_bytes,
                             void* stream) {
  if (w == nullptr || t == nullptr) return BATQ_ERR_NULL;
  batq_status st = check_x(x_bf16, s, w->n, ld);
  if (st != BATQ_OK) return st;
  if (t->n != w->n) return BATQ_ERR_SHAPE;
  if (!w->has_u4 || t->bf16_mid) return BATQ_ERR_UNSUPPORTED;
  if (s == 0) return BATQ_OK;
  if (y == nullptr || workspace == nullptr) return BATQ_ERR_NULL;
  st = check_y(y, y_dtype, ldy, w->m);
  if (st != BATQ_OK) return st;
  if (!aligned(workspace, 1024)) return BATQ_ERR_ALIGN;
  if (workspace_bytes < batq_linear_w4a8_workspace_bytes(w, s)) return BATQ_ERR_WORKSPACE;
  int dev;
  const DeviceInfo* info;
  st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (t->device != dev || w->device != dev) return BATQ_ERR_CUDA;
  uint8_t* codes = static_cast<uint8_t*>(workspace);
  uint8_t* sf = codes + round_up(static_cast<size_t>(s * w->n), 1024);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  st = launch_quantize_tc(t, x_bf16, s, w->n, ld, codes, sf, BATQ_SF_MMA, nullptr, cs, info->sm_count, true);
  if (st != BATQ_OK) return st;
  return launch_gemm_w4a8(codes, sf, w, s, y, y_dtype, ldy, cs, true);
}

size_t batq_gemm_small_s_scratch_bytes(const batq_weight* w, int64_t s) {
  if (w == nullptr || s <= 0 || s > kSmallSMax) return 0;
  return small_scratch(w, s).total();
}

batq_status batq_gemm_mxfp4_small_s(const void* x_codes, const void* x_scales_mma, const batq_weight* w, int64_t s,
                                    void* y, int32_t y_dtype, int64_t ldy, void* scratch, size_t scratch_bytes,
                                    void* stream) {
  if (w == nullptr) return BATQ_ERR_NULL;
  if (s < 0 || s > kSmallSMax) return BATQ_ERR_SHAPE;
  if (s == 0) return BATQ_OK;
  if (x_codes == nullptr || x_scales_mma == nullptr || y == nullptr || scratch == nullptr) return BATQ_ERR_NULL;
  if (!aligned(x_codes, 16) || !aligned(x_scales_mma, 16) || !aligned(scratch, 1024)) return BATQ_ERR_ALIGN;
  batq_status st = check_y(y, y_dtype, ldy, w->m);
  if (st != BATQ_OK) return st;
  const SmallScratch sc = small_scratch(w, s);
  if (scratch_bytes < sc.total()) return BATQ_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint8_t* sp = static_cast<uint8_t*>(scratch);
  if (cudaMemsetAsync(sp + sc.partial_bytes, 0, sc.ticket_bytes, cs) != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return launch_gemm_small(x_codes, x_scales_mma, w, s, y, y_dtype, ldy, sp, sc, cs, false);
}

// The whole layer takes the small-s path (per-block quantiser + swapped-operand split-K GEMM) up
// to 32 tokens, and up to 128 where the layer is large enough for the weight stream to dominate
// (>= 40 M weights, e.g. 4096 x 14336).  The path's cost grows with the tokens (split-K reduction
// of tokens x 128 partial sums per CTA), while the one-CTA-per-tile GEMM behind the same per-block
// quantiser costs about the same from 33 to 128 tokens.  Measured, 4096 -> 6144 at 32 / 48 / 64 /
// 96 / 128 tokens: 9.0 / 10.4 / 11.4 / 14.1 / 16.0 us on the small-s path, 9.7 / 8.8 / 9.6 / 10.1 us
// from 48 tokens on the other; 4096 -> 28672 at 96 tokens: 17.9 against 19.5 us.
static bool layer_takes_small_path(const batq_weight* w, int64_t s) {
  return s <= 32 || (s <= kSmallSMax && w->m * w->n >= 40000000);
}

size_t batq_linear_workspace_bytes(const batq_weight* w, int64_t s) {
  if (w == nullptr || s < 0) return 0;
  const size_t q = round_up(static_cast<size_t>(s * (w->n / 2)), 1024) + round_up(batq_sf_bytes(s, w->n, BATQ_SF_MMA), 1024);
  if (s > 128) return q + prefill_flag_bytes(w);   // flag words of the one-kernel prefill path
  return q + (s > 0 && layer_takes_small_path(w, s) ? small_scratch(w, s).total() : 0);
}

int32_t batq_linear_kernel_launches(const batq_transform* t, const batq_weight* w, int64_t s) {
  if (w == nullptr || s <= 0) return 0;
  return (use_fused_small(t, w, s) || use_fused_prefill(t, w, s)) ? 1 : 2;
}

batq_status batq_linear_w4a4(const batq_transform* t, const batq_weight* w, const void* x_bf16, int64_t s, int64_t ld,
                             void* y, int32_t y_dtype, int64_t ldy, void* workspace, size_t workspace_bytes,
                             void* stream) {
  if (w == nullptr) return BATQ_ERR_NULL;
  batq_status st = check_x(x_bf16, s, w->n, ld);
  if (st != BATQ_OK) return st;
  if (t != nullptr && t->n != w->n) return BATQ_ERR_SHAPE;
  if (s == 0) return BATQ_OK;
  if (y == nullptr || workspace == nullptr) return BATQ_ERR_NULL;
  st = check_y(y, y_dtype, ldy, w->m);
  if (st != BATQ_OK) return st;
  if (!aligned(workspace, 1024)) return BATQ_ERR_ALIGN;
  if (workspace_bytes < batq_linear_workspace_bytes(w, s)) return BATQ_ERR_WORKSPACE;
  uint8_t* codes = static_cast<uint8_t*>(workspace);
  uint8_t* sf = codes + round_up(static_cast<size_t>(s * (w->n / 2)), 1024);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (use_fused_small(t, w, s)) return launch_linear_fused(t, w, x_bf16, s, ld, y, y_dtype, ldy, cs);
  if (layer_takes_small_path(w, s)) {
    // A handful of tokens: the quantiser also clears the split-K tickets, and the GEMM is launched
    // as its programmatic dependent so that the weight stream starts while it still runs.
    uint8_t* scratch = sf + round_up(batq_sf_bytes(s, w->n, BATQ_SF_MMA), 1024);
    const SmallScratch sc = small_scratch(w, s);
    st = launch_quantize(t, x_bf16, s, w->n, ld, codes, sf, BATQ_SF_MMA, nullptr, cs,
                         reinterpret_cast<uint32_t*>(scratch + sc.partial_bytes), static_cast<int32_t>(sc.tiles));
    if (st != BATQ_OK) return st;
    return launch_gemm_small(codes, sf, w, s, y, y_dtype, ldy, scratch, sc, cs, true);
  }
  if (use_fused_prefill(t, w, s))
    return launch_linear_prefill_fused(t, w, x_bf16, s, ld, y, y_dtype, ldy, codes, sf,
                                       sf + round_up(batq_sf_bytes(s, w->n, BATQ_SF_MMA), 1024), cs);
  st = launch_quantize(t, x_bf16, s, w->n, ld, codes, sf, BATQ_SF_MMA, nullptr, cs);
  if (st != BATQ_OK) return st;
  return launch_gemm(codes, sf, w, s, y, y_dtype, ldy, cs, true);
}

// Streams of the host entry points' copy pipeline, one pair per device, made on first use and kept
// for the life of the process.
constexpr int kHostChunks = 4;
struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
};
static std::mutex g_host_pipe_mutex;
static HostPipe g_host_pipe[kMaxDevices];

static batq_status host_pipe(int dev, HostPipe** out) {   // caller holds g_host_pipe_mutex
  if (dev < 0 || dev >= kMaxDevices) return BATQ_ERR_CUDA;
  HostPipe& hp = g_host_pipe[dev];
  if (!hp.ready) {
    if (cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) != cudaSuccess) {
      cudaGetLastError();
      return BATQ_ERR_CUDA;
    }
    hp.ready = true;
  }
  *out = &hp;
  return BATQ_OK;
}

// src_stream has reached this point before dst_stream goes on.  The event is destroyed at once:
// the runtime keeps it alive until the wait has been served.
static bool stream_follows(cudaStream_t dst_stream, cudaStream_t src_stream) {
  cudaEvent_t ev;
  if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return false;
  const bool ok = cudaEventRecord(ev, src_stream) == cudaSuccess && cudaStreamWaitEvent(dst_stream, ev, 0) == cudaSuccess;
  cudaEventDestroy(ev);
  return ok;
}

// Enqueues copy-in, layer and copy-out; nothing is waited for.
static batq_status host_enqueue(const batq_transform* t, const batq_weight* w, const void* x_host, int64_t s, void* y_host,
                                int32_t y_dtype, void* x_stage_dev, void* y_stage_dev, void* workspace,
                                size_t workspace_bytes, void* stream, bool a8) {
  if (w == nullptr || (a8 && t == nullptr)) return BATQ_ERR_NULL;
  auto ws_bytes = [&](int64_t rows) { return a8 ? batq_linear_w4a8_workspace_bytes(w, rows) : batq_linear_workspace_bytes(w, rows); };
  if (s < 0) return BATQ_ERR_SHAPE;
  if (s == 0) return BATQ_OK;
  if (x_host == nullptr || y_host == nullptr || x_stage_dev == nullptr || y_stage_dev == nullptr) return BATQ_ERR_NULL;
  if (y_dtype != BATQ_F32 && y_dtype != BATQ_BF16) return BATQ_ERR_UNSUPPORTED;
  if (workspace_bytes < ws_bytes(s)) return BATQ_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const size_t ysz = y_dtype == BATQ_F32 ? 4 : 2;
  // Token rows are independent, so a large batch goes through in up to four chunks of rows: the
  // copy-in of chunk i + 1 and the copy-out of chunk i - 1 run on streams of their own beside
  // the kernels of chunk i (PCIe carries both directions at once).  A small batch is one chunk.
  int64_t rows_per_chunk = s >= 512 ? ((s + kHostChunks - 1) / kHostChunks + 127) / 128 * 128 : s;
  int n_chunks = static_cast<int>((s + rows_per_chunk - 1) / rows_per_chunk);
  if (n_chunks > 1) {   // the workspace was sized for s rows at once: every chunk must fit it too
    const int64_t last = s - (n_chunks - 1) * rows_per_chunk;
    if (ws_bytes(rows_per_chunk) > workspace_bytes || ws_bytes(last) > workspace_bytes) {
      rows_per_chunk = s;
      n_chunks = 1;
    }
  }
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  std::lock_guard<std::mutex> lock(g_host_pipe_mutex);
  HostPipe* hp;
  st = host_pipe(dev, &hp);
  if (st != BATQ_OK) return st;
  // earlier work on the caller's stream may still use the staging buffers and the workspace
  bool ok = stream_follows(hp->in, cs);
  for (int c = 0; c < n_chunks && ok && st == BATQ_OK; ++c) {
    const int64_t r0 = c * rows_per_chunk;
    const int64_t rows = std::min<int64_t>(rows_per_chunk, s - r0);
    const uint8_t* xh = static_cast<const uint8_t*>(x_host) + static_cast<size_t>(r0 * w->n) * 2;
    uint8_t* xd = static_cast<uint8_t*>(x_stage_dev) + static_cast<size_t>(r0 * w->n) * 2;
    uint8_t* yd = static_cast<uint8_t*>(y_stage_dev) + static_cast<size_t>(r0 * w->m) * ysz;
    uint8_t* yh = static_cast<uint8_t*>(y_host) + static_cast<size_t>(r0 * w->m) * ysz;
    ok = cudaMemcpyAsync(xd, xh, static_cast<size_t>(rows * w->n) * 2, cudaMemcpyHostToDevice, hp->in) == cudaSuccess &&
         stream_follows(cs, hp->in);
    if (!ok) break;
    st = a8 ? batq_linear_w4a8(t, w, xd, rows, w->n, yd, y_dtype, w->m, workspace, workspace_bytes, stream)
            : batq_linear_w4a4(t, w, xd, rows, w->n, yd, y_dtype, w->m, workspace, workspace_bytes, stream);
    if (st != BATQ_OK) break;
    ok = stream_follows(hp->out, cs) &&
         cudaMemcpyAsync(yh, yd, static_cast<size_t>(rows * w->m) * ysz, cudaMemcpyDeviceToHost, hp->out) == cudaSuccess;
  }
  if (st != BATQ_OK) return st;
  if (!ok) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

batq_status batq_host_drain(void* stream) {
  int dev;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BATQ_ERR_CUDA;
  cudaStream_t in = nullptr, out = nullptr;
  bool have = false;
  {
    std::lock_guard<std::mutex> lock(g_host_pipe_mutex);
    have = g_host_pipe[dev].ready;
    in = g_host_pipe[dev].in;
    out = g_host_pipe[dev].out;
  }
  bool ok = !have || cudaStreamSynchronize(in) == cudaSuccess;
  ok = (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) == cudaSuccess) && ok;
  ok = (!have || cudaStreamSynchronize(out) == cudaSuccess) && ok;
  if (!ok) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  return BATQ_OK;
}

batq_status batq_linear_w4a4_host_async(const batq_transform* t, const batq_weight* w, const void* x_host, int64_t s,
                                        void* y_host, int32_t y_dtype, void* x_stage_dev, void* y_stage_dev,
                                        void* workspace, size_t workspace_bytes, void* stream) {
  return host_enqueue(t, w, x_host, s, y_host, y_dtype, x_stage_dev, y_stage_dev, workspace, workspace_bytes, stream, false);
}

batq_status batq_linear_w4a8_host_async(const batq_transform* t, const batq_weight* w, const void* x_host, int64_t s,
                                        void* y_host, int32_t y_dtype, void* x_stage_dev, void* y_stage_dev,
                                        void* workspace, size_t workspace_bytes, void* stream) {
  return host_enqueue(t, w, x_host, s, y_host, y_dtype, x_stage_dev, y_stage_dev, workspace, workspace_bytes, stream, true);
}

batq_status batq_linear_w4a4_host(const batq_transform* t, const batq_weight* w, const void* x_host, int64_t s,
                                  void* y_host, int32_t y_dtype, void* x_stage_dev, void* y_stage_dev, void* workspace,
                                  size_t workspace_bytes, void* stream) {
  const batq_status st = host_enqueue(t, w, x_host, s, y_host, y_dtype, x_stage_dev, y_stage_dev, workspace,
                                      workspace_bytes, stream, false);
  // whatever happened above: nothing of this call is left in flight when it returns
  const batq_status dr = (w != nullptr && s > 0) ? batq_host_drain(stream) : BATQ_OK;
  return st != BATQ_OK ? st : dr;
}

void batq_debug_force_tile_width(int32_t bn) { g_force_bn.store(bn, std::memory_order_relaxed); }

int32_t batq_debug_pair_schedule(int64_t s, int64_t m, int64_t n, int32_t sm_count, int32_t pair, int32_t* tiles,
                                 int32_t max_tiles) {
  if (s <= 0 || m <= 0 || n <= 0 || sm_count < 2) return -1;
  PairParams p{};
  int pairs = 0;
  if (!pair_schedule(s, m, (n + 255) / 256, sm_count, &p, &pairs)) return -1;
  if (pair < 0) return pairs;
  if (pair >= pairs) return 0;
  PairWalk w(p, pair, pairs);
  PairTile t;
  int32_t cnt = 0;
  while (w.next(t)) {
    if (tiles != nullptr && cnt < max_tiles) {
      tiles[3 * cnt] = t.mp;
      tiles[3 * cnt + 1] = t.n0;
      tiles[3 * cnt + 2] = t.bn;
    }
    ++cnt;
  }
  return cnt;
}
int32_t batq_debug_wide_schedule(int64_t s, int64_t m, int64_t n, int32_t sm_count, int32_t pair, int32_t* tiles,
                                 int32_t max_tiles) {
  if (s <= 0 || m <= 0 || n <= 0 || sm_count < 2) return -1;
  PairParams p{};
  int pairs = 0;
  double us = 0.0;
  const int force_bn = g_force_bn.load(std::memory_order_relaxed);
  const bool fw = force_bn >= 64 && force_bn <= kWideMaxBn && force_bn % 64 == 0;
  if (!wide_schedule(s, m, (n + 255) / 256, sm_count, fw ? force_bn : 0, false, &p, &pairs, &us)) return -1;
  if (pair < 0) return pairs;
  if (pair >= pairs) return 0;
  PairWalk w(p, pair, pairs);
  PairTile t;
  int32_t cnt = 0;
  while (w.next(t)) {
    if (tiles != nullptr && cnt < max_tiles) {
      tiles[3 * cnt] = t.mp;
      tiles[3 * cnt + 1] = t.n0;
      tiles[3 * cnt + 2] = t.bn;
    }
    ++cnt;
  }
  return cnt;
}
void batq_debug_force_quantizer(int32_t which) { g_force_quantizer.store(which, std::memory_order_relaxed); }
void batq_debug_force_gemm_kernel(int32_t which) { g_force_gemm_kernel.store(which, std::memory_order_relaxed); }
void batq_debug_force_small_s_splits(int32_t splits) { g_force_splits.store(splits, std::memory_order_relaxed); }
void batq_debug_force_small_s_path(int32_t which) { g_force_small_path.store(which, std::memory_order_relaxed); }
void batq_debug_force_small_s_reduce(int32_t which) { g_small_reduce.store(which, std::memory_order_relaxed); }
void batq_debug_force_prefill_path(int32_t which) { g_force_prefill_path.store(which, std::memory_order_relaxed); }

batq_status batq_debug_wait_timeout(int64_t limit_ns, void* stream) {
  batq_status st = device_setup(nullptr, nullptr);
  if (st != BATQ_OK) return st;
  const uint64_t lim = static_cast<uint64_t>(std::min<int64_t>(std::max<int64_t>(limit_ns, 1000), 10000000));
  wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(lim);
  return cudaGetLastError() == cudaSuccess ? BATQ_OK : BATQ_ERR_CUDA;
}

std::atomic<int> g_peak_load_stages{4};
std::atomic<int> g_peak_load_sharing{1};
std::atomic<int> g_peak_load_from_peer{0};
std::atomic<int> g_peak_a8{0};
std::atomic<int> g_peak_bn2{0};
std::atomic<int> g_peak_gemm_loop{0};
std::atomic<int> g_peak_sf_col{0};

static batq_status launch_mma_peak(const batq_weight* w, int32_t pair, int32_t bn, int32_t iters, int32_t sf_copies,
                                   int32_t load_iters, int32_t store_iters, double* flops_out, double* bytes_out,
                                   cudaStream_t stream) {
  if (bn != 64 && bn != 128 && bn != 192 && bn != 256) return BATQ_ERR_SHAPE;
  if (iters < 0 || iters > (1 << 24) || load_iters < 0 || load_iters > (1 << 24) || store_iters < 0 ||
      store_iters > (1 << 24) || iters + load_iters + store_iters == 0)
    return BATQ_ERR_SHAPE;
  if (load_iters > 0 && (w == nullptr || w->m < 256 || w->n < 256)) return BATQ_ERR_SHAPE;
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  if (w != nullptr && w->device != dev) return BATQ_ERR_CUDA;
  PeakParams p{};
  p.iters = iters;
  p.bn = bn;
  p.sf_copies = sf_copies ? 1 : 0;
  p.load_iters = load_iters;
  p.store_iters = store_iters;
  p.load_stages = g_peak_load_stages.load(std::memory_order_relaxed);
  p.load_sharing = g_peak_load_sharing.load(std::memory_order_relaxed);
  p.load_from_peer = pair ? g_peak_load_from_peer.load(std::memory_order_relaxed) : 0;
  const bool a8 = g_peak_a8.load(std::memory_order_relaxed) != 0;
  p.bn2 = a8 ? 0 : g_peak_bn2.load(std::memory_order_relaxed);
  const int kind = a8 ? 2 : (p.bn2 > 0 ? 1 : (g_peak_gemm_loop.load(std::memory_order_relaxed) != 0 ? 3 : 0));
  {
    const int want = g_peak_sf_col.load(std::memory_order_relaxed);
    const int lowest = p.bn2 > 0 ? 448 : 256;
    p.sf_col = (want >= lowest && want <= 512 - kPeakSfCols && want % 4 == 0) ? want : lowest;
  }
  p.w_row_tiles = load_iters > 0 ? static_cast<int32_t>(w->m / 128) : 1;   // whole boxes only
  p.w_k_steps = load_iters > 0 ? static_cast<int32_t>(w->n / 256) : 1;
  CUtensorMap none{};
  const CUtensorMap& map = load_iters > 0 ? w->tmap_b128 : none;
  const int ctas = pair ? (info->sm_count / 2) * 2 : info->sm_count;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(ctas));
  cfg.blockDim = dim3(kPeakThreads);
  cfg.dynamicSmemBytes = load_iters + store_iters > 0 ? kPeakSmemBytesLoads : kPeakSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pair ? 1 : 0;
  cudaError_t e;
  if (kind == 0)      e = pair ? cudaLaunchKernelEx(&cfg, mma_peak_kernel<true, 0>, map, p) : cudaLaunchKernelEx(&cfg, mma_peak_kernel<false, 0>, map, p);
  else if (kind == 1) e = pair ? cudaLaunchKernelEx(&cfg, mma_peak_kernel<true, 1>, map, p) : cudaLaunchKernelEx(&cfg, mma_peak_kernel<false, 1>, map, p);
  else if (kind == 3) e = pair ? cudaLaunchKernelEx(&cfg, mma_peak_kernel<true, 3>, map, p) : cudaLaunchKernelEx(&cfg, mma_peak_kernel<false, 3>, map, p);
  else                e = pair ? cudaLaunchKernelEx(&cfg, mma_peak_kernel<true, 2>, map, p) : cudaLaunchKernelEx(&cfg, mma_peak_kernel<false, 2>, map, p);
  if (e != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  if (flops_out != nullptr)
    *flops_out = 2.0 * (pair ? 256.0 : 128.0) * (bn + p.bn2) * (a8 ? 128.0 : 256.0) * iters * (pair ? ctas / 2 : ctas);
  if (bytes_out != nullptr) *bytes_out = static_cast<double>(kPeakLoadStageBytes) * (load_iters + store_iters) * ctas;
  return BATQ_OK;
}

void batq_debug_mma_peak_load_stages(int32_t stages) {
  g_peak_load_stages.store(stages < 1 ? 1 : (stages > kPeakLoadStages ? kPeakLoadStages : stages), std::memory_order_relaxed);
}
void batq_debug_mma_peak_gemm_loop(int32_t on) { g_peak_gemm_loop.store(on != 0, std::memory_order_relaxed); }
void batq_debug_mma_peak_sf_column(int32_t col) { g_peak_sf_col.store(col, std::memory_order_relaxed); }
void batq_debug_mma_peak_second_width(int32_t bn2) {
  g_peak_bn2.store((bn2 == 64 || bn2 == 128 || bn2 == 192) ? bn2 : 0, std::memory_order_relaxed);
}
void batq_debug_mma_peak_kind(int32_t a8) { g_peak_a8.store(a8 != 0, std::memory_order_relaxed); }
void batq_debug_mma_peak_load_from_peer(int32_t on) { g_peak_load_from_peer.store(on != 0, std::memory_order_relaxed); }
void batq_debug_mma_peak_load_sharing(int32_t ctas) {
  g_peak_load_sharing.store(ctas < 1 ? 1 : (ctas > 1024 ? 1024 : ctas), std::memory_order_relaxed);
}

batq_status batq_debug_mma_peak(int32_t pair, int32_t bn, int32_t iters, int32_t sf_copies, double* flops_out, void* stream) {
  if (iters <= 0) return BATQ_ERR_SHAPE;
  return launch_mma_peak(nullptr, pair, bn, iters, sf_copies, 0, 0, flops_out, nullptr, static_cast<cudaStream_t>(stream));
}

batq_status batq_debug_mma_peak_with_loads(const batq_weight* w, int32_t pair, int32_t bn, int32_t iters,
                                           int32_t load_iters, int32_t store_iters, double* flops_out,
                                           double* bytes_out, void* stream) {
  return launch_mma_peak(w, pair, bn, iters, 1, load_iters, store_iters, flops_out, bytes_out,
                         static_cast<cudaStream_t>(stream));
}

size_t batq_static_workspace_capacity(void) { return BATQ_STATIC_WORKSPACE_BYTES - 1024; }

batq_status batq_linear_w4a4_noalloc(const batq_transform* t, const batq_weight* w, const void* x_bf16, int64_t s,
                                     int64_t ld, void* y, int32_t y_dtype, int64_t ldy, void* stream) {
  if (w == nullptr) return BATQ_ERR_NULL;
  if (s < 0) return BATQ_ERR_SHAPE;
  if (batq_linear_workspace_bytes(w, s) > batq_static_workspace_capacity()) return BATQ_ERR_WORKSPACE;
  int dev;
  const DeviceInfo* info;
  batq_status st = device_setup(&dev, &info);
  if (st != BATQ_OK) return st;
  uint8_t* ws = nullptr;
  {
    // Once per device, with that device current: resolve the array's device address.
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo& d = g_dev[dev];
    if (d.static_ws == nullptr) {
      void* sym = nullptr;
      if (cudaGetSymbolAddress(&sym, g_static_workspace) != cudaSuccess || sym == nullptr) {
        cudaGetLastError();
        return BATQ_ERR_CUDA;
      }
      d.static_ws = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(sym) + 1023) & ~uintptr_t(1023));
    }
    ws = d.static_ws;
  }
  return batq_linear_w4a4(t, w, x_bf16, s, ld, y, y_dtype, ldy, ws, batq_static_workspace_capacity(), stream);
}

batq_status batq_last_device_status(void* stream) {
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  int flag = 0;
  if (cudaMemcpyFromSymbol(&flag, g_device_error, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return BATQ_ERR_CUDA; }
  if (flag != 0) {
    const int zero = 0;
    cudaMemcpyToSymbol(g_device_error, &zero, sizeof(int));
    return BATQ_ERR_TIMEOUT;
  }
  return BATQ_OK;
}

}  // extern "C"
