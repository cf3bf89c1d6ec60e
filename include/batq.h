/* batq -- the inference-time W4A4 linear layer of BATQuant on one B200 (sm_100a).
 *
 * Y ~= Q(X P) * Q(P^-1 W^T)   (the paper's arg-min objective, Sec. 3.1)
 *
 *   X [s x n] bf16 activations, W [m x n] bf16 weights, n = k * 32.
 *   P = diag(P_1..P_k) is block diagonal on the 32-element MX groups (Eq. 1)
 *   and every block is a Kronecker product P_j = L_j (x) R_j (Eq. 2; the paper
 *   writes B_i (x) A).  A block x of 32 channels is the matrix V[r][c],
 *   element index e = r*gc + c (Algorithm 1's reshape [-1, k, g2, g1]), and
 *   x P_j  <=>  L_j^T V R_j  (the vec identity after Eq. 2).
 *   Q is MXFP4: E2M1 elements, one UE8M0 scale per 32 elements (Sec. 2),
 *   round-to-nearest-even, OCP scale rule e = floor(log2 amax) - 2.
 *
 * Conventions.  Every pointer says "dev" (device memory of the current CUDA
 * device, owned by the caller) or "host".  Calls validate on the host and
 * return a status; nothing throws or aborts.  Kernel launches are asynchronous
 * on the given stream (a cudaStream_t passed as void*; NULL = default stream).
 * The library allocates device memory in batq_transform_create (held by the
 * handle) and, temporarily, in batq_prepare_weight (offline: it allocates, frees
 * and synchronises); every call on the online path (quantise, GEMM, layer) only
 * uses the caller's buffers.  Device-side waits are bounded: a kernel that
 * gives up records BATQ_ERR_TIMEOUT, read back by batq_last_device_status.
 * Test and tuning hooks live in batq_debug.h.
 */
#ifndef BATQ_H_
#define BATQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BATQ_OK = 0,
  BATQ_ERR_NULL = 1,        /* a required pointer is NULL                          */
  BATQ_ERR_SHAPE = 2,       /* n % 32 != 0, a size <= 0, ld < n, sizes too large   */
  BATQ_ERR_ALIGN = 3,       /* pointer not 16-byte aligned, ld % 8 != 0            */
  BATQ_ERR_UNSUPPORTED = 4, /* dtype, layout, architecture                         */
  BATQ_ERR_WORKSPACE = 5,   /* workspace smaller than batq_linear_workspace_bytes  */
  BATQ_ERR_SINGULAR = 6,    /* a transform factor is not invertible                */
  BATQ_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed                 */
  BATQ_ERR_TIMEOUT = 8      /* a bounded device-side wait ran out                  */
} batq_status;

enum { BATQ_SF_ROWMAJOR = 0, BATQ_SF_MMA = 1 };  /* scale-byte layouts, see batq_sf_bytes */
enum { BATQ_F32 = 0, BATQ_BF16 = 1 };            /* output dtypes of the GEMM             */

typedef struct batq_transform batq_transform; /* Theta of one layer: factors + clip ratios */
typedef struct batq_weight batq_weight;       /* one prepared (transformed, quantized) W   */

const char* batq_status_string(batq_status s);
int batq_version(void);

/* Theta = {A, {B_i}, {alpha_i}}, the parameter set Algorithm 2 keeps for the online
 * activation transform (its last step), as two Kronecker factors and clip ratios.
 *   n            channels, n % 32 == 0, k = n / 32 blocks.
 *   gr, gc       factor sizes, gr * gc == 32: (4, 8) is the paper's default (g2 = 4, g1 = 8);
 *                (1, 32), (2, 16), (8, 4), (16, 2), (32, 1) cover its ablation of the shared
 *                factor's size and, as (1, 32) with private right factors, the undecomposed
 *                32 x 32 block matrices of Table 1's "w/o" row.
 *   left         host fp32, row-major gr x gr matrices: one if left_stride == 0
 *                (shared by all blocks) else k of them, left_stride (= gr*gr)
 *                floats apart.  Acts on the slow index r of a block.
 *   right        host fp32, gc x gc, same rule with right_stride; acts on the
 *                contiguous index c.  The paper's default GPK is left = B_i
 *                (private 4x4), right = A (shared 8x8).
 *   clip_lo/hi   host fp32 [k] post-sigmoid ratios of Eq. 4, or both NULL for no
 *                clipping.
 * The arrays are copied (host copy for the inverse, device copy for the
 * kernels); the handle belongs to the CUDA device current at creation. */
batq_status batq_transform_create(batq_transform** out, int32_t n, int32_t gr, int32_t gc,
                                  const float* left, int64_t left_stride,
                                  const float* right, int64_t right_stride,
                                  const float* clip_lo, const float* clip_hi);
batq_status batq_transform_destroy(batq_transform* t);

/* Emulation of a BF16 implementation of the transform (Sec. 3.2 keeps the pre-quantization
 * transforms in BF16; Algorithm 1 is two contractions, each of which then stores a bf16 tensor).
 * on != 0: later calls with this transform round V R to bf16 before L^T is applied and round the
 * result to bf16 again, then clip and quantise as usual; on == 0 (the default): fp32 throughout,
 * nothing is rounded before the quantiser.  Needs the factored form, so only (gr, gc) = (4, 8)
 * (else UNSUPPORTED) and only MXFP4 (batq_quantize_act_mxfp8 and batq_linear_w4a8 return
 * UNSUPPORTED while it is on); the activation quantiser then always runs on the ALUs.  The
 * offline weight side is not affected (it is computed in fp64).  Not thread-safe against calls
 * that use the transform at the same time. */
batq_status batq_transform_set_bf16_intermediates(batq_transform* t, int32_t on);

/* Size in bytes of a scale-byte buffer for a [rows x n] tensor.
 *   BATQ_SF_ROWMAJOR: rows * k bytes, byte (row, j) at row*k + j.
 *   BATQ_SF_MMA: the layout the block-scaled tensor-core instruction reads.
 *     The tensor is cut into atoms of 128 rows x 4 blocks = 512 bytes; with
 *     KA = 2*ceil(k/8) atoms per 128-row tile, byte (row, j) is at
 *       ((row/128)*KA + j/4)*512 + (row%32)*16 + ((row%128)/32)*4 + j%4.
 *     rows are padded to a multiple of 128 and blocks to a multiple of 8.
 * Returns 0 for invalid arguments. */
size_t batq_sf_bytes(int64_t rows, int64_t n, int32_t layout);

/* Stages 1+2 of the path: x~ = x P (Eq. 1-2), block clip (Eq. 3-4), MXFP4
 * quantisation (Sec. 2), in that order (transform, clip, quantise: the paper's
 * algorithm flow).
 *   t        transform or NULL (identity, no clip: plain MXFP4 of X).
 *   x_bf16   dev, [s x n] bf16, row stride ld elements (ld >= n, ld % 8 == 0),
 *            16-byte aligned.
 *   n        channels (must equal t's n when t is given).
 *   codes    dev, s * n/2 bytes row-major; element 2i in bits 0-3 of byte i,
 *            element 2i+1 in bits 4-7; bit 3 of a code is the sign.
 *   scales   dev, batq_sf_bytes(s, n, scale_layout) bytes of E8M0 (e + 127).
 * s == 0 is a no-op.  Errors: NULL / SHAPE / ALIGN / UNSUPPORTED / CUDA. */
batq_status batq_quantize_act(const batq_transform* t, const void* x_bf16, int64_t s, int64_t n,
                              int64_t ld, void* codes, void* scales, int32_t scale_layout,
                              void* stream);

/* The same stages with 8-bit elements: MXFP8 with E4M3 codes (the MXFP8 element type Sec. 2 settles on),
 * the activation format of the paper's W4A8 configurations and of the 8-bit KV cache (the key and
 * value transforms P_k, P_v of Sec. 3.2 are applied head by head: pass the cache as
 * [tokens * heads x head_dim] with a transform of n = head_dim).  Shared scale
 * e = floor(log2 amax) - 8, elements round to nearest even and saturate at +-448.
 *   t        transform (required; an identity transform gives plain MXFP8 of X).
 *   codes    dev, s * n bytes row-major, one E4M3 code per element.
 *   scales   as batq_quantize_act.
 * Errors as batq_quantize_act, plus NULL for t == NULL. */
batq_status batq_quantize_act_mxfp8(const batq_transform* t, const void* x_bf16, int64_t s, int64_t n,
                                    int64_t ld, void* codes, void* scales, int32_t scale_layout,
                                    void* stream);

/* Offline weight fusion (the deployment part of Algorithm 2):
 * W~ = W P^-T per 32-block of each weight row, optional block
 * clip (Eq. 3-4 applied to weights), MXFP4 quantisation, written in the GEMM's
 * layout into a caller-provided buffer.  Computed in fp64 (inverse factors by
 * Gauss-Jordan on the host); not on the timed path.
 *   t            transform or NULL (identity).
 *   w_bf16       dev [m x n] bf16, row stride ld.
 *   w_clip_lo/hi dev fp32 [m * k] ratios per (row, block), or both NULL.
 *   weight_buf   dev, batq_weight_bytes(m, n) bytes, 1024-byte aligned; holds
 *                codes [m x n/2] row-major then scales in BATQ_SF_MMA layout.
 *                Must outlive the handle.
 * The call synchronises the stream (it is offline).  SINGULAR if a factor has
 * no inverse. */
size_t batq_weight_bytes(int64_t m, int64_t n);
batq_status batq_prepare_weight(const batq_transform* t, const void* w_bf16, int64_t m, int64_t n,
                                int64_t ld, const float* w_clip_lo, const float* w_clip_hi,
                                void* weight_buf, batq_weight** out, void* stream);
batq_status batq_weight_destroy(batq_weight* w);
/* Copies a prepared weight out as row-major packed codes [m x n/2] and row-major
 * scale bytes [m x k] (dev buffers), for inspection and tests. */
batq_status batq_weight_export(const batq_weight* w, void* codes_rowmajor, void* scales_rowmajor,
                               void* stream);
/* The way back: a prepared weight from stored codes and scales (what batq_weight_export
 * wrote: dev buffers, packed codes [m x n/2] and scale bytes [m x n/32], both
 * row-major), so that the offline fusion runs once per checkpoint and a server
 * only loads its result.  weight_buf as for batq_prepare_weight.  Codes and
 * scales are taken as they are (a scale byte of 255 is a NaN to the tensor
 * cores).  Synchronises the stream. */
batq_status batq_weight_import(const void* codes_rowmajor, const void* scales_rowmajor, int64_t m,
                               int64_t n, void* weight_buf, batq_weight** out, void* stream);

/* Stage 3 alone: Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} qx[s,j,i] * qw[m,j,i]
 * (the low-bit matrix multiplication of Sec. 3.2) on the block-scaled FP4
 * tensor cores, fp32 accumulation.
 *   x_codes       dev [s x n/2], 16-byte aligned, as written by batq_quantize_act.
 *   x_scales_mma  dev, BATQ_SF_MMA layout for [s x n].
 *   y             dev [s x m] row-major with row stride ldy elements, fp32 or bf16
 *                 (bf16 = round-to-nearest-even of the fp32 accumulator).
 * s == 0 is a no-op. */
batq_status batq_gemm_mxfp4(const void* x_codes, const void* x_scales_mma, const batq_weight* w,
                            int64_t s, void* y, int32_t y_dtype, int64_t ldy, void* stream);

/* Stage 3 of the W4A8 configurations (Sec. 4: MXFP8 activations, MXFP4 weights; E4M3 is the MXFP8
 * element type of Sec. 2):  Y[s, m] = sum_j 2^(ex[s,j] + ew[m,j]) * sum_{i<32} q8x[s,j,i] * qw[m,j,i]
 * on the block-scaled tensor cores, fp32 accumulation.
 *   x_codes8      dev [s x n] bytes, one E4M3 code per element, 16-byte aligned, as written by
 *                 batq_quantize_act_mxfp8.
 *   x_scales_mma  dev, BATQ_SF_MMA layout for [s x n].
 *   w             a prepared weight with n % 128 == 0 (else UNSUPPORTED): the same 4-bit codes
 *                 and scales as for batq_gemm_mxfp4, nothing is stored twice.
 *   y             as batq_gemm_mxfp4.
 * s == 0 is a no-op. */
batq_status batq_gemm_mxfp8_mxfp4(const void* x_codes8, const void* x_scales_mma, const batq_weight* w,
                                  int64_t s, void* y, int32_t y_dtype, int64_t ldy, void* stream);

/* The whole W4A8 layer: transform + clip + MXFP8 quantisation of X into the workspace (Eq. 1-4,
 * Sec. 2), then batq_gemm_mxfp8_mxfp4, launched as a programmatic dependent of the quantiser.
 *   t          transform (required, as for batq_quantize_act_mxfp8).
 *   workspace  dev, at least batq_linear_w4a8_workspace_bytes(w, s) bytes, 1024-byte aligned.
 * Errors as batq_linear_w4a4, plus UNSUPPORTED for n % 128 != 0. */
size_t batq_linear_w4a8_workspace_bytes(const batq_weight* w, int64_t s);
batq_status batq_linear_w4a8(const batq_transform* t, const batq_weight* w, const void* x_bf16,
                             int64_t s, int64_t ld, void* y, int32_t y_dtype, int64_t ldy,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Stage 3 alone for a handful of tokens (decode), s <= 128: the same contraction as
 * batq_gemm_mxfp4, organised for the case where streaming the weights from HBM once is the
 * whole cost.  The weights are the 128-row tensor-core operand and the tokens the narrow one;
 * the grid is (128-row weight tiles) x (K splits), and the partial sums of the splits meet in
 * `scratch` (added in split order, so results are deterministic).
 *   scratch        dev, batq_gemm_small_s_scratch_bytes(w, s) bytes, 1024-byte aligned; contents
 *                  need not be initialised; calls sharing it must be ordered on one stream.
 *   y              dev [s x m], fp32 or bf16, row stride ldy.
 * Errors as batq_gemm_mxfp4, plus SHAPE for s > 128 and WORKSPACE for a short scratch. */
size_t batq_gemm_small_s_scratch_bytes(const batq_weight* w, int64_t s);
batq_status batq_gemm_mxfp4_small_s(const void* x_codes, const void* x_scales_mma, const batq_weight* w,
                                    int64_t s, void* y, int32_t y_dtype, int64_t ldy, void* scratch,
                                    size_t scratch_bytes, void* stream);

/* The whole layer, stages 1+2+3: quantise X into the workspace, then the GEMM.  Up to 32
 * tokens (up to 128 on layers of at least 40 M weights) take the small-s GEMM, launched so that
 * its weight stream overlaps the quantiser; the smallest cases take a single kernel that
 * quantises the activations inside the GEMM (no workspace traffic at all).  In every other case
 * the GEMM is launched as a programmatic dependent of the quantiser as well.
 *   workspace  dev, at least batq_linear_workspace_bytes(w, s) bytes, 1024-byte
 *              aligned; overwritten by every call (calls sharing a workspace
 *              must be ordered on one stream). */
size_t batq_linear_workspace_bytes(const batq_weight* w, int64_t s);
/* How many kernels one batq_linear_w4a4(t, w, ., s, ...) call launches with the current dispatch
 * (1 = the fused kernel, 2 = quantiser + GEMM); 0 for a NULL weight or s <= 0.  Host only. */
int32_t batq_linear_kernel_launches(const batq_transform* t, const batq_weight* w, int64_t s);
batq_status batq_linear_w4a4(const batq_transform* t, const batq_weight* w, const void* x_bf16,
                             int64_t s, int64_t ld, void* y, int32_t y_dtype, int64_t ldy,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Same layer with HOST input and output: copies x_host (pinned or pageable host
 * memory, [s x n] bf16 dense) to x_stage_dev, runs batq_linear_w4a4, copies the
 * result from y_stage_dev to y_host; returns after everything has drained.
 * The copies run on two streams the library keeps per device; from 512 tokens
 * on the rows go through in up to four chunks, so that with pinned host memory
 * the copy-in of one chunk, the kernels of the one before and the copy-out of
 * the one before that overlap (token rows are independent: the result is that
 * of one call on all rows).  x_stage_dev (s*n*2 bytes) and y_stage_dev
 * (s*m*{4,2} bytes) are caller-provided device staging buffers; workspace as
 * for batq_linear_w4a4 with s rows. */
batq_status batq_linear_w4a4_host(const batq_transform* t, const batq_weight* w, const void* x_host,
                                  int64_t s, void* y_host, int32_t y_dtype, void* x_stage_dev,
                                  void* y_stage_dev, void* workspace, size_t workspace_bytes,
                                  void* stream);
/* The same, enqueued only: returns without waiting, so that the copies of several
 * layers (each with staging buffers and a workspace of its own) overlap one
 * another and the kernels.  y_host, and the right to reuse x_host, the staging
 * buffers and the workspace, are the caller's again after batq_host_drain(stream)
 * on the same device has returned BATQ_OK.  An error found while enqueueing is
 * returned at once; what was enqueued before it still runs. */
batq_status batq_linear_w4a4_host_async(const batq_transform* t, const batq_weight* w,
                                        const void* x_host, int64_t s, void* y_host, int32_t y_dtype,
                                        void* x_stage_dev, void* y_stage_dev, void* workspace,
                                        size_t workspace_bytes, void* stream);
/* The W4A8 layer (batq_linear_w4a8) with host input and output, enqueued only; the rest as for
 * batq_linear_w4a4_host_async, with a workspace of batq_linear_w4a8_workspace_bytes(w, s). */
batq_status batq_linear_w4a8_host_async(const batq_transform* t, const batq_weight* w,
                                        const void* x_host, int64_t s, void* y_host, int32_t y_dtype,
                                        void* x_stage_dev, void* y_stage_dev, void* workspace,
                                        size_t workspace_bytes, void* stream);
/* Waits for everything the host entry points have enqueued on the current device:
 * the library's copy streams and `stream`. */
batq_status batq_host_drain(void* stream);

/* The same layer for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of this library.)  Some hosts of
 * this code may not call cudaMalloc at the point where they run a layer: a serving
 * process that gave the whole device to its own memory pool at start-up, or a
 * latency-critical loop where an allocation's implicit device-wide synchronisation
 * is unacceptable.  For them the quantised activations (codes + scale bytes, the
 * scratch that batq_linear_w4a4 takes as `workspace`) live in one array that is
 * part of the library image: BATQ_STATIC_WORKSPACE_BYTES bytes of device memory on
 * every GPU that loads the library, held until the process exits.
 *   - Arguments as batq_linear_w4a4 minus the workspace; x and y are still the
 *     caller's.  The call itself performs no cudaMalloc / cudaFree and uses no
 *     allocating library routine.
 *   - BATQ_ERR_WORKSPACE if batq_linear_workspace_bytes(w, s) exceeds
 *     batq_static_workspace_capacity() (the array minus alignment slack); with the
 *     default size that admits e.g. s * n <= ~15.8 M elements (2048 x 4096 tokens
 *     x channels uses 4.3 MB).
 *   - The first call on each device looks up the array's device address (with that
 *     device current) and caches it; make that first call before any stream
 *     capture begins.
 *   - All calls on a device share the one array and it keeps the previous call's
 *     bytes.  Nothing in it has to start at zero (every byte the GEMM's result
 *     depends on is rewritten by the quantiser of the same call), but two calls
 *     whose kernels overlap on the GPU -- different streams, no ordering --
 *     race on it: order them. */
#define BATQ_STATIC_WORKSPACE_BYTES (8u << 20)
size_t batq_static_workspace_capacity(void);
batq_status batq_linear_w4a4_noalloc(const batq_transform* t, const batq_weight* w,
                                     const void* x_bf16, int64_t s, int64_t ld, void* y,
                                     int32_t y_dtype, int64_t ldy, void* stream);

/* Synchronises `stream` and returns BATQ_ERR_TIMEOUT if any kernel of this
 * library gave up a bounded wait since the last query (the record is cleared),
 * BATQ_ERR_CUDA if the stream reports an error, else BATQ_OK. */
batq_status batq_last_device_status(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BATQ_H_ */
