/* batq_debug -- test, tuning and measurement hooks of the batq library.
 *
 * Nothing here is part of the layer's public contract (batq.h).  The batq_debug_force_* setters
 * change how later calls of the whole process pick their kernels; each is one atomic word that
 * every call reads once, so setting them from one thread while others launch is well defined
 * (a call sees either the old or the new value), but they are process-wide: use them from tests
 * and tuning runs, not from a server.  At their defaults (0) they change nothing.
 */
#ifndef BATQ_DEBUG_H_
#define BATQ_DEBUG_H_

#include "batq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* The exact fp32 values the quantiser rounds (after the transform of Eq. 1-2 and the clip of
 * Eq. 3-4, before scaling), out dev fp32 [s x n] row-major.  Uses the same kernel choice as
 * batq_quantize_act, so the tests can feed the oracle's quantiser identical inputs. */
batq_status batq_debug_transform_clip_f32(const batq_transform* t, const void* x_bf16, int64_t s,
                                          int64_t n, int64_t ld, float* out, void* stream);

/* Forces the GEMM's output-tile width to 64, 128, 192 or 256 columns for all later calls in this
 * process (the CTA-pair kernel also takes 448 for columns of 256 and 192 alternating, and 1 for
 * its automatic choice restricted to one width pattern for the whole layer); any other value
 * restores the automatic choice. */
void batq_debug_force_tile_width(int32_t bn);

/* Host only, no GPU needed: the work distribution of the CTA-pair GEMM for an s x m output
 * over n input channels on a device with sm_count SMs.  pair < 0: returns the number of CTA pairs
 * launched.  Otherwise returns the number of tiles pair `pair` works through, in order, and
 * writes the first max_tiles of them to tiles (host, 3 ints each: index of the 256-token row
 * block, first output feature, width in features).  -1 for arguments out of range. */
int32_t batq_debug_pair_schedule(int64_t s, int64_t m, int64_t n, int32_t sm_count, int32_t pair,
                                 int32_t* tiles, int32_t max_tiles);

/* The same for the wide-tile CTA-pair GEMM (tiles of up to 448 features, one accumulator). */
int32_t batq_debug_wide_schedule(int64_t s, int64_t m, int64_t n, int32_t sm_count, int32_t pair,
                                 int32_t* tiles, int32_t max_tiles);

/* Which prefill GEMM kernel later calls use.  0 = automatic (CTA pairs sharing a 256-token tile
 * for s > 128 -- with tiles of up to 256 features and two accumulators, or tiles of up to 448
 * features and one, whichever the cost model expects to finish first --, one CTA per 128-token
 * tile otherwise), 1 = always one CTA per tile, 2 = always CTA pairs with two accumulators,
 * 3 = always CTA pairs with wide tiles (batq_debug_force_tile_width then takes any multiple of 64
 * up to 448 and makes every column that wide). */
void batq_debug_force_gemm_kernel(int32_t which);

/* Which activation quantiser later calls use.  0 = automatic (up to 128 tokens the per-block ALU
 * kernel, above that the tensor-core dense-block kernel; the identity transform above 128 tokens
 * and nothing else takes the streaming ALU kernel), 1 = the streaming ALU kernel (Kronecker
 * form), 2 = the tensor-core kernel, 3 = the per-block ALU kernel.  The streaming ALU kernel is
 * built for 4 x 8 factors and the per-block ALU kernel for 4 x 8, 8 x 4 and 16 x 2; a transform
 * of another size takes the tensor-core kernel where the forced one cannot run it. */
void batq_debug_force_quantizer(int32_t which);

/* Number of K splits of the small-s GEMM (clamped to the number of 256-element K steps and to
 * 32); 0 restores the automatic choice.  Scratch sizes follow it. */
void batq_debug_force_small_s_splits(int32_t splits);

/* How the small-s GEMM adds the partial tiles of its K splits.  0 = automatic (through a
 * thread-block cluster's shared memory where the grid leaves room for clusters, else through
 * scratch and tickets), 1 = always scratch and tickets, 2 = the cluster whenever there are at
 * most 8 splits. */
void batq_debug_force_small_s_reduce(int32_t which);

/* How batq_linear_w4a4 runs a handful of tokens.  0 = automatic (one fused kernel that quantises
 * the activations inside the GEMM where that is the faster one -- tokens x K-steps per CTA <= 4
 * and a grid of one wave --, else the quantiser kernel followed by the small-s GEMM), 1 = always
 * the two kernels, 2 = the fused kernel up to 16 tokens.  The fused kernel needs n <= 16384;
 * other shapes take the two kernels. */
void batq_debug_force_small_s_path(int32_t which);

/* How batq_linear_w4a4 runs prefill shapes (s > 128, m >= 192, a transform, k % 8 == 0).
 * 0 = automatic, 1 = always two kernels (quantiser, then the CTA-pair GEMM as its programmatic
 * dependent), 2 = one kernel (quantise phase and GEMM phase on the same grid) wherever it applies. */
void batq_debug_force_prefill_path(int32_t which);

/* Failure-detection check that harms nothing: launches one warp that waits, with the library's
 * bounded wait and a limit of limit_ns nanoseconds (clamped to [1000, 10000000]), on a barrier
 * that nothing ever signals.  The wait runs out, the kernel records it exactly as a product
 * kernel would and returns normally; the next batq_last_device_status reports BATQ_ERR_TIMEOUT
 * once.  The context stays usable. */
batq_status batq_debug_wait_timeout(int64_t limit_ns, void* stream);

/* Measurement: the block-scaled FP4 tensor-core rate of this GPU with nothing else in the way.
 * Every CTA (one per SM; pair != 0: every pair of CTAs, tcgen05 cta_group::2) issues `iters`
 * K-steps of four tcgen05.mma kind::mxf4.block_scale (K = 64 each, 128 or 256 rows x bn columns)
 * on operands that stay resident in shared memory (seeded pseudo-random codes, scale bytes near
 * 2^0), accumulating in tensor memory; nothing is loaded or stored in the loop.  sf_copies != 0:
 * the scale factors are copied from shared to tensor memory (tcgen05.cp) again before every
 * K-step, as a GEMM whose scales change with K has to; 0: once, before the loop.  The caller
 * times the launch; *flops_out (host) receives the floating-point operations of the launch
 * (2 * rows * bn * 256 per K-step and CTA or pair).  bn in {64, 128, 192, 256}. */
batq_status batq_debug_mma_peak(int32_t pair, int32_t bn, int32_t iters, int32_t sf_copies,
                                double* flops_out, void* stream);

/* Measurement: the same loop with a load stream beside it.  While warp 1 of every CTA issues the
 * MMAs of batq_debug_mma_peak (scale copies repeated every K-step) on its resident operands,
 * warp 0 loads `load_iters` stages of 32 KiB (two TMA boxes of 128 rows x 128 bytes of w's codes,
 * the size of a GEMM stage) into a ring of four stages (batq_debug_mma_peak_load_stages: 1..5)
 * that nobody reads; neither waits for the other.
 * iters = 0: the loads alone; load_iters = 0: the MMAs alone.  w (m, n >= 256; may be NULL when
 * load_iters = 0) is only read; 58 MB or less keeps it in L2.  store_iters > 0: warps 2-3 write
 * that many 32 KiB stages into the same ring with ordinary st.shared instructions (no global
 * memory traffic), to tell a shared-memory bandwidth limit from one of the path from L2.
 * *flops_out and *bytes_out (host, may be NULL) receive the launch's floating-point operations and
 * loaded plus stored bytes.  What the numbers show: whether the tensor cores and a stream into
 * shared memory slow one another down when no barrier couples them. */
/* a8 != 0: the loops below issue tcgen05.mma kind::mxf8f6f4 (E4M3 x E2M1 in 8-bit containers, K = 32
 * per MMA, 128 elements per K-step: the W4A8 GEMM's instruction) instead of kind::mxf4; the flops
 * reported follow. */
void batq_debug_mma_peak_kind(int32_t a8);
/* bn2 in {64, 128, 192} (kind::mxf4 only; anything else switches it off): every MMA of the loops
 * below is followed by one of width bn2 on the same operands into a second accumulator (tensor
 * memory columns 256..), the issue pattern of the wide-tile GEMM. */
void batq_debug_mma_peak_second_width(int32_t bn2);
/* on != 0 (kind::mxf4, one accumulator): the MMAs are issued by the CTA-pair GEMM's own loop, statement
 * for statement (a wait on a completed barrier phase, a fence, the scale copies into alternating
 * slots, four MMAs from descriptors that depend on a run-time stage index and a commit per K-step),
 * on the same resident operands: what that loop costs with the operand stream taken away. */
void batq_debug_mma_peak_gemm_loop(int32_t on);
/* Tensor-memory column at which the loops below keep their scale factors: a multiple of 4 behind
 * the accumulators (from 256, from 448 with a second accumulator) up to 488; anything else = right
 * behind the accumulators. */
void batq_debug_mma_peak_sf_column(int32_t col);
void batq_debug_mma_peak_load_stages(int32_t stages);   /* ring depth of the load stream, 1..5 (default 4) */
/* How many CTAs (consecutive block indices) load the same boxes at the same time, as the tiles of a
 * GEMM that share a row or column block do; 1 (default) = every CTA its own boxes. */
void batq_debug_mma_peak_load_sharing(int32_t ctas);
/* on != 0, pairs only: half of every stage (16 KiB) is not loaded from L2 but copied by the other
 * CTA of the pair from its shared memory (cp.async.bulk shared::cta -> shared::cluster, no
 * multicast), as a GEMM would forward an operand tile that two CTAs need. */
void batq_debug_mma_peak_load_from_peer(int32_t on);
batq_status batq_debug_mma_peak_with_loads(const batq_weight* w, int32_t pair, int32_t bn, int32_t iters,
                                           int32_t load_iters, int32_t store_iters, double* flops_out,
                                           double* bytes_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BATQ_DEBUG_H_ */
