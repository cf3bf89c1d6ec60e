"""Parity of the CUDA path against the CPU oracle, through the C-ABI.  GPU only."""
import numpy as np
import pytest
import torch

from oracle import batq_oracle as O
from paper_2603_16590_b200 import synth
from tests.helpers import (code_mismatch_report, fp32_transform_bound, near_rounding_boundary,
                           sf_mma_to_rowmajor)

pytestmark = pytest.mark.gpu

# A-priori bounds on the fp32 transform error, relative to sum_e |x_e| |P_ef| of the block, per kernel
# (quantiser mode: 1 = streaming ALU, 2 = tensor cores, 3 = per-block ALU).
#   ALU kernels (Kronecker form, fused multiply-adds): an 8-term chain for V R and a 4-term chain for
#   L^T (V R), each step 2^-24: (gc + gr) * 2^-24 to first order; with margin (gr + gc + 3) * 2^-24.
#   Tensor-core kernel (dense form): P rounded to fp32 (2^-24), three-term bf16 split (exact),
#   products exact, 16-term sums inside the tensor core and six accumulating MMAs whose fp32
#   additions may truncate (2^-23 each; only the two high-term MMAs matter): about 10 * 2^-24; the
#   same 15 * 2^-24 is asserted.
# Every end-to-end test prints the largest observed |v^ - V| / (2^-24 * sum|x||P|) next to it.
FP32_REL_ULPS = {1: 15.0, 2: 15.0, 3: 15.0}
FP32_REL = 15 * 2.0 ** -24


@pytest.fixture(params=[1, 2, 3], ids=["alu", "tensorcore", "perblock"])
def qmode(request, batq):
    """Runs a test once per activation-quantiser implementation."""
    batq.batq_debug_force_quantizer(request.param)
    yield request.param
    batq.batq_debug_force_quantizer(0)


@pytest.fixture(params=[1, 2, 3], ids=["cta", "ctapair", "widepair"])
def gkernel(request, batq):
    """Runs a test once per prefill GEMM kernel (one CTA per tile / CTA pairs with two accumulators
    / CTA pairs with tiles of up to 448 features)."""
    batq.batq_debug_force_gemm_kernel(request.param)
    yield request.param
    batq.batq_debug_force_gemm_kernel(0)


def _mk_transform(batq, t):
    return batq.batq_transform_create(t.n, t.left, t.right, t.clip_lo, t.clip_hi, gr=t.left.shape[1],
                                      gc=t.right.shape[1])


def _gpu_quantize(batq, tr, xb, layout=0, ld=None):
    S, N = xb.shape
    x = batq.bits_to_cuda_bf16(xb)
    if ld is not None:
        xp = torch.zeros((S, ld), dtype=torch.bfloat16, device="cuda")
        xp[:, :N] = x
        x = xp[:, :N]
    codes = torch.full((S * N // 2 + 64,), 0xEE, dtype=torch.uint8, device="cuda")
    nsf = batq.batq_sf_bytes(S, N, layout)
    scales = torch.full((nsf + 64,), 0xEE, dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act(tr, x, codes, scales, layout)
    assert batq.batq_last_device_status() == 0
    torch.cuda.synchronize()
    c, s = codes.cpu().numpy(), scales.cpu().numpy()
    assert (c[S * N // 2:] == 0xEE).all() and (s[nsf:] == 0xEE).all(), "wrote past the output buffers"
    c = O.unpack_codes(c[:S * N // 2].reshape(S, N // 2))
    s = s[:nsf]
    s = s.reshape(S, N // 32) if layout == 0 else sf_mma_to_rowmajor(s, S, N // 32)
    return c, s


SHAPES = [(1, 32), (3, 96), (128, 1024), (77, 3584), (300, 4096), (257, 2048 + 32)]


@pytest.mark.parametrize("S,N", SHAPES)
@pytest.mark.parametrize("geometry", ["baseline", "paper"])
def test_quantizer_bit_exact_on_identical_transformed_input(batq, qmode, S, N, geometry):
    """Feed the oracle's Q(.) the GPU's own fp32 transformed+clipped values:
    codes and scale bytes must match exactly, every element."""
    xb = synth.make_activations(S, N, 100 + S)
    t = synth.make_transform(N, 7, geometry)
    tr = _mk_transform(batq, t)
    x = batq.bits_to_cuda_bf16(xb)
    vhat = torch.empty((S, N), dtype=torch.float32, device="cuda")
    batq.batq_debug_transform_clip_f32(tr, x, vhat)
    gc, gs = _gpu_quantize(batq, tr, xb)
    oc, os_ = O.mxfp4_quantize(vhat.cpu().numpy().astype(np.float64))
    assert np.array_equal(gs, os_)
    assert np.array_equal(gc, oc)


@pytest.mark.parametrize("S,N", SHAPES)
@pytest.mark.parametrize("geometry,clip", [("baseline", True), ("paper", True), ("naive", False)])
def test_quantizer_end_to_end_vs_oracle(batq, qmode, S, N, geometry, clip):
    xb = synth.make_activations(S, N, 200 + S)
    t = synth.make_transform(N, 8, geometry, clip=clip)
    tr = _mk_transform(batq, t)
    gc, gs = _gpu_quantize(batq, tr, xb)
    V = O.transform_clip(xb, t.left, t.right, t.clip_lo, t.clip_hi)
    oc, os_ = O.mxfp4_quantize(V)
    # the fp32 transform output vs the fp64 one
    vhat = torch.empty((S, N), dtype=torch.float32, device="cuda")
    batq.batq_debug_transform_clip_f32(tr, batq.bits_to_cuda_bf16(xb), vhat)
    X = np.abs(O.bf16_bits_to_f64(xb)).reshape(S, N // 32, 32)
    P = np.abs(O.block_matrices(t.left, t.right, N // 32))
    unit = fp32_transform_bound(X, P, 2.0 ** -24)
    err = np.abs(vhat.cpu().numpy().astype(np.float64) - V)
    worst = float(np.max(err / np.maximum(unit, 1e-300)))
    bound = FP32_REL_ULPS[qmode] * unit
    assert np.all(err <= bound + 1e-300), f"max |v^ - V| = {worst:.2f} x 2^-24 sum|x||P|"
    rep = code_mismatch_report(gc, gs, oc, os_, V, bound)
    print(f"quantiser mode {qmode} {S}x{N} {geometry}: max err {worst:.2f} x 2^-24 sum|x||P|; {rep}")
    # scale bytes: bit-exact, except blocks whose amax sits within the fp32 error of a power of two
    assert rep["scale_unexplained"] == 0 and rep["scale_mismatch"] <= 1e-5 * rep["blocks"] + 1
    # codes: at most 1e-4 of the elements differ, each next to a rounding boundary -- within 1 fp32
    # ulp of it (the strict count) or within the a-priori bound (the bound-based count) -- and only
    # to the neighbouring code
    assert rep["code_mismatch"] <= 1e-4 * rep["elements"] + 1
    assert rep["unexplained"] == 0 and rep["not_neighbour"] == 0
    assert rep["strict"] + rep["bound_only"] == rep["code_mismatch"]


@pytest.mark.parametrize("S,N", SHAPES)
def test_identity_transform_is_bit_exact_plain_mxfp4(batq, S, N):
    xb = synth.make_activations(S, N, 300 + S)
    gc, gs = _gpu_quantize(batq, None, xb)
    oc, os_ = O.quantize_act(xb, None, None)
    assert np.array_equal(gs, os_) and np.array_equal(gc, oc)
    # identity *factors* through either transform kernel give the same bits
    t = synth.make_transform(N, 1, identity=True, clip=False)
    for mode in (1, 2, 3):
        batq.batq_debug_force_quantizer(mode)
        try:
            gc2, gs2 = _gpu_quantize(batq, _mk_transform(batq, t), xb)
        finally:
            batq.batq_debug_force_quantizer(0)
        assert np.array_equal(gs2, os_) and np.array_equal(gc2, oc)


def test_quantizer_special_values(batq):
    """Zero blocks, signed zeros, ties, saturation, tiny and huge magnitudes."""
    N = 256
    X = np.zeros((4, N), np.float32)
    X[0, 32:64] = np.array([6, 5, 3.5, 2.5, 1.75, 1.25, 0.75, 0.25, -0.25, -7, 0.1, -0.1, 7, 7.5, 4, 3] * 2, np.float32)
    X[1, :32] = -0.0
    X[1, 64:96] = np.linspace(-1, 1, 32) * 2.0 ** -120
    X[2, :] = np.random.default_rng(0).standard_normal(N).astype(np.float32) * 2.0 ** 100
    X[3, 96:128] = 2.0 ** -133   # below the normal range: flushes into the clamped scale
    xb = synth.f32_to_bf16_bits(X)
    gc, gs = _gpu_quantize(batq, None, xb)
    oc, os_ = O.quantize_act(xb, None, None)
    assert np.array_equal(gs, os_) and np.array_equal(gc, oc)
    assert gs[0, 0] == 0 and gc[1, 0] == 8


def _special_rows(N):
    X = np.zeros((6, N), np.float32)
    X[0, 32:64] = np.array([6, 5, 3.5, 2.5, 1.75, 1.25, 0.75, 0.25, -0.25, -7, 0.1, -0.1, 7, 7.5, 4, 3] * 2, np.float32)
    X[1, :32] = -0.0
    X[1, 64:96] = np.linspace(-1, 1, 32) * 2.0 ** -120
    X[2, :] = np.random.default_rng(0).standard_normal(N).astype(np.float32) * 2.0 ** 100
    X[3, 96:128] = 2.0 ** -133   # below the normal range of bf16: the scale clamps at 2^-127
    X[4, 128:160] = np.array([7, -7] * 16, np.float32)              # saturation on both signs
    X[5, 0:32] = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 4.0] * 4, np.float32)   # every tie point
    X[5, 32:64] = -X[5, 0:32]
    return X


@pytest.mark.parametrize("layout", [0, 1], ids=["rowmajor", "mma"])
@pytest.mark.parametrize("mode", [1, 2, 3], ids=["alu", "tensorcore", "perblock"])
def test_every_quantiser_on_special_values_with_identity_factors(batq, mode, layout):
    """Zero blocks, signed zeros, ties at every threshold, saturation at +-7, 2^+-100 and a
    subnormal block through each of the three quantiser kernels (identity factors, no clip, so the
    transform is exact and the result must be the plain MXFP4 of X; a zero's sign bit alone is free:
    a sum of products with the identity's zeros gives +0)."""
    N = 256
    xb = synth.f32_to_bf16_bits(_special_rows(N))
    t = synth.make_transform(N, 1, identity=True, clip=False)
    batq.batq_debug_force_quantizer(mode)
    try:
        tr = _mk_transform(batq, t)
        gc, gs = _gpu_quantize(batq, tr, xb, layout=layout)
        vhat = torch.empty(xb.shape, dtype=torch.float32, device="cuda")
        batq.batq_debug_transform_clip_f32(tr, batq.bits_to_cuda_bf16(xb), vhat)
    finally:
        batq.batq_debug_force_quantizer(0)
    # bit-exact on the values the kernel rounded (signs of zeros included) ...
    oc, os_ = O.mxfp4_quantize(vhat.cpu().numpy().astype(np.float64))
    assert np.array_equal(gs, os_) and np.array_equal(gc, oc)
    # ... and equal to the plain MXFP4 of X up to the sign bit of zero codes
    pc, ps = O.quantize_act(xb, None, None)
    assert np.array_equal(gs, ps)
    assert np.array_equal(gc & 7, pc & 7)
    nz = (pc & 7) != 0
    assert np.array_equal(gc[nz], pc[nz])
    assert gs[0, 0] == 0 and gs[3, 3] == 0


@pytest.mark.parametrize("layout", [0, 1], ids=["rowmajor", "mma"])
@pytest.mark.parametrize("mode", [1, 2, 3], ids=["alu", "tensorcore", "perblock"])
def test_transform_output_on_exact_ties(batq, mode, layout):
    """A transform with power-of-two entries whose outputs land exactly on rounding boundaries:
    out[r][c] = v[r][c] + v[r][c-1] / 2 (right factor I + shift / 2, left factor I).  Every product
    and sum is exact in fp32, so all kernels must agree with the fp64 oracle bit for bit, ties to
    the even code included."""
    N = 96
    R = np.eye(8, dtype=np.float32)
    for c in range(1, 8):
        R[c - 1, c] = 0.5
    L = np.eye(4, dtype=np.float32)
    t = synth.Transform(N, L[None], np.repeat(R[None], N // 32, axis=0), None, None)
    rows = [
        [4, 0.5, 1, 0.5, 2, 1, 3, 1],            # -> 4, 2.5, 1.25, 1, 2.25, 2, 3.5, 2.5
        [0.5, 0, 0.5, 1.5, 1, 4, 2, 0],          # -> 0.5, 0.25, 0.5, 1.75, 1.75, 4.5, 4, 1
        [-4, -0.5, -1, -0.5, -2, -1, -3, -1],
        [2, 4, 0, 1.5, -0.5, 0.5, 0.25, 6],      # -> 2, 5, 2, 1.5, 0.25, 0.25, 0.5, 6.125 (saturates)
    ]
    blk = np.array(rows, np.float32).reshape(32)
    X = np.zeros((5, N), np.float32)
    X[0, 0:32] = blk
    X[1, 32:64] = blk * 2.0 ** -9
    X[2, 64:96] = -blk * 2.0 ** 20
    X[3, :] = np.tile(blk, 3)
    X[4, 0:32] = blk[::-1]
    xb = synth.f32_to_bf16_bits(X)
    assert np.array_equal(O.bf16_bits_to_f64(xb), X.astype(np.float64))      # the inputs are bf16 values
    batq.batq_debug_force_quantizer(mode)
    try:
        gc, gs = _gpu_quantize(batq, _mk_transform(batq, t), xb, layout=layout)
    finally:
        batq.batq_debug_force_quantizer(0)
    V = O.transform_clip(xb, t.left, t.right)
    ties = np.isin(np.abs(V[0, :32]) / 1.0, [0.25, 1.25, 1.75, 2.5, 3.5, 5.0])
    assert ties.sum() >= 6                                                    # the case does hit ties
    oc, os_ = O.mxfp4_quantize(V)
    assert np.array_equal(gs, os_)
    assert np.array_equal(gc & 7, oc & 7)
    nz = (oc & 7) != 0
    assert np.array_equal(gc[nz], oc[nz])


def test_bounded_wait_runs_out_and_is_reported_once(batq):
    """Failure detection without a fault: one warp waits 1 ms on a barrier nothing signals; the wait
    gives up, the kernel returns, the host reads BATQ_ERR_TIMEOUT exactly once, and the layer that
    ran before gives the same bits afterwards."""
    S, M, N = 300, 264, 1024
    t = synth.make_transform(N, 21, "baseline")
    tr = _mk_transform(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 21)))
    x = batq.bits_to_cuda_bf16(synth.make_activations(S, N, 21))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y0 = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, x, y0, ws)
    assert batq.batq_last_device_status() == 0
    batq.batq_debug_wait_timeout(1_000_000)
    assert batq.batq_last_device_status() == 8       # BATQ_ERR_TIMEOUT
    assert batq.batq_last_device_status() == 0       # the record was cleared by the query
    y1 = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, x, y1, ws)
    assert batq.batq_last_device_status() == 0
    assert torch.equal(y0, y1)


@pytest.mark.parametrize("S,N", [(5, 96), (130, 1024), (257, 3584)])
def test_scale_layout_mma_matches_rowmajor(batq, qmode, S, N):
    xb = synth.make_activations(S, N, 400 + S)
    tr = _mk_transform(batq, synth.make_transform(N, 9, "baseline"))
    c0, s0 = _gpu_quantize(batq, tr, xb, layout=0)
    c1, s1 = _gpu_quantize(batq, tr, xb, layout=1)
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1)


def test_quantizer_row_stride_and_determinism(batq, qmode):
    S, N = 70, 1024
    xb = synth.make_activations(S, N, 55)
    tr = _mk_transform(batq, synth.make_transform(N, 9, "baseline"))
    a = _gpu_quantize(batq, tr, xb)
    b = _gpu_quantize(batq, tr, xb, ld=N + 72)
    c = _gpu_quantize(batq, tr, xb)
    for u, v, w in zip(a, b, c):
        assert np.array_equal(u, v) and np.array_equal(u, w)


@pytest.mark.parametrize("S", [48, 1000])
def test_quantizer_is_independent_of_the_row_order(batq, qmode, S):
    """Mixed vision/text batch (first 75 % of the rows heavy-tailed Student-t, the rest Gaussian
    with outlier channels): quantising the rows interleaved gives exactly the interleaved result of
    quantising them in blocks, and a whole layer on the shuffled batch the shuffled output: no
    statistic crosses a token row."""
    N = 1792
    xb = synth.make_activations(S, N, 77, outlier_channel_frac=0.005, vision_rows=(3 * S) // 4)
    perm = np.random.default_rng(5).permutation(S)
    t = synth.make_transform(N, 9, "baseline")
    tr = _mk_transform(batq, t)
    c0, s0 = _gpu_quantize(batq, tr, xb)
    c1, s1 = _gpu_quantize(batq, tr, np.ascontiguousarray(xb[perm]))
    assert np.array_equal(c0[perm], c1) and np.array_equal(s0[perm], s1)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(264, N, 77)))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y0 = torch.empty((S, 264), dtype=torch.float32, device="cuda")
    y1 = torch.empty((S, 264), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, batq.bits_to_cuda_bf16(xb), y0, ws)
    batq.batq_linear_w4a4(tr, w, batq.bits_to_cuda_bf16(np.ascontiguousarray(xb[perm])), y1, ws)
    assert batq.batq_last_device_status() == 0
    assert torch.equal(y0[torch.from_numpy(perm).cuda()], y1)


def test_measurement_loops_leave_the_device_clean(batq):
    """The MMA-only loop and its variants with a TMA load stream or ordinary shared-memory stores
    beside it (the roofline denominators of the GEMM): every combination runs to the end, reports
    the work it did and leaves no device status behind; a weight is only read."""
    M, N = 1024, 1024
    wb = synth.make_weight(M, N, 77)
    w = batq.batq_prepare_weight(None, batq.bits_to_cuda_bf16(wb))
    codes0, sf0 = batq.batq_weight_export(w)
    for pair in (False, True):
        ctas = 148 if not pair else 74
        for it, lit, sit in ((40, 0, 0), (0, 37, 0), (0, 0, 9), (40, 37, 0), (33, 0, 9), (16, 5, 3)):
            flops, nbytes = batq.batq_debug_mma_peak_with_loads(w, pair, 256, it, lit, sit)
            torch.cuda.synchronize()
            assert batq.batq_last_device_status() == 0
            assert flops > 0 if it else flops == 0
            assert nbytes % 32768 == 0 and nbytes >= (lit + sit) * 32768 * ctas * 0.9
    try:
        for a8, gemm_loop, bn2, col in ((True, False, 0, 0), (False, True, 0, 0), (False, False, 192, 0),
                                        (False, False, 128, 480), (False, False, 0, 320)):
            batq.batq_debug_mma_peak_kind(a8)
            batq.batq_debug_mma_peak_gemm_loop(gemm_loop)
            batq.batq_debug_mma_peak_second_width(bn2)
            batq.batq_debug_mma_peak_sf_column(col)
            for pair in (True, False):
                flops = batq.batq_debug_mma_peak(pair, 256, 50, True)
                assert flops == 2.0 * (256 if pair else 128) * (256 + bn2) * (128 if a8 else 256) * 50 * (74 if pair else 148)
                torch.cuda.synchronize()
                assert batq.batq_last_device_status() == 0
    finally:
        batq.batq_debug_mma_peak_kind(False)
        batq.batq_debug_mma_peak_gemm_loop(False)
        batq.batq_debug_mma_peak_second_width(0)
        batq.batq_debug_mma_peak_sf_column(0)
    try:
        for stages, sharing, peer in ((1, 1, 0), (5, 8, 0), (2, 1, 1), (4, 148, 1), (4, 1, 0)):
            batq.batq_debug_mma_peak_load_stages(stages)
            batq.batq_debug_mma_peak_load_sharing(sharing)
            batq.batq_debug_mma_peak_load_from_peer(peer)
            for pair in (True, False):   # copies between the CTAs of a pair: ignored without pairs
                batq.batq_debug_mma_peak_with_loads(w, pair, 128, 20, 23, 0)
                batq.batq_debug_mma_peak_with_loads(w, pair, 256, 0, 11, 0)
                torch.cuda.synchronize()
                assert batq.batq_last_device_status() == 0
    finally:
        batq.batq_debug_mma_peak_load_stages(4)
        batq.batq_debug_mma_peak_load_sharing(1)
        batq.batq_debug_mma_peak_load_from_peer(0)
    codes1, sf1 = batq.batq_weight_export(w)
    assert torch.equal(codes0, codes1) and torch.equal(sf0, sf1)


# ---------------------------------------------------------------------------- other factorisations of the block
FACTOR_SIZES = [(1, 32), (2, 16), (8, 4), (16, 2), (32, 1)]


@pytest.mark.parametrize("gr,gc", FACTOR_SIZES)
@pytest.mark.parametrize("geometry", ["baseline", "paper", "naive"])
@pytest.mark.parametrize("S,N", [(3, 96), (130, 1024)])
def test_quantizer_other_factor_sizes(batq, gr, gc, geometry, S, N):
    """The paper's ablation of the factor sizes (g1 in {1, 2, 4, 8, 16, 32}); (1, 32) with private
    right factors is the undecomposed 32 x 32 block matrix."""
    xb = synth.make_activations(S, N, 250 + S)
    t = synth.make_transform(N, 12, geometry, gr=gr, gc=gc)
    tr = _mk_transform(batq, t)
    vhat = torch.empty((S, N), dtype=torch.float32, device="cuda")
    batq.batq_debug_transform_clip_f32(tr, batq.bits_to_cuda_bf16(xb), vhat)
    for layout in (0, 1):
        gc_, gs = _gpu_quantize(batq, tr, xb, layout=layout)
        # bit-exact on the GPU's own transformed values ...
        oc, os_ = O.mxfp4_quantize(vhat.cpu().numpy().astype(np.float64))
        assert np.array_equal(gs, os_) and np.array_equal(gc_, oc)
    # ... which are the fp64 transform within the fp32 bound
    V = O.transform_clip(xb, t.left, t.right, t.clip_lo, t.clip_hi)
    X = np.abs(O.bf16_bits_to_f64(xb)).reshape(S, N // 32, 32)
    P = np.abs(O.block_matrices(t.left, t.right, N // 32))
    bound = FP32_REL * np.einsum("sje,jef->sjf", X, P).reshape(S, N)
    assert np.all(np.abs(vhat.cpu().numpy().astype(np.float64) - V) <= bound + 1e-300)


@pytest.mark.parametrize("gr,gc", FACTOR_SIZES)
@pytest.mark.parametrize("S", [2, 40, 300])
def test_linear_other_factor_sizes(batq, gr, gc, S):
    M, N = 264, 1024
    xb = synth.make_activations(S, N, 260 + S)
    wb = synth.make_weight(M, N, 261)
    t = synth.make_transform(N, 13, "paper", gr=gr, gc=gc)
    tr = _mk_transform(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, batq.bits_to_cuda_bf16(xb), y, ws)
    assert batq.batq_last_device_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    Y, Sabs, _, _ = O.linear_w4a4(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)
    assert np.mean(np.abs(got - Y) > 1e-3 * Sabs + 1e-30) <= 1e-3
    assert np.linalg.norm(got - Y) <= 1e-4 * np.linalg.norm(Sabs)


@pytest.mark.parametrize("gr,gc", [(8, 4), (16, 2)])
@pytest.mark.parametrize("geometry", ["paper", "naive"])
@pytest.mark.parametrize("S,N", [(1, 4096), (16, 1056), (128, 544)])
def test_small_quantizer_other_factor_sizes_vs_dense_form(batq, gr, gc, geometry, S, N):
    """Right factors of 4 and 2 columns run through the four-lanes-per-block ALU quantiser at
    decode sizes (Kronecker form, Algorithm 1) and through the tensor-core quantiser (dense block
    matrices, Eq. 1-2) when forced: both within the fp32 bound of the fp64 transform, each
    bit-exact on its own transformed values."""
    xb = synth.make_activations(S, N, 270 + S)
    t = synth.make_transform(N, 15, geometry, gr=gr, gc=gc)
    tr = _mk_transform(batq, t)
    V = O.transform_clip(xb, t.left, t.right, t.clip_lo, t.clip_hi)
    X = np.abs(O.bf16_bits_to_f64(xb)).reshape(S, N // 32, 32)
    P = np.abs(O.block_matrices(t.left, t.right, N // 32))
    bound = FP32_REL * np.einsum("sje,jef->sjf", X, P).reshape(S, N)
    vh = {}
    try:
        for mode in (3, 2):
            batq.batq_debug_force_quantizer(mode)
            vhat = torch.empty((S, N), dtype=torch.float32, device="cuda")
            batq.batq_debug_transform_clip_f32(tr, batq.bits_to_cuda_bf16(xb), vhat)
            vh[mode] = vhat.cpu().numpy().astype(np.float64)
            assert np.all(np.abs(vh[mode] - V) <= bound + 1e-300)
            for layout in (0, 1):
                gc_, gs = _gpu_quantize(batq, tr, xb, layout=layout)
                oc, os_ = O.mxfp4_quantize(vh[mode])
                assert np.array_equal(gs, os_) and np.array_equal(gc_, oc)
    finally:
        batq.batq_debug_force_quantizer(0)
    assert batq.batq_last_device_status() == 0
    # two different summation orders of the same product: not the same bits everywhere
    assert np.all(np.abs(vh[2] - vh[3]) <= 2 * bound + 1e-300)


@pytest.mark.parametrize("gr,gc", [(8, 4), (16, 2)])
@pytest.mark.parametrize("S,M,N", [(1, 1032, 4096), (4, 520, 2048), (16, 264, 1056)])
def test_linear_fused_small_s_other_factor_sizes(batq, gr, gc, S, M, N):
    """The single-kernel decode path with 8 x 4 and 16 x 2 factors: against the oracle, and equal
    to the two-kernel path (the same four-lane arithmetic in both)."""
    xb = synth.make_activations(S, N, 280 + S)
    wb = synth.make_weight(M, N, 281)
    t = synth.make_transform(N, 16, "paper", gr=gr, gc=gc)
    tr = _mk_transform(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    x = batq.bits_to_cuda_bf16(xb)
    outs = {}
    try:
        for path in (1, 2):
            batq.batq_debug_force_small_s_path(path)
            assert batq.batq_linear_kernel_launches(tr, w, S) == (2 if path == 1 else 1)
            ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
            y = torch.full((S + 1, M + 8), float("nan"), dtype=torch.float32, device="cuda")
            batq.batq_linear_w4a4(tr, w, x, y[:S, :M], ws)
            assert batq.batq_last_device_status() == 0
            yh = y.cpu().numpy()
            assert np.isnan(yh[S]).all() and np.isnan(yh[:S, M:]).all(), "wrote outside [S x M]"
            outs[path] = yh[:S, :M].astype(np.float64)
    finally:
        batq.batq_debug_force_small_s_path(0)
    Y, Sabs, _, _ = O.linear_w4a4(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)
    for got in outs.values():
        assert np.mean(np.abs(got - Y) > 1e-3 * Sabs + 1e-30) <= 1e-3
        assert np.linalg.norm(got - Y) <= 1e-4 * np.linalg.norm(Sabs)
    assert np.linalg.norm(outs[1] - outs[2]) <= 1e-4 * np.linalg.norm(Sabs)


# ---------------------------------------------------------------------------- MXFP8 activations / KV cache
@pytest.mark.parametrize("S,N", [(1, 32), (3, 96), (130, 1024), (257, 3584), (300, 4096 + 32)])
@pytest.mark.parametrize("geometry", ["baseline", "paper"])
def test_mxfp8_quantizer_vs_oracle(batq, S, N, geometry):
    xb = synth.make_activations(S, N, 270 + S)
    t = synth.make_transform(N, 14, geometry)
    tr = _mk_transform(batq, t)
    x = batq.bits_to_cuda_bf16(xb)
    vhat = torch.empty((S, N), dtype=torch.float32, device="cuda")
    batq.batq_debug_transform_clip_f32(tr, x, vhat)
    V32 = vhat.cpu().numpy().astype(np.float64)
    for layout in (0, 1):
        codes = torch.full((S * N + 64,), 0xEE, dtype=torch.uint8, device="cuda")
        nsf = batq.batq_sf_bytes(S, N, layout)
        scales = torch.full((nsf + 64,), 0xEE, dtype=torch.uint8, device="cuda")
        batq.batq_quantize_act_mxfp8(tr, x, codes, scales, layout)
        assert batq.batq_last_device_status() == 0
        c, sc = codes.cpu().numpy(), scales.cpu().numpy()
        assert (c[S * N:] == 0xEE).all() and (sc[nsf:] == 0xEE).all(), "wrote past the output buffers"
        gc_ = c[:S * N].reshape(S, N)
        gs = sc[:nsf].reshape(S, N // 32) if layout == 0 else sf_mma_to_rowmajor(sc[:nsf], S, N // 32)
        # bit-exact on the GPU's own transformed values
        oc, os_ = O.mxfp8_quantize(V32)
        assert np.array_equal(gs, os_) and np.array_equal(gc_, oc)
    # and close to the fp64 path: neighbouring codes at most, rarely
    oc64, os64 = O.quantize_act_mxfp8(xb, t.left, t.right, t.clip_lo, t.clip_hi)
    same = np.repeat(gs == os64, 32, axis=1)
    assert (gs != os64).mean() <= 1e-4
    d = np.abs((gc_ & 0x7F).astype(int) - (oc64 & 0x7F).astype(int))
    assert np.all(d[same] <= 1) and (d[same] != 0).mean() <= 1e-3


def test_kv_cache_head_by_head(batq):
    """Key/value transforms act head by head (Sec. 3.2): the cache [tokens, heads, head_dim] is the
    matrix [tokens * heads, head_dim] with one transform of n = head_dim; KV4 and KV8."""
    tokens, heads, hd = 70, 8, 128
    xb = synth.make_activations(tokens * heads, hd, 31)
    t = synth.make_transform(hd, 15, "paper")
    tr = _mk_transform(batq, t)
    x = batq.bits_to_cuda_bf16(xb)                       # contiguous [tokens, heads, head_dim]
    vhat = torch.empty((tokens * heads, hd), dtype=torch.float32, device="cuda")
    batq.batq_debug_transform_clip_f32(tr, x, vhat)
    V32 = vhat.cpu().numpy().astype(np.float64)
    c4, s4 = _gpu_quantize(batq, tr, xb)
    o4, os4 = O.mxfp4_quantize(V32)
    assert np.array_equal(c4, o4) and np.array_equal(s4, os4)
    codes = torch.empty((tokens * heads, hd), dtype=torch.uint8, device="cuda")
    scales = torch.empty((tokens * heads, hd // 32), dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act_mxfp8(tr, x, codes, scales, 0)
    o8, os8 = O.mxfp8_quantize(V32)
    assert np.array_equal(codes.cpu().numpy(), o8) and np.array_equal(scales.cpu().numpy(), os8)
    # per head it is the oracle applied to that head's rows alone
    h = 3
    rows = np.arange(tokens) * heads + h
    oh, osh = O.quantize_act_mxfp8(xb[rows], t.left, t.right, t.clip_lo, t.clip_hi)
    assert (np.abs((codes.cpu().numpy()[rows] & 0x7F).astype(int) - (oh & 0x7F).astype(int)) <= 1).all()


# ---------------------------------------------------------------------------- weights
def _weight_mismatch_ok(gc, gs, oc, os_, Wt):
    sdiff = gs != os_
    assert sdiff.mean() <= 1e-6
    cdiff = (gc != oc) & np.repeat(~sdiff, 32, axis=1)
    assert cdiff.mean() <= 1e-5
    if cdiff.any():  # fp64 on both sides: only exact-tie neighbourhoods may differ
        scale = np.repeat(np.exp2(os_.astype(np.float64) - 127), 32, axis=1)
        assert np.all(near_rounding_boundary((np.abs(Wt) / scale)[cdiff], 1e-9))


@pytest.mark.parametrize("M,N,geometry", [(1024, 1024, "baseline"), (200, 96, "paper"), (129, 3584, "baseline"),
                                          (64, 256, None)])
def test_prepare_weight_vs_oracle(batq, M, N, geometry):
    wb = synth.make_weight(M, N, 500 + M)
    t = synth.make_transform(N, 10, geometry, clip=False) if geometry else None
    tr = _mk_transform(batq, t) if t else None
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    codes, scales = batq.batq_weight_export(w)
    torch.cuda.synchronize()
    gc, gs = O.unpack_codes(codes.cpu().numpy()), scales.cpu().numpy()
    Wt = O.transform_weight(wb, t.left if t else None, t.right if t else None)
    oc, os_ = O.mxfp4_quantize(Wt)
    _weight_mismatch_ok(gc, gs, oc, os_, Wt)


def test_prepare_weight_with_clip(batq):
    M, N = 96, 512
    wb = synth.make_weight(M, N, 77)
    t = synth.make_transform(N, 11, "baseline", clip=False)
    rng = np.random.default_rng(5)
    lo = rng.uniform(0.7, 1.0, (M, N // 32)).astype(np.float32)
    hi = rng.uniform(0.7, 1.0, (M, N // 32)).astype(np.float32)
    w = batq.batq_prepare_weight(_mk_transform(batq, t), batq.bits_to_cuda_bf16(wb),
                                 torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda())
    codes, scales = batq.batq_weight_export(w)
    gc, gs = O.unpack_codes(codes.cpu().numpy()), scales.cpu().numpy()
    Wt = O.block_clip(O.transform_weight(wb, t.left, t.right), lo, hi)
    oc, os_ = O.mxfp4_quantize(Wt)
    _weight_mismatch_ok(gc, gs, oc, os_, Wt)


@pytest.mark.parametrize("S,M,N", [(300, 520, 1024), (16, 264, 2048), (77, 200, 96), (2048, 1100, 768)])
def test_weight_import_reproduces_the_prepared_weight(batq, S, M, N):
    """Export -> import gives a weight that exports the same bytes and computes the same layer, bit
    for bit, on every path (prefill GEMMs, small-s GEMM, fused small-s kernel), W4A8 included; the
    scale layout's padding (rows past m, blocks past k) is finite whatever the buffer held before."""
    t = synth.make_transform(N, 21, "baseline")
    tr = _mk_transform(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 21)))
    codes, scales = batq.batq_weight_export(w)
    junk = torch.full((1 << 22,), 0xFF, dtype=torch.uint8, device="cuda")   # what a recycled buffer may hold
    del junk
    w2 = batq.batq_weight_import(codes, scales)
    c2, s2 = batq.batq_weight_export(w2)
    assert torch.equal(codes, c2) and torch.equal(scales, s2)
    x = batq.bits_to_cuda_bf16(synth.make_activations(S, N, 22))
    for ww in (w, w2):
        ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(ww, S))
        y = torch.full((S, M + (-M) % 8), float("nan"), dtype=torch.float32, device="cuda")
        batq.batq_linear_w4a4(tr, ww, x, y[:, :M], ws)
        if ww is w:
            y_ref = y.clone()
    assert batq.batq_last_device_status() == 0
    assert torch.equal(y[:, :M], y_ref[:, :M]) and torch.isfinite(y[:, :M]).all()
    if N % 128 == 0:
        outs = []
        for ww in (w, w2):
            ws = batq.aligned_workspace(batq.batq_linear_w4a8_workspace_bytes(ww, S))
            y8 = torch.empty((S, M + (-M) % 8), dtype=torch.float32, device="cuda")
            batq.batq_linear_w4a8(tr, ww, x, y8[:, :M], ws)
            outs.append(y8[:, :M].clone())
        assert torch.equal(outs[0], outs[1])


def test_weight_import_checks_its_arguments(batq):
    z = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    for args, status in (((z, z, 0, 64), 2), ((z, z, 8, 48), 2), ((None, z, 8, 64), 1), ((z, None, 8, 64), 1)):
        h = batq.C.c_void_p()
        buf = batq.aligned_workspace(4096)
        st = batq.load().batq_weight_import(args[0].data_ptr() if args[0] is not None else None,
                                            args[1].data_ptr() if args[1] is not None else None, args[2], args[3],
                                            buf.data_ptr(), batq.C.byref(h), None)
        assert st == status


def test_singular_factor_is_reported(batq):
    N = 64
    t = synth.make_transform(N, 3, "baseline", clip=False)
    t.left[0][:, 1] = t.left[0][:, 0]
    tr = _mk_transform(batq, t)
    with pytest.raises(batq.BatqError) as e:
        batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(8, N, 1)))
    assert e.value.status == 6


# ---------------------------------------------------------------------------- GEMM
def _gemm_case(batq, S, M, N, seed, xb=None, wb=None, out_dtype=torch.float32):
    """Quantise X and W on the GPU (identity transform), run the GEMM on those
    codes, and compare with the oracle GEMM fed the *same* codes and scales."""
    xb = synth.make_activations(S, N, seed) if xb is None else xb
    wb = synth.make_weight(M, N, seed) if wb is None else wb
    x = batq.bits_to_cuda_bf16(xb)
    w = batq.batq_prepare_weight(None, batq.bits_to_cuda_bf16(wb))
    codes = torch.empty((S, N // 2), dtype=torch.uint8, device="cuda")
    sf = torch.empty(batq.batq_sf_bytes(S, N, 1), dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act(None, x, codes, sf, 1)
    ldy = M + (-M) % 8
    y = torch.full((S + 1, ldy), float("nan"), dtype=out_dtype, device="cuda")
    batq.batq_gemm_mxfp4(codes, sf, w, S, y)
    assert batq.batq_last_device_status() == 0
    torch.cuda.synchronize()
    yh = y.float().cpu().numpy()
    assert np.isnan(yh[S]).all() and np.isnan(yh[:S, M:]).all(), "wrote outside [S x M]"
    xc = O.unpack_codes(codes.cpu().numpy())
    xs = sf_mma_to_rowmajor(sf.cpu().numpy(), S, N // 32)
    wc, ws = batq.batq_weight_export(w)
    Y, Sabs = O.gemm_mxfp4(xc, xs, O.unpack_codes(wc.cpu().numpy()), ws.cpu().numpy())
    return yh[:S, :M].astype(np.float64), Y, Sabs


GEMM_SHAPES = [(128, 1024, 1024), (128, 128, 256), (1, 8, 32), (77, 200, 96), (300, 520, 3584), (16, 4096, 4096),
               (260, 384, 512), (129, 257, 2048 + 32), (1000, 1100, 768)]


@pytest.mark.parametrize("S,M,N", GEMM_SHAPES)
def test_gemm_vs_oracle_same_codes(batq, gkernel, S, M, N):
    got, Y, Sabs = _gemm_case(batq, S, M, N, 600 + S)
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got - Y) <= 1e-3 * Sabs + 1e-30)
    # fp32 accumulation of exact products: in fact far tighter than the stated tolerance
    assert np.max(np.abs(got - Y) / (Sabs + 1e-30)) < 1e-5


@pytest.mark.parametrize("bn", [64, 128, 192, 256, 320, 384, 448])
@pytest.mark.parametrize("S,M,N", [(300, 520, 3584), (129, 257, 2048 + 32), (260, 1000, 512), (600, 2300, 768)])
def test_gemm_every_tile_width(batq, gkernel, bn, S, M, N):
    if bn in (320, 384) and gkernel != 3:
        pytest.skip("only the wide-tile kernel has these widths")
    batq.batq_debug_force_tile_width(bn)
    try:
        got, Y, Sabs = _gemm_case(batq, S, M, N, 700 + S)
        got16, _, _ = _gemm_case(batq, S, M, N, 700 + S, out_dtype=torch.bfloat16)
    finally:
        batq.batq_debug_force_tile_width(0)
    assert np.max(np.abs(got - Y) / (Sabs + 1e-30)) < 1e-5
    want16 = torch.from_numpy(got.astype(np.float32)).bfloat16().float().numpy()
    assert np.array_equal(got16.astype(np.float32), want16)


@pytest.mark.parametrize("bn", [64, 128, 192, 256, 320, 384, 448])
def test_gemm_scale_layout_localising_case_every_tile_width(batq, gkernel, bn):
    if bn in (320, 384) and gkernel != 3:
        pytest.skip("only the wide-tile kernel has these widths")
    batq.batq_debug_force_tile_width(bn)
    try:
        test_gemm_scale_layout_localising_case(batq)
    finally:
        batq.batq_debug_force_tile_width(0)


def test_gemm_scale_layout_localising_case(batq):
    """All codes = 4.0 and a distinct power-of-two scale per (row, block): any
    mistake in the scale layout or in the operand/scale pairing shows up as a
    wrong power of two in a specific output."""
    S, M, N = 200, 300, 1024
    k = N // 32
    ex = ((np.arange(S)[:, None] * 7 + np.arange(k)[None, :] * 3) % 21) - 10
    ew = ((np.arange(M)[:, None] * 5 + np.arange(k)[None, :] * 11) % 21) - 10
    X = np.repeat(4.0 * np.exp2(ex), 32, axis=1).astype(np.float32)
    W = np.repeat(4.0 * np.exp2(ew), 32, axis=1).astype(np.float32)
    got, Y, Sabs = _gemm_case(batq, S, M, N, 0, synth.f32_to_bf16_bits(X), synth.f32_to_bf16_bits(W))
    want = 32 * 16.0 * (np.exp2(ex.astype(np.float64)) @ np.exp2(ew.astype(np.float64)).T)
    assert np.array_equal(Y, want)
    assert np.all(np.abs(got - want) <= 1e-6 * want)


def test_gemm_bf16_output_is_rounded_fp32(batq):
    S, M, N = 130, 264, 1024
    a, _, _ = _gemm_case(batq, S, M, N, 42, out_dtype=torch.float32)
    b, _, _ = _gemm_case(batq, S, M, N, 42, out_dtype=torch.bfloat16)
    want = torch.from_numpy(a.astype(np.float32)).bfloat16().float().numpy()
    assert np.array_equal(b.astype(np.float32), want)


# ---------------------------------------------------------------------------- small-s (decode) GEMM
def _small_case(batq, S, M, N, seed, out_dtype=torch.float32, splits=0):
    """Quantise X and W on the GPU (identity transform), run the small-s GEMM on those codes and
    compare with the oracle GEMM fed the same codes and scales."""
    xb = synth.make_activations(S, N, seed)
    wb = synth.make_weight(M, N, seed)
    w = batq.batq_prepare_weight(None, batq.bits_to_cuda_bf16(wb))
    codes = torch.empty((S, N // 2), dtype=torch.uint8, device="cuda")
    sf = torch.full((batq.batq_sf_bytes(S, N, 1),), 0xFF, dtype=torch.uint8, device="cuda")  # NaN scales in the padding
    batq.batq_quantize_act(None, batq.bits_to_cuda_bf16(xb), codes, sf, 1)
    batq.batq_debug_force_small_s_splits(splits)
    try:
        scratch = batq.aligned_workspace(batq.batq_gemm_small_s_scratch_bytes(w, S))
        scratch.fill_(0xA5)
        ldy = M + (-M) % 8
        ys = []
        for _ in range(2):   # twice: the tickets must be back at zero after a call
            y = torch.full((S + 1, ldy), float("nan"), dtype=out_dtype, device="cuda")
            batq.batq_gemm_mxfp4_small_s(codes, sf, w, S, y, scratch)
            ys.append(y)
        assert batq.batq_last_device_status() == 0
    finally:
        batq.batq_debug_force_small_s_splits(0)
    torch.cuda.synchronize()
    assert torch.equal(ys[0][:S, :M], ys[1][:S, :M]), "not deterministic"
    yh = ys[0].float().cpu().numpy()
    assert np.isnan(yh[S]).all() and np.isnan(yh[:S, M:]).all(), "wrote outside [S x M]"
    xc = O.unpack_codes(codes.cpu().numpy())
    xs = sf_mma_to_rowmajor(sf.cpu().numpy(), S, N // 32)
    wc, ws = batq.batq_weight_export(w)
    Y, Sabs = O.gemm_mxfp4(xc, xs, O.unpack_codes(wc.cpu().numpy()), ws.cpu().numpy())
    return yh[:S, :M].astype(np.float64), Y, Sabs


SMALL_SHAPES = [(1, 8, 32), (1, 1024, 1024), (4, 300, 544), (16, 4096, 4096), (17, 257, 2048 + 32), (32, 520, 3584),
                (33, 128, 256), (64, 1000, 1024), (65, 264, 512), (100, 1032, 3584), (128, 4096, 2048)]


@pytest.mark.parametrize("S,M,N", SMALL_SHAPES)
@pytest.mark.parametrize("splits", [0, 1, 3])
@pytest.mark.parametrize("reduce", [2, 1], ids=["cluster", "tickets"])
def test_gemm_small_s_vs_oracle_same_codes(batq, S, M, N, splits, reduce):
    batq.batq_debug_force_small_s_reduce(reduce)
    try:
        got, Y, Sabs = _small_case(batq, S, M, N, 800 + S, splits=splits)
    finally:
        batq.batq_debug_force_small_s_reduce(0)
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got - Y) <= 1e-3 * Sabs + 1e-30)
    assert np.max(np.abs(got - Y) / (Sabs + 1e-30)) < 1e-5


def test_gemm_small_s_many_splits_and_bf16(batq):
    S, M, N = 16, 264, 14336
    a, Y, Sabs = _small_case(batq, S, M, N, 900, splits=32)
    assert np.max(np.abs(a - Y) / (Sabs + 1e-30)) < 1e-5
    b, _, _ = _small_case(batq, S, M, N, 900, out_dtype=torch.bfloat16, splits=32)
    want = torch.from_numpy(a.astype(np.float32)).bfloat16().float().numpy()
    assert np.array_equal(b.astype(np.float32), want)


def test_gemm_small_s_rejects_large_s_and_short_scratch(batq):
    w = batq.batq_prepare_weight(None, batq.bits_to_cuda_bf16(synth.make_weight(128, 256, 1)))
    z = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    y = torch.empty((129, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(batq.BatqError) as e:
        batq.batq_gemm_mxfp4_small_s(z, z, w, 129, y, batq.aligned_workspace(4096))
    assert e.value.status == 2
    with pytest.raises(batq.BatqError) as e:
        batq.batq_gemm_mxfp4_small_s(z, z, w, 8, y, batq.aligned_workspace(4096)[:512])
    assert e.value.status == 5


# ---------------------------------------------------------------------------- whole layer
@pytest.mark.parametrize("S,M,N,geometry", [(128, 1024, 1024, "baseline"), (128, 1024, 1024, "paper"),
                                            (50, 136, 544, "baseline"), (4, 1024, 1024, "baseline"),
                                            (1, 4096, 4096, "baseline"), (16, 6144, 4096, "paper"),
                                            (64, 520, 1024, "baseline"), (65, 520, 1024, "baseline"),
                                            (100, 1032, 3584, "paper"), (128, 4096, 4096, "baseline"),
                                            (100, 10240, 4096, "baseline"),   # 65..128 tokens on a large layer: small-s path
                                            (129, 520, 1024, "baseline"),
                                            (520, 1032, 1024, "baseline")])
def test_linear_w4a4_vs_oracle(batq, qmode, S, M, N, geometry):
    # automatic kernel choice: the small-s GEMM up to 64 tokens, one CTA per tile up to 128, CTA pairs above
    xb = synth.make_activations(S, N, synth.BASE_SEED)
    wb = synth.make_weight(M, N, synth.BASE_SEED)
    t = synth.make_transform(N, synth.BASE_SEED, geometry)
    tr = _mk_transform(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, batq.bits_to_cuda_bf16(xb), y, ws)
    assert batq.batq_last_device_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    Y, Sabs, (oc, os_), _ = O.linear_w4a4(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)
    # a few activation codes may legitimately differ (fp32 vs fp64 transform); each shifts an
    # output by at most one grid step of one element, far inside 1e-3 * Sabs unless K is tiny
    frac_bad = np.mean(np.abs(got - Y) > 1e-3 * Sabs + 1e-30)
    assert frac_bad <= 1e-3
    assert np.linalg.norm(got - Y) <= 1e-4 * np.linalg.norm(Sabs)
    # and the quantised layer tracks the full-precision one
    ref = O.bf16_bits_to_f64(xb) @ O.bf16_bits_to_f64(wb).T
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 0.5


@pytest.mark.parametrize("S,M,N,geometry", [(1, 4096, 4096, "baseline"), (4, 6144, 4096, "paper"), (16, 1032, 2048, "baseline"),
                                            (3, 136, 544, "naive"), (2, 264, 14336, "baseline"), (5, 520, 1024, None)])
@pytest.mark.parametrize("splits", [0, 2])
def test_linear_fused_small_s_vs_oracle(batq, S, M, N, geometry, splits):
    """The single-kernel path (activations quantised inside the GEMM kernel) against the oracle
    and against the two-kernel path."""
    xb = synth.make_activations(S, N, synth.BASE_SEED + S)
    wb = synth.make_weight(M, N, synth.BASE_SEED + S)
    t = synth.make_transform(N, synth.BASE_SEED + S, geometry) if geometry else None
    tr = _mk_transform(batq, t) if t else None
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    x = batq.bits_to_cuda_bf16(xb)
    outs = {}
    batq.batq_debug_force_small_s_splits(splits)
    try:
        for path in (1, 2):
            batq.batq_debug_force_small_s_path(path)
            ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
            y = torch.full((S + 1, M + 8), float("nan"), dtype=torch.float32, device="cuda")
            for _ in range(2):
                batq.batq_linear_w4a4(tr, w, x, y[:S, :M], ws)
            yb = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
            batq.batq_linear_w4a4(tr, w, x, yb, ws)
            assert batq.batq_last_device_status() == 0
            yh = y.cpu().numpy()
            assert np.isnan(yh[S]).all() and np.isnan(yh[:S, M:]).all(), "wrote outside [S x M]"
            outs[path] = yh[:S, :M].astype(np.float64)
            assert torch.equal(yb, y[:S, :M].bfloat16())
    finally:
        batq.batq_debug_force_small_s_path(0)
        batq.batq_debug_force_small_s_splits(0)
    L, R = (t.left, t.right) if t else (None, None)
    Y, Sabs, _, _ = O.linear_w4a4(xb, wb, L, R, t.clip_lo if t else None, t.clip_hi if t else None)
    for got in outs.values():
        assert np.all(np.isfinite(got))
        assert np.mean(np.abs(got - Y) > 1e-3 * Sabs + 1e-30) <= 1e-3
        assert np.linalg.norm(got - Y) <= 1e-4 * np.linalg.norm(Sabs)
    # the two paths round the same fp32 arithmetic; at most a few boundary codes may differ
    assert np.linalg.norm(outs[1] - outs[2]) <= 1e-4 * np.linalg.norm(Sabs)


@pytest.mark.parametrize("S", [1, 4, 16, 48, 100, 300])
def test_linear_calls_back_to_back_share_a_workspace(batq, S):
    """Layers called one after the other on one stream, with one workspace, inside a replayed CUDA
    graph: every kernel is a programmatic dependent of the one before it (the next layer's
    quantiser or fused kernel is scheduled while the previous GEMM still runs), so a kernel that
    touched the workspace, x or y before its wait would show up here.  Each output must be bit for
    bit what the same call gives when it runs alone."""
    shapes = [(1024, 1536), (1024, 1024), (1024, 2304), (2048, 1024), (1024, 264)]   # (n, m)
    layers = []
    for i, (n, m) in enumerate(shapes):
        t = synth.make_transform(n, 40 + i, "baseline")
        tr = _mk_transform(batq, t)
        w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(m, n, 40 + i)))
        x = batq.bits_to_cuda_bf16(synth.make_activations(S, n, 40 + i))
        layers.append((tr, w, x, m))
    ws = batq.aligned_workspace(max(batq.batq_linear_workspace_bytes(w, S) for _, w, _, _ in layers))
    alone = []
    for tr, w, x, m in layers:
        y = torch.empty((S, m), dtype=torch.bfloat16, device="cuda")
        batq.batq_linear_w4a4(tr, w, x, y, ws)
        torch.cuda.synchronize()
        alone.append(y)
    outs = [torch.zeros((S, m), dtype=torch.bfloat16, device="cuda") for _, _, _, m in layers]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(3):
                for (tr, w, x, m), y in zip(layers, outs):
                    batq.batq_linear_w4a4(tr, w, x, y, ws)
        for _ in range(3):
            g.replay()
    torch.cuda.synchronize()
    assert batq.batq_last_device_status() == 0
    for a, b in zip(alone, outs):
        assert torch.equal(a, b)


def test_linear_kernel_launches_reports_the_dispatch(batq):
    """1 = the fused kernel (a token or so on a layer whose K slices are short), 2 = quantiser + GEMM."""
    t = synth.make_transform(4096, 3, "baseline")
    tr = _mk_transform(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(4096, 4096, 3)))
    assert batq.batq_linear_kernel_launches(tr, w, 1) == 1
    assert batq.batq_linear_kernel_launches(tr, w, 16) == 2
    assert batq.batq_linear_kernel_launches(tr, w, 2048) == 2
    assert batq.batq_linear_kernel_launches(tr, w, 0) == 0
    batq.batq_debug_force_small_s_path(1)
    try:
        assert batq.batq_linear_kernel_launches(tr, w, 1) == 2
    finally:
        batq.batq_debug_force_small_s_path(0)


@pytest.mark.parametrize("S,M,N,pinned", [(96, 256, 512, True), (2048, 520, 1024, True), (640, 264, 2048, True),
                                          (1000, 1104, 768, False)])
def test_linear_host_entry_point_matches_device_entry_point(batq, S, M, N, pinned):
    """Host buffers in and out.  From 512 tokens on the rows go through in chunks whose copies and
    kernels overlap; token rows are independent, so the result is bit for bit that of one device
    call on all rows, also when a second call follows at once and when the host memory is pageable."""
    xb = synth.make_activations(S, N, 5)
    t = synth.make_transform(N, 5, "baseline")
    tr = _mk_transform(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 5)))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, batq.bits_to_cuda_bf16(xb), y, ws)
    xh = torch.from_numpy(xb.view(np.int16))
    yh = torch.full((S, M), float("nan"), dtype=torch.float32)
    if pinned:
        xh, yh = xh.pin_memory(), yh.pin_memory()
    xs = torch.empty((S, N), dtype=torch.bfloat16, device="cuda")
    ys = torch.empty((S, M), dtype=torch.float32, device="cuda")
    for _ in range(2):
        yh.fill_(float("nan"))
        batq.batq_linear_w4a4_host(tr, w, xh, yh, xs, ys, ws)
        assert batq.batq_last_device_status() == 0
        assert torch.equal(yh, y.cpu())
    yb = torch.empty((S, M), dtype=torch.bfloat16)
    ysb = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
    batq.batq_linear_w4a4_host(tr, w, xh, yb, xs, ysb, ws)
    assert torch.equal(yb, y.cpu().bfloat16())
    # enqueued only: two layers' copies and kernels in flight together, one wait
    w2 = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M + 8, N, 6)))
    ws2 = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w2, S))
    y2 = torch.empty((S, M + 8), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w2, batq.bits_to_cuda_bf16(xb), y2, ws2)
    yh.fill_(float("nan"))
    yh2 = torch.full((S, M + 8), float("nan"), dtype=torch.float32)
    yh2 = yh2.pin_memory() if pinned else yh2
    xs2 = torch.empty((S, N), dtype=torch.bfloat16, device="cuda")
    ys2 = torch.empty((S, M + 8), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4_host_async(tr, w, xh, yh, xs, ys, ws)
    batq.batq_linear_w4a4_host_async(tr, w2, xh, yh2, xs2, ys2, ws2)
    batq.batq_host_drain()
    assert batq.batq_last_device_status() == 0
    assert torch.equal(yh, y.cpu()) and torch.equal(yh2, y2.cpu())


def test_empty_input_is_a_noop(batq):
    tr = _mk_transform(batq, synth.make_transform(64, 1, "baseline"))
    x = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    batq.batq_quantize_act(tr, x, None, None, 0, ld=64, s=0, n=64)
