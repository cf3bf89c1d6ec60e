"""W4A8: MXFP8 (E4M3) activations x MXFP4 weights (the paper's near-lossless settings, Sec. 4),
GEMM and whole layer against the CPU oracle, through the C-ABI.  GPU only."""
import numpy as np
import pytest
import torch

from oracle import batq_oracle as O
from paper_2603_16590_b200 import synth
from tests.helpers import sf_mma_to_rowmajor

pytestmark = pytest.mark.gpu


def _identity(N):
    return synth.make_transform(N, 1, identity=True, clip=False)


def _mk(batq, t):
    return batq.batq_transform_create(t.n, t.left, t.right, t.clip_lo, t.clip_hi, gr=t.left.shape[1], gc=t.right.shape[1])


def _gemm_case(batq, S, M, N, seed, xb=None, wb=None, out_dtype=torch.float32):
    """Quantise X to MXFP8 and W to MXFP4 on the GPU (identity transform), run the W4A8 GEMM on those
    codes and compare with the oracle contraction fed the same codes and scales."""
    xb = synth.make_activations(S, N, seed) if xb is None else xb
    wb = synth.make_weight(M, N, seed) if wb is None else wb
    w = batq.batq_prepare_weight(None, batq.bits_to_cuda_bf16(wb))
    codes = torch.empty((S, N), dtype=torch.uint8, device="cuda")
    sf = torch.full((batq.batq_sf_bytes(S, N, 1),), 0xFF, dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act_mxfp8(_mk(batq, _identity(N)), batq.bits_to_cuda_bf16(xb), codes, sf, 1)
    ldy = M + (-M) % 8
    y = torch.full((S + 1, ldy), float("nan"), dtype=out_dtype, device="cuda")
    batq.batq_gemm_mxfp8_mxfp4(codes, sf, w, S, y)
    assert batq.batq_last_device_status() == 0
    yh = y.float().cpu().numpy()
    assert np.isnan(yh[S]).all() and np.isnan(yh[:S, M:]).all(), "wrote outside [S x M]"
    xs = sf_mma_to_rowmajor(sf.cpu().numpy(), S, N // 32)
    wc, ws = batq.batq_weight_export(w)
    Y, Sabs = O.gemm_mxfp8_mxfp4(codes.cpu().numpy(), xs, O.unpack_codes(wc.cpu().numpy()), ws.cpu().numpy())
    return yh[:S, :M].astype(np.float64), Y, Sabs


@pytest.fixture(params=[1, 2, 3], ids=["cta", "ctapair", "widepair"])
def gkernel(request, batq):
    """Runs a test once per W4A8 GEMM kernel (one CTA per tile / CTA pairs sharing a 256-token tile
    with two accumulators / CTA pairs with tiles of up to 448 features)."""
    batq.batq_debug_force_gemm_kernel(request.param)
    yield request.param
    batq.batq_debug_force_gemm_kernel(0)


SHAPES = [(128, 128, 256), (128, 1024, 1024), (1, 8, 128), (77, 200, 384), (300, 520, 3584), (260, 384, 512),
          (129, 257, 2048 + 128), (1000, 1100, 768)]


@pytest.mark.parametrize("bn", [0, 64, 128, 192, 256, 320, 384, 448])
@pytest.mark.parametrize("S,M,N", SHAPES)
def test_w4a8_gemm_vs_oracle_same_codes(batq, gkernel, S, M, N, bn):
    if gkernel == 1 and bn not in (0, 128, 256):
        pytest.skip("the one-CTA kernel has tiles of 128 and 256 features")
    if gkernel == 2 and bn in (320, 384):
        pytest.skip("only the wide-tile kernel has these widths")
    batq.batq_debug_force_tile_width(bn)
    try:
        got, Y, Sabs = _gemm_case(batq, S, M, N, 1600 + S)
    finally:
        batq.batq_debug_force_tile_width(0)
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got - Y) <= 1e-3 * Sabs + 1e-30)
    # products of an E4M3 and an E2M1 value are exact in fp32; only the accumulation rounds
    assert np.max(np.abs(got - Y) / (Sabs + 1e-30)) < 1e-5


@pytest.mark.parametrize("bn", [64, 128, 192, 256, 320, 384, 448])
def test_w4a8_scale_layout_localising_case(batq, gkernel, bn):
    """Constant codes and a distinct power-of-two scale per (row, block) on both sides: a mistake in
    the scale layout, in the byte of the scale column an MMA takes, or in the operand pairing shows
    up as a wrong power of two in a specific output."""
    S, M, N = 200, 300, 1024
    k = N // 32
    ex = ((np.arange(S)[:, None] * 7 + np.arange(k)[None, :] * 3) % 21) - 10
    ew = ((np.arange(M)[:, None] * 5 + np.arange(k)[None, :] * 11) % 21) - 10
    X = np.repeat(256.0 * np.exp2(ex), 32, axis=1).astype(np.float32)     # amax 2^8 * 2^ex: element code 1.0 * 2^8
    W = np.repeat(4.0 * np.exp2(ew), 32, axis=1).astype(np.float32)
    if gkernel == 1 and bn not in (128, 256):
        pytest.skip("the one-CTA kernel has tiles of 128 and 256 features")
    if gkernel == 2 and bn in (320, 384):
        pytest.skip("only the wide-tile kernel has these widths")
    batq.batq_debug_force_tile_width(bn)
    try:
        got, Y, Sabs = _gemm_case(batq, S, M, N, 0, synth.f32_to_bf16_bits(X), synth.f32_to_bf16_bits(W))
    finally:
        batq.batq_debug_force_tile_width(0)
    want = 32 * 1024.0 * (np.exp2(ex.astype(np.float64)) @ np.exp2(ew.astype(np.float64)).T)
    assert np.array_equal(Y, want)
    # all terms are positive: k accumulating MMAs per output, each fp32 addition within 2^-23 of the running sum
    assert np.all(np.abs(got - want) <= k * 2.0 ** -23 * want)


def test_w4a8_distinct_codes_in_every_position(batq, gkernel):
    """Every K position of a block carries a different weight code and a different activation code,
    rows differ too: a permutation of elements inside a 16-code container, a swapped nibble or a
    shifted K sub-block changes the exact result."""
    S, M, N = 128, 128, 256
    rng = np.random.default_rng(3)
    X = rng.choice([0.5, 1, 1.5, 2, 3, 4, 6, -1, -2, -3, 8, 12, 16, 24, 28, -20], size=(S, N)).astype(np.float32)
    W = rng.choice([0.5, 1, 1.5, 2, 3, 4, 6, -0.5, -1, -1.5, -2, -3, -4, -6, 0], size=(M, N)).astype(np.float32)
    got, Y, Sabs = _gemm_case(batq, S, M, N, 0, synth.f32_to_bf16_bits(X), synth.f32_to_bf16_bits(W))
    assert np.array_equal(got, Y)          # small integers and halves: fp32 accumulation is exact


def test_w4a8_bf16_output_is_rounded_fp32(batq, gkernel):
    a, _, _ = _gemm_case(batq, 130, 264, 1024, 42, out_dtype=torch.float32)
    b, _, _ = _gemm_case(batq, 130, 264, 1024, 42, out_dtype=torch.bfloat16)
    want = torch.from_numpy(a.astype(np.float32)).bfloat16().float().numpy()
    assert np.array_equal(b.astype(np.float32), want)


@pytest.mark.parametrize("S,M,N,geometry", [(128, 1024, 1024, "baseline"), (128, 1024, 1024, "paper"),
                                            (50, 136, 640, "baseline"), (300, 520, 2048, "baseline"),
                                            (4, 1024, 1024, "baseline")])
def test_linear_w4a8_vs_oracle(batq, S, M, N, geometry):
    xb = synth.make_activations(S, N, synth.BASE_SEED)
    wb = synth.make_weight(M, N, synth.BASE_SEED)
    t = synth.make_transform(N, synth.BASE_SEED, geometry)
    tr = _mk(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    ws = batq.aligned_workspace(batq.batq_linear_w4a8_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a8(tr, w, batq.bits_to_cuda_bf16(xb), y, ws)
    assert batq.batq_last_device_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    Y, Sabs, _, _ = O.linear_w4a8(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)
    # a few activation codes may differ by one E4M3 step (fp32 vs fp64 transform): far inside the bound
    assert np.mean(np.abs(got - Y) > 1e-3 * Sabs + 1e-30) <= 1e-3
    assert np.linalg.norm(got - Y) <= 1e-4 * np.linalg.norm(Sabs)
    # and W4A8 is nearer the full-precision layer than W4A4 on the same inputs
    ref = O.bf16_bits_to_f64(xb) @ O.bf16_bits_to_f64(wb).T
    ws4 = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y4 = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, batq.bits_to_cuda_bf16(xb), y4, ws4)
    assert np.linalg.norm(got - ref) < np.linalg.norm(y4.cpu().numpy().astype(np.float64) - ref)


@pytest.mark.parametrize("N,M", [(4096, 6144), (4096, 28672)])
def test_w4a8_full_size_sampled(batq, N, M):
    """Config 1's qkv (2048 x 4096 -> 6144: CTA pairs with two accumulators) and gate/up (-> 28672:
    wide tiles) projections through the W4A8 layer in the launch configuration the benchmark times,
    bf16 output, checked on sampled rows and columns from the codes the GPU itself produced."""
    S = 2048
    rng = np.random.default_rng(11)
    xb = synth.make_activations(S, N, synth.BASE_SEED)
    wb = synth.make_weight(M, N, synth.BASE_SEED + 2)
    t = synth.make_transform(N, synth.BASE_SEED + 1, "baseline")
    tr = _mk(batq, t)
    x = batq.bits_to_cuda_bf16(xb)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    ws = batq.aligned_workspace(batq.batq_linear_w4a8_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
    batq.batq_linear_w4a8(tr, w, x, y, ws)
    assert batq.batq_last_device_status() == 0
    codes = torch.empty((S, N), dtype=torch.uint8, device="cuda")
    sf = torch.empty(batq.batq_sf_bytes(S, N, 1), dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act_mxfp8(tr, x, codes, sf, 1)
    rows = np.sort(rng.choice(S, size=48, replace=False))
    cols = np.sort(np.concatenate([rng.choice(M, size=376, replace=False), [0, 255, 256, 447, 448, M - 449, M - 257, M - 1]]))
    cols = np.unique(cols)
    gc = codes[torch.from_numpy(rows).cuda()].cpu().numpy()
    gs = sf_mma_to_rowmajor(sf.cpu().numpy(), S, N // 32)[rows]
    wc_d, wsc_d = batq.batq_weight_export(w)
    wc = O.unpack_codes(wc_d[torch.from_numpy(cols).cuda()].cpu().numpy())
    wsc = wsc_d[torch.from_numpy(cols).cuda()].cpu().numpy()
    Y, Sabs = O.gemm_mxfp8_mxfp4(gc, gs, wc, wsc)
    got = y[torch.from_numpy(rows).cuda()][:, torch.from_numpy(cols).cuda()].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - Y) <= 1e-3 * Sabs + 2.0 ** -8 * np.abs(Y) + 1e-30)


def test_w4a8_rejects_channel_counts_the_tensor_map_cannot_take(batq):
    N, M, S = 96, 64, 8      # n % 128 != 0
    w = batq.batq_prepare_weight(None, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 1)))
    z = torch.zeros(1 << 14, dtype=torch.uint8, device="cuda")
    y = torch.empty((S, M), dtype=torch.float32, device="cuda")
    with pytest.raises(batq.BatqError) as e:
        batq.batq_gemm_mxfp8_mxfp4(z, z, w, S, y)
    assert e.value.status == 4


def test_linear_w4a8_with_row_strides_and_bf16_output(batq):
    S, M, N = 200, 264, 1024
    xb = synth.make_activations(S, N, 61)
    t = synth.make_transform(N, 61, "baseline")
    tr = _mk(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 61)))
    ws = batq.aligned_workspace(batq.batq_linear_w4a8_workspace_bytes(w, S))
    x = batq.bits_to_cuda_bf16(xb)
    y32 = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a8(tr, w, x, y32, ws)
    xp = torch.zeros((S, N + 40), dtype=torch.bfloat16, device="cuda")
    xp[:, :N] = x
    yp = torch.full((S, M + 16), 3.0, dtype=torch.bfloat16, device="cuda")
    batq.batq_linear_w4a8(tr, w, xp[:, :N], yp[:, :M], ws)
    assert batq.batq_last_device_status() == 0
    assert torch.equal(yp[:, :M], y32.bfloat16()) and (yp[:, M:] == 3.0).all()


@pytest.mark.parametrize("S", [96, 2048])
def test_linear_w4a8_host_entry_point_matches_device_entry_point(batq, S):
    """Host buffers in and out for the W4A8 layer (row chunks from 512 tokens on): bit for bit the
    device entry point's result."""
    M, N = 520, 1024
    xb = synth.make_activations(S, N, 31)
    t = synth.make_transform(N, 31, "baseline")
    tr = _mk(batq, t)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 31)))
    ws = batq.aligned_workspace(batq.batq_linear_w4a8_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a8(tr, w, batq.bits_to_cuda_bf16(xb), y, ws)
    xh = torch.from_numpy(xb.view(np.int16)).pin_memory()
    yh = torch.full((S, M), float("nan"), dtype=torch.float32).pin_memory()
    xs = torch.empty((S, N), dtype=torch.bfloat16, device="cuda")
    ys = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a8_host_async(tr, w, xh, yh, xs, ys, ws)
    batq.batq_host_drain()
    assert batq.batq_last_device_status() == 0
    assert torch.equal(yh, y.cpu())
