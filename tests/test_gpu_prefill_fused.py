"""The prefill layer as ONE kernel (quantise phase + GEMM phase on the same grid of CTA pairs, the
quantiser-in-the-GEMM form of the path for s > 128) against the two-kernel path and the oracle."""
import numpy as np
import pytest
import torch

from oracle import batq_oracle as O
from paper_2603_16590_b200 import synth
from tests.helpers import sf_mma_to_rowmajor

pytestmark = pytest.mark.gpu


@pytest.fixture
def fused(batq):
    batq.batq_debug_force_prefill_path(2)
    yield
    batq.batq_debug_force_prefill_path(0)


def _layer(batq, S, M, N, seed, geometry="baseline", clip=True):
    t = synth.make_transform(N, seed, geometry, clip=clip)
    tr = batq.batq_transform_create(N, t.left, t.right, t.clip_lo, t.clip_hi)
    wb = synth.make_weight(M, N, seed)
    xb = synth.make_activations(S, N, seed)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    return t, tr, w, xb, wb


def _two_kernel(batq, tr, w, x, S, M, dtype):
    batq.batq_debug_force_prefill_path(1)
    try:
        ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
        y = torch.empty((S, M + (-M) % 8), dtype=dtype, device="cuda")[:, :M]
        batq.batq_linear_w4a4(tr, w, x, y, ws)
        torch.cuda.synchronize()
    finally:
        batq.batq_debug_force_prefill_path(2)
    return y


SHAPES = [(129, 520, 1024), (256, 192, 256), (300, 520, 2048), (520, 1032, 1024), (1000, 1100, 768), (257, 264, 3584),
          (2048, 1536, 4096)]


@pytest.mark.parametrize("S,M,N", SHAPES)
@pytest.mark.parametrize("geometry,clip", [("baseline", True), ("paper", False)])
def test_one_kernel_prefill_equals_two_kernels_and_tracks_the_oracle(batq, fused, S, M, N, geometry, clip):
    t, tr, w, xb, wb = _layer(batq, S, M, N, 2000 + S, geometry, clip)
    x = batq.bits_to_cuda_bf16(xb)
    assert batq.batq_linear_kernel_launches(tr, w, S) == 1
    nws = batq.batq_linear_workspace_bytes(w, S)
    ws = batq.aligned_workspace(nws + 64)
    ws.fill_(0xA7)                                   # stale bytes everywhere, counters included
    y = torch.full((S + 1, M + 8), float("nan"), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, x, y[:S, :M], ws[:nws])
    assert batq.batq_last_device_status() == 0
    assert (ws[nws:] == 0xA7).all(), "wrote past the workspace"
    yh = y.cpu().numpy()
    assert np.isnan(yh[S]).all() and np.isnan(yh[:S, M:]).all(), "wrote outside [S x M]"
    # the workspace holds the same codes and scale atoms as the standalone quantiser writes
    codes = torch.empty((S, N // 2), dtype=torch.uint8, device="cuda")
    sf = torch.zeros(batq.batq_sf_bytes(S, N, 1), dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act(tr, x, codes, sf, 1)
    assert torch.equal(ws[:S * N // 2].view(S, N // 2), codes)
    off = (S * N // 2 + 1023) // 1024 * 1024
    k = N // 32
    assert np.array_equal(sf_mma_to_rowmajor(ws[off:off + sf.numel()].cpu().numpy(), S, k),
                          sf_mma_to_rowmajor(sf.cpu().numpy(), S, k))
    # same kernels' arithmetic, same schedule: bit-identical to the two-kernel path, fp32 and bf16
    assert torch.equal(y[:S, :M], _two_kernel(batq, tr, w, x, S, M, torch.float32))
    yb = torch.empty((S, M + (-M) % 8), dtype=torch.bfloat16, device="cuda")[:, :M]
    batq.batq_linear_w4a4(tr, w, x, yb, ws[:nws])     # second call on the same workspace
    assert batq.batq_last_device_status() == 0
    assert torch.equal(yb, _two_kernel(batq, tr, w, x, S, M, torch.bfloat16))
    # and against the oracle
    if S * M * N <= 300 * 600 * 4096:
        got = yh[:S, :M].astype(np.float64)
        Y, Sabs, _, _ = O.linear_w4a4(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)
        assert np.mean(np.abs(got - Y) > 1e-3 * Sabs + 1e-30) <= 1e-3
        assert np.linalg.norm(got - Y) <= 1e-4 * np.linalg.norm(Sabs)


@pytest.mark.parametrize("S,N,M", [(2048, 4096, 6144), (2048, 14336, 4096), (8192, 3584, 4608)])
def test_one_kernel_prefill_at_benchmark_sizes(batq, fused, S, N, M):
    t, tr, w, xb, wb = _layer(batq, S, M, N, synth.BASE_SEED)
    x = batq.bits_to_cuda_bf16(xb)
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
    for _ in range(3):
        batq.batq_linear_w4a4(tr, w, x, y, ws)
    assert batq.batq_last_device_status() == 0
    assert torch.equal(y, _two_kernel(batq, tr, w, x, S, M, torch.bfloat16))


def test_one_kernel_prefill_in_a_replayed_graph(batq, fused):
    """Layers back to back on one workspace inside a replayed CUDA graph: every replay carries the
    same call tags, so the counters must be back at zero when a launch ends."""
    S = 300
    shapes = [(1024, 1536), (1024, 1024), (2048, 1024), (1024, 264)]   # (n, m)
    layers = []
    for i, (n, m) in enumerate(shapes):
        t, tr, w, xb, wb = _layer(batq, S, m, n, 60 + i)
        layers.append((tr, w, batq.bits_to_cuda_bf16(xb), m))
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
            for _ in range(2):
                for (tr, w, x, m), y in zip(layers, outs):
                    batq.batq_linear_w4a4(tr, w, x, y, ws)
        for _ in range(3):
            g.replay()
    torch.cuda.synchronize()
    assert batq.batq_last_device_status() == 0
    for a, b in zip(alone, outs):
        assert torch.equal(a, b)


def test_one_kernel_prefill_with_row_strides(batq, fused):
    """x with a row stride larger than n and y with a row stride larger than m: same bits as the
    dense call, nothing written between the rows."""
    S, M, N = 300, 520, 1024
    t, tr, w, xb, wb = _layer(batq, S, M, N, 77)
    x = batq.bits_to_cuda_bf16(xb)
    xp = torch.zeros((S, N + 72), dtype=torch.bfloat16, device="cuda")
    xp[:, :N] = x
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
    batq.batq_linear_w4a4(tr, w, x, y, ws)
    yp = torch.full((S, M + 24), 7.0, dtype=torch.bfloat16, device="cuda")
    batq.batq_linear_w4a4(tr, w, xp[:, :N], yp[:, :M], ws)
    assert batq.batq_last_device_status() == 0
    assert torch.equal(yp[:, :M], y) and (yp[:, M:] == 7.0).all()


def test_empty_batches_are_no_ops(batq):
    N, M = 256, 192
    t = synth.make_transform(N, 5, "baseline")
    tr = batq.batq_transform_create(N, t.left, t.right, t.clip_lo, t.clip_hi)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 5)))
    lib = batq.load()
    x = torch.zeros((8, N), dtype=torch.bfloat16, device="cuda")
    assert lib.batq_linear_w4a4(tr.handle, w.handle, x.data_ptr(), 0, N, None, 1, M, None, 0, None) == 0
    assert lib.batq_linear_w4a8(tr.handle, w.handle, x.data_ptr(), 0, N, None, 1, M, None, 0, None) == 0
    assert lib.batq_gemm_mxfp8_mxfp4(None, None, w.handle, 0, None, 1, M, None) == 0
