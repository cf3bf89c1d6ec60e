"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (whole-layer
entry point, bf16 output, automatic kernel choice), on samples the oracle can compute one by one:
token rows for the quantiser, weight rows for the offline fusion, (row, column) entries for the GEMM."""
import numpy as np
import pytest
import torch

from oracle import batq_oracle as O
from paper_2603_16590_b200 import synth
from tests.helpers import code_mismatch_report, fp32_transform_bound, sf_mma_to_rowmajor

pytestmark = pytest.mark.gpu

FP32_REL = 15 * 2.0 ** -24   # a-priori bound of the fp32 transform, see test_gpu_parity.py

CASES = [  # (tokens, projection list entry, vision-row fraction, outlier-channel fraction)
    (2048, synth.LLAMA8B_PREFILL[0], 0.0, 0.01), (2048, synth.LLAMA8B_PREFILL[1], 0.0, 0.01),
    (2048, synth.LLAMA8B_PREFILL[2], 0.0, 0.01), (2048, synth.LLAMA8B_PREFILL[3], 0.0, 0.01),
    (8192, synth.QWEN2VL7B_PREFILL[0], 0.75, 0.005), (8192, synth.QWEN2VL7B_PREFILL[3], 0.75, 0.005),
    (16, synth.LLAMA8B_PREFILL[2], 0.0, 0.01), (1, synth.LLAMA8B_PREFILL[3], 0.0, 0.01),
]


@pytest.mark.parametrize("S,proj,vis,och", CASES, ids=[f"{c[0]}x{c[1][0]}_{c[1][1]}to{c[1][2]}" for c in CASES])
def test_full_size_layer_on_samples(batq, S, proj, vis, och):
    name, N, M = proj
    k = N // 32
    rng = np.random.default_rng(S + M)
    xb = synth.make_activations(S, N, synth.BASE_SEED, outlier_channel_frac=och, vision_rows=int(S * vis))
    wb = synth.make_weight(M, N, synth.BASE_SEED + 2)
    t = synth.make_transform(N, synth.BASE_SEED + 1, "baseline")
    tr = batq.batq_transform_create(N, t.left, t.right, t.clip_lo, t.clip_hi)
    x = batq.bits_to_cuda_bf16(xb)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
    batq.batq_linear_w4a4(tr, w, x, y, ws)
    assert batq.batq_last_device_status() == 0

    # --- offline weight fusion on sampled weight rows
    wrows = np.sort(rng.choice(M, size=min(M, 96), replace=False))
    wc_d, wsc_d = batq.batq_weight_export(w)
    wc = O.unpack_codes(wc_d[torch.from_numpy(wrows).cuda()].cpu().numpy())
    wsc = wsc_d[torch.from_numpy(wrows).cuda()].cpu().numpy()
    oc, osc = O.prepare_weight(wb[wrows], t.left, t.right)
    assert (wsc != osc).mean() <= 1e-5
    assert ((wc != oc) & np.repeat(wsc == osc, 32, axis=1)).mean() <= 1e-5

    # --- activation quantiser on sampled token rows (the same kernel choice as the layer call)
    codes = torch.empty((S, N // 2), dtype=torch.uint8, device="cuda")
    sf = torch.empty(batq.batq_sf_bytes(S, N, 1), dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act(tr, x, codes, sf, 1)
    xrows = np.sort(rng.choice(S, size=min(S, 48), replace=False))
    gc = O.unpack_codes(codes[torch.from_numpy(xrows).cuda()].cpu().numpy())
    gs = sf_mma_to_rowmajor(sf.cpu().numpy(), S, k)[xrows]
    V = O.transform_clip(xb[xrows], t.left, t.right, t.clip_lo, t.clip_hi)
    oc, os_ = O.mxfp4_quantize(V)
    X = np.abs(O.bf16_bits_to_f64(xb[xrows])).reshape(len(xrows), k, 32)
    P = np.abs(O.block_matrices(t.left, t.right, k))
    bound = fp32_transform_bound(X, P, FP32_REL)
    rep = code_mismatch_report(gc, gs, oc, os_, V, bound)
    print(f"{name} {S}x{N}: {rep}")
    # scale bytes bit-exact unless amax sits within the fp32 bound of a power of two
    assert rep["scale_unexplained"] == 0 and rep["scale_mismatch"] <= 1e-4 * rep["blocks"] + 1
    assert rep["code_mismatch"] <= 1e-4 * rep["elements"] + 1
    assert rep["unexplained"] == 0 and rep["not_neighbour"] == 0

    # --- GEMM on sampled outputs, from the codes and scales the GPU itself produced
    cols = np.sort(rng.choice(M, size=min(M, 384), replace=False))
    wcols_c = O.unpack_codes(wc_d[torch.from_numpy(cols).cuda()].cpu().numpy())
    wcols_s = wsc_d[torch.from_numpy(cols).cuda()].cpu().numpy()
    Y, Sabs = O.gemm_mxfp4(gc, gs, wcols_c, wcols_s)
    got = y[torch.from_numpy(xrows).cuda()][:, torch.from_numpy(cols).cuda()].float().cpu().numpy().astype(np.float64)
    # bf16 output: the fp32 accumulator within 1e-3 * Sabs, then one bf16 rounding (2^-9 relative)
    assert np.all(np.abs(got - Y) <= 1e-3 * Sabs + 2.0 ** -8 * np.abs(Y) + 1e-30)
    # the layer call quantised X itself: it must have used the same codes (deterministic kernels)
    y2 = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
    batq.batq_linear_w4a4(tr, w, x, y2, ws)
    assert torch.equal(y, y2)
