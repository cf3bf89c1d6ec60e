"""The standalone quantiser at the sizes of the quantiser sweep (32768 tokens x {2048, 4096, 8192}
channels), in the launch configuration bench.py times (automatic kernel choice, tensor-core scale
layout): transform + clip to MXFP4 and to MXFP8, and the T = I ablation (plain MXFP4).  Checked on
sampled rows spread over the first, a middle and the last 128-token row tile plus random rows, and
on every element for 32768 x 2048."""
import numpy as np
import pytest
import torch

from oracle import batq_oracle as O
from paper_2603_16590_b200 import synth
from tests.helpers import code_mismatch_report, fp32_transform_bound, sf_mma_to_rowmajor

pytestmark = pytest.mark.gpu

S_BIG = 32768
FP32_REL = 15 * 2.0 ** -24   # a-priori bound of the fp32 transform, see test_gpu_parity.py


def _sample_rows(S, rng):
    mid = (S // 2 // 128) * 128
    rows = np.concatenate([np.arange(0, 128), np.arange(mid, mid + 128), np.arange(S - 128, S),
                           rng.choice(S, size=128, replace=False)])
    return np.unique(rows)


def _run_all(batq, xb, t):
    """Runs the four launches of the sweep on X; returns device tensors."""
    S, N = xb.shape
    tr = batq.batq_transform_create(N, t.left, t.right, t.clip_lo, t.clip_hi)
    x = batq.bits_to_cuda_bf16(xb)
    nsf = batq.batq_sf_bytes(S, N, batq.SF_MMA)
    out = {"vhat": torch.empty((S, N), dtype=torch.float32, device="cuda")}
    batq.batq_debug_transform_clip_f32(tr, x, out["vhat"])
    for name in ("gpk", "identity", "gpk8"):
        out[name + "_codes"] = torch.empty((S, N if name == "gpk8" else N // 2), dtype=torch.uint8, device="cuda")
        out[name + "_sf"] = torch.empty(nsf, dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act(tr, x, out["gpk_codes"], out["gpk_sf"], batq.SF_MMA)
    batq.batq_quantize_act(None, x, out["identity_codes"], out["identity_sf"], batq.SF_MMA)
    batq.batq_quantize_act_mxfp8(tr, x, out["gpk8_codes"], out["gpk8_sf"], batq.SF_MMA)
    assert batq.batq_last_device_status() == 0
    return out


def _rows_of(t, rows):
    return t[torch.from_numpy(rows).cuda()].cpu().numpy()


@pytest.mark.parametrize("N", [2048, 4096, 8192])
def test_config4_sizes_on_sampled_rows(batq, N):
    S, k = S_BIG, N // 32
    rng = np.random.default_rng(N)
    xb = synth.make_activations(S, N, synth.BASE_SEED + 4)
    t = synth.make_transform(N, synth.BASE_SEED + 5, "baseline")
    out = _run_all(batq, xb, t)
    rows = _sample_rows(S, rng)
    assert len(rows) >= 384 + 100
    V32 = _rows_of(out["vhat"], rows).astype(np.float64)

    # transform + clip -> MXFP4: bit-exact on the values the kernel rounded
    gc = O.unpack_codes(_rows_of(out["gpk_codes"], rows))
    gs = sf_mma_to_rowmajor(out["gpk_sf"].cpu().numpy(), S, k)[rows]
    oc, os_ = O.mxfp4_quantize(V32)
    assert np.array_equal(gs, os_) and np.array_equal(gc, oc)
    # ... and against the fp64 transform: differences only where the fp32 bound allows them
    V = O.transform_clip(xb[rows], t.left, t.right, t.clip_lo, t.clip_hi)
    X = np.abs(O.bf16_bits_to_f64(xb[rows])).reshape(len(rows), k, 32)
    unit = fp32_transform_bound(X, np.abs(O.block_matrices(t.left, t.right, k)), 2.0 ** -24)
    worst = float(np.max(np.abs(V32 - V) / np.maximum(unit, 1e-300)))
    assert worst <= 15.0, f"max |v^ - V| = {worst:.2f} x 2^-24 sum|x||P|"
    o64c, o64s = O.mxfp4_quantize(V)
    rep = code_mismatch_report(gc, gs, o64c, o64s, V, 15.0 * unit)
    print(f"{S}x{N} gpk mxfp4: max err {worst:.2f} x 2^-24 sum|x||P|; {rep}")
    assert rep["scale_unexplained"] == 0 and rep["scale_mismatch"] <= 1e-5 * rep["blocks"] + 1
    assert rep["code_mismatch"] <= 1e-4 * rep["elements"] + 1
    assert rep["unexplained"] == 0 and rep["not_neighbour"] == 0

    # transform + clip -> MXFP8: bit-exact on the same values
    g8 = _rows_of(out["gpk8_codes"], rows)
    g8s = sf_mma_to_rowmajor(out["gpk8_sf"].cpu().numpy(), S, k)[rows]
    o8, o8s = O.mxfp8_quantize(V32)
    assert np.array_equal(g8s, o8s) and np.array_equal(g8, o8)

    # T = I ablation (plain MXFP4 of X): bit-exact against the oracle, no transform involved
    ic = O.unpack_codes(_rows_of(out["identity_codes"], rows))
    is_ = sf_mma_to_rowmajor(out["identity_sf"].cpu().numpy(), S, k)[rows]
    oic, ois = O.quantize_act(xb[rows], None, None)
    assert np.array_equal(is_, ois) and np.array_equal(ic, oic)


def test_config4_32768x2048_every_element(batq):
    S, N = S_BIG, 2048
    k = N // 32
    xb = synth.make_activations(S, N, synth.BASE_SEED + 6)
    t = synth.make_transform(N, synth.BASE_SEED + 7, "baseline")
    out = _run_all(batq, xb, t)
    vhat = out["vhat"].cpu().numpy()
    gc_all = out["gpk_codes"].cpu().numpy()
    gs_all = sf_mma_to_rowmajor(out["gpk_sf"].cpu().numpy(), S, k)
    ic_all = out["identity_codes"].cpu().numpy()
    is_all = sf_mma_to_rowmajor(out["identity_sf"].cpu().numpy(), S, k)
    g8_all = out["gpk8_codes"].cpu().numpy()
    g8s_all = sf_mma_to_rowmajor(out["gpk8_sf"].cpu().numpy(), S, k)
    step = 2048
    for r0 in range(0, S, step):
        sl = slice(r0, r0 + step)
        V32 = vhat[sl].astype(np.float64)
        oc, os_ = O.mxfp4_quantize(V32)
        assert np.array_equal(gs_all[sl], os_) and np.array_equal(O.unpack_codes(gc_all[sl]), oc), f"rows {r0}.."
        o8, o8s = O.mxfp8_quantize(V32)
        assert np.array_equal(g8s_all[sl], o8s) and np.array_equal(g8_all[sl], o8), f"mxfp8 rows {r0}.."
        oic, ois = O.quantize_act(xb[sl], None, None)
        assert np.array_equal(is_all[sl], ois) and np.array_equal(O.unpack_codes(ic_all[sl]), oic), f"T=I rows {r0}.."
