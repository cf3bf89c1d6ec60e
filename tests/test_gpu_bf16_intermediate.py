"""The transform with BF16 intermediates (the paper keeps its pre-quantization transforms in BF16,
Sec. 3.2): kernel option against the oracle's emulation, and how far its codes are from the fp32
path's.  GPU only."""
import numpy as np
import pytest
import torch

from oracle import batq_oracle as O
from paper_2603_16590_b200 import synth

pytestmark = pytest.mark.gpu


def _mk(batq, t, on=True):
    tr = batq.batq_transform_create(t.n, t.left, t.right, t.clip_lo, t.clip_hi)
    batq.batq_transform_set_bf16_intermediates(tr, on)
    return tr


def _quantize(batq, tr, xb):
    S, N = xb.shape
    x = batq.bits_to_cuda_bf16(xb)
    codes = torch.empty((S, N // 2), dtype=torch.uint8, device="cuda")
    scales = torch.empty((S, N // 32), dtype=torch.uint8, device="cuda")
    batq.batq_quantize_act(tr, x, codes, scales, 0)
    vhat = torch.empty((S, N), dtype=torch.float32, device="cuda")
    batq.batq_debug_transform_clip_f32(tr, x, vhat)
    assert batq.batq_last_device_status() == 0
    return O.unpack_codes(codes.cpu().numpy()), scales.cpu().numpy(), vhat.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("S", [77, 300], ids=["perblock", "streaming"])
@pytest.mark.parametrize("geometry,clip", [("baseline", True), ("paper", False)])
def test_bf16_intermediates_vs_oracle_emulation(batq, S, geometry, clip):
    N = 1024
    xb = synth.make_activations(S, N, 900 + S)
    t = synth.make_transform(N, 31, geometry, clip=clip)
    gc, gs, vhat = _quantize(batq, _mk(batq, t), xb)
    # the quantiser itself: bit-exact on the values it rounded
    oc, os_ = O.mxfp4_quantize(vhat)
    assert np.array_equal(gs, os_) and np.array_equal(gc, oc)
    if not clip:
        assert np.array_equal(O.round_to_bf16(vhat), vhat)          # what leaves the transform is a bf16 tensor
    # the transform: equal to the oracle's emulation except where the fp32 sum of a contraction sits
    # within its own rounding error of a bf16 rounding boundary (then one bf16 step apart)
    V = O.transform_clip(xb, t.left, t.right, t.clip_lo, t.clip_hi, round_intermediate_bf16=True)
    far = np.abs(vhat - V) > 2.0 ** -20 * np.abs(V) + 1e-300
    print(f"bf16 intermediates {S}x{N} {geometry}: {far.mean():.2e} of the transformed values differ from the emulation")
    assert far.mean() <= 2e-3
    Xa = np.abs(O.bf16_bits_to_f64(xb)).reshape(S, N // 32, 32)
    bound = np.einsum("sje,jef->sjf", Xa, np.abs(O.block_matrices(t.left, t.right, N // 32))).reshape(S, N)
    assert np.all(np.abs(vhat - V) <= 2.0 ** -6 * bound + 1e-300)
    ec, es = O.mxfp4_quantize(V)
    assert (gs != es).mean() <= 1e-3
    assert (gc != ec).mean() <= 2e-3
    assert np.all(np.abs((gc & 7).astype(int) - (ec & 7).astype(int))[np.repeat(gs == es, 32, axis=1)] <= 1)


def test_code_mismatch_rate_against_the_fp32_path_on_config_0(batq):
    """Config 0 (128 x 1024): how many codes change when the transform stores bf16 intermediates,
    as the paper's implementation does, instead of staying in fp32."""
    S, N = 128, 1024
    xb = synth.make_activations(S, N, synth.BASE_SEED)
    t = synth.make_transform(N, synth.BASE_SEED, "baseline")
    c32, s32, _ = _quantize(batq, _mk(batq, t, on=False), xb)
    c16, s16, _ = _quantize(batq, _mk(batq, t, on=True), xb)
    same_scale = np.repeat(s32 == s16, 32, axis=1)
    rate = float((c32 != c16)[same_scale].mean())
    print(f"config 0: {rate:.4f} of the codes and {(s32 != s16).mean():.5f} of the scale bytes differ "
          f"between bf16 and fp32 intermediates")
    assert 0.0 < rate < 0.1 and (s32 != s16).mean() < 0.01
    # the oracle sees the same: its two modes differ at about the same rate
    o32 = O.quantize_act(xb, t.left, t.right, t.clip_lo, t.clip_hi)
    o16 = O.quantize_act(xb, t.left, t.right, t.clip_lo, t.clip_hi, round_intermediate_bf16=True)
    orate = float((o32[0] != o16[0])[np.repeat(o32[1] == o16[1], 32, axis=1)].mean())
    assert abs(rate - orate) <= 0.25 * orate + 1e-3


@pytest.mark.parametrize("S", [16, 100, 300])
def test_layer_with_bf16_intermediates_vs_oracle(batq, S):
    M, N = 264, 1024
    xb = synth.make_activations(S, N, 910 + S)
    wb = synth.make_weight(M, N, 911)
    t = synth.make_transform(N, 32, "baseline")
    tr = _mk(batq, t)
    assert batq.batq_linear_kernel_launches(tr, batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb)), S) == 2
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(wb))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    y = torch.empty((S, M), dtype=torch.float32, device="cuda")
    batq.batq_linear_w4a4(tr, w, batq.bits_to_cuda_bf16(xb), y, ws)
    assert batq.batq_last_device_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    qx = O.quantize_act(xb, t.left, t.right, t.clip_lo, t.clip_hi, round_intermediate_bf16=True)
    qw = O.prepare_weight(wb, t.left, t.right)
    Y, Sabs = O.gemm_mxfp4(qx[0], qx[1], qw[0], qw[1])
    assert np.mean(np.abs(got - Y) > 1e-3 * Sabs + 1e-30) <= 5e-3
    assert np.linalg.norm(got - Y) <= 3e-4 * np.linalg.norm(Sabs)


def test_bf16_intermediates_need_the_factored_4x8_form(batq):
    t = synth.make_transform(256, 3, "baseline", gr=8, gc=4)
    tr = batq.batq_transform_create(256, t.left, t.right, t.clip_lo, t.clip_hi, gr=8, gc=4)
    with pytest.raises(batq.BatqError) as e:
        batq.batq_transform_set_bf16_intermediates(tr, True)
    assert e.value.status == 4
    t = synth.make_transform(256, 3, "baseline")
    tr = _mk(batq, t)
    x = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    z = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(batq.BatqError) as e:
        batq.batq_quantize_act_mxfp8(tr, x, z, z, 0)
    assert e.value.status == 4


def test_switching_the_emulation_off_restores_the_fp32_path(batq):
    S, N = 50, 512
    xb = synth.make_activations(S, N, 41)
    t = synth.make_transform(N, 41, "paper")
    ref = _quantize(batq, _mk(batq, t, on=False), xb)
    tr = _mk(batq, t, on=True)
    on = _quantize(batq, tr, xb)
    batq.batq_transform_set_bf16_intermediates(tr, False)
    off = _quantize(batq, tr, xb)
    assert np.array_equal(off[0], ref[0]) and np.array_equal(off[1], ref[1]) and np.array_equal(off[2], ref[2])
    assert not np.array_equal(on[2], ref[2])
