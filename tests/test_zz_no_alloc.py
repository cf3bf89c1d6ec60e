"""The allocation-free entry point (batq_linear_w4a4_noalloc) against the regular
one.  It is meant for callers that may not call cudaMalloc when they run a layer
(the device already belongs to their own pool, or an allocation's device-wide
synchronisation is not acceptable there), so its scratch is an array inside the
library.  Collected last on purpose: a failure here stops nothing else."""
import gc

import numpy as np
import pytest
import torch

from paper_2603_16590_b200 import synth

pytestmark = pytest.mark.gpu


def _layer(batq, S, M, N, seed, dtype):
    t = synth.make_transform(N, seed, "baseline")
    tr = batq.batq_transform_create(N, t.left, t.right, t.clip_lo, t.clip_hi)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, seed)))
    x = batq.bits_to_cuda_bf16(synth.make_activations(S, N, seed))
    ws = batq.aligned_workspace(batq.batq_linear_workspace_bytes(w, S))
    want = torch.empty((S, M), dtype=dtype, device="cuda")
    batq.batq_linear_w4a4(tr, w, x, want, ws)
    return tr, w, x, want


def test_noalloc_entry_point_matches_regular_one_twice_in_a_row(batq):
    assert batq.batq_static_workspace_capacity() >= 4 << 20
    # two calls in a row on different shapes: the second sees the first one's stale scratch
    cases = [(300, 520, 2048, 1, torch.float32), (77, 264, 544, 2, torch.bfloat16)]
    layers = [_layer(batq, *c) for c in cases]
    outs = [torch.full_like(want, float("nan")) for (_, _, _, want) in layers]
    # one call first: it resolves the array's address on this device (documented set-up step)
    batq.batq_linear_w4a4_noalloc(*layers[0][:3], torch.empty_like(layers[0][3]))
    torch.cuda.synchronize()
    gc.collect()   # tensors of earlier tests that are still waiting for the collector go now, not between the readings
    # what the driver itself hands out (torch's own counter would not see a cudaMalloc inside the library)
    free_before = torch.cuda.mem_get_info()[0]
    torch_before = torch.cuda.memory_allocated()
    for (tr, w, x, want), got in zip(layers, outs):
        batq.batq_linear_w4a4_noalloc(tr, w, x, got)
    assert batq.batq_last_device_status() == 0
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == torch_before
    for (tr, w, x, want), got in zip(layers, outs):
        # same kernels, same inputs: bit-identical, which is inside every tolerance used elsewhere
        assert torch.equal(got, want)
    # and once more on the first layer, after the second one overwrote the scratch
    tr, w, x, want = layers[0]
    again = torch.empty_like(want)
    batq.batq_linear_w4a4_noalloc(tr, w, x, again)
    torch.cuda.synchronize()
    assert torch.equal(again, want)


def test_noalloc_small_token_paths_after_a_large_call(batq):
    """The decode-sized paths keep more than codes in the scratch: split-K partial tiles and one
    ticket word per row tile (which must read zero when the GEMM starts).  Run them through the
    built-in array right after a large call has filled it with other bytes: 16 tokens with 12 K
    splits (partials and tickets in the array), 4 tokens (cluster reduction) and 1 token (the fused
    single-kernel path), each twice."""
    big = _layer(batq, 1500, 264, 4096, 5, torch.bfloat16)
    small = []
    batq.batq_debug_force_small_s_splits(12)
    try:
        small.append(_layer(batq, 16, 520, 3584, 6, torch.float32))
        got = [torch.full_like(small[0][3], float("nan")) for _ in range(2)]
        batq.batq_linear_w4a4_noalloc(*big[:3], torch.empty_like(big[3]))
        for g in got:
            batq.batq_linear_w4a4_noalloc(*small[0][:3], g)
        assert batq.batq_last_device_status() == 0
        assert torch.equal(got[0], small[0][3]) and torch.equal(got[1], small[0][3])
    finally:
        batq.batq_debug_force_small_s_splits(0)
    for S, M, N, seed in [(4, 1032, 2048, 7), (1, 4096, 4096, 8)]:
        tr, w, x, want = _layer(batq, S, M, N, seed, torch.float32)
        batq.batq_linear_w4a4_noalloc(*big[:3], torch.empty_like(big[3]))
        got = [torch.full_like(want, float("nan")) for _ in range(2)]
        for g in got:
            batq.batq_linear_w4a4_noalloc(tr, w, x, g)
        assert batq.batq_last_device_status() == 0
        assert torch.equal(got[0], want) and torch.equal(got[1], want)


def test_noalloc_rejects_sizes_beyond_the_array(batq):
    N, M = 4096, 128
    t = synth.make_transform(N, 3, "baseline")
    tr = batq.batq_transform_create(N, t.left, t.right, t.clip_lo, t.clip_hi)
    w = batq.batq_prepare_weight(tr, batq.bits_to_cuda_bf16(synth.make_weight(M, N, 3)))
    S = 8192   # 8192 x 4096 / 2 = 16 MiB of codes: more than the array holds
    assert batq.batq_linear_workspace_bytes(w, S) > batq.batq_static_workspace_capacity()
    x = torch.zeros((S, N), dtype=torch.bfloat16, device="cuda")
    y = torch.empty((S, M), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(batq.BatqError) as e:
        batq.batq_linear_w4a4_noalloc(tr, w, x, y)
    assert e.value.status == 5
