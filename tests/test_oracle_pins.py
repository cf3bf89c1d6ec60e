"""Pins for the CPU oracle: everything here is fixed by the paper or by
mathematics, not by the oracle itself.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import batq_oracle as O
from paper_2603_16590_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- E2M1 grid
def test_e2m1_decode_matches_paper_value_list():
    vals = [float(v) for v in _rows("e2m1_values.txt")[0]]
    assert len(vals) == 7
    # codes 1..7 are the 7 positive values in increasing order, 0 is zero,
    # codes 8..15 their negatives
    assert list(O.e2m1_decode(np.arange(1, 8))) == vals
    assert O.e2m1_decode(np.array([0]))[0] == 0.0
    assert list(O.e2m1_decode(np.arange(9, 16))) == [-v for v in vals]
    # bit layout 1 sign / 2 exponent / 1 mantissa: value = (-1)^s 2^(E-1) (1 + M/2), E>0; M/2 for E=0
    for code in range(16):
        s, E, M = code >> 3, (code >> 1) & 3, code & 1
        v = (M * 0.5) if E == 0 else (2.0 ** (E - 1)) * (1 + M / 2)
        assert O.e2m1_decode(np.array([code]))[0] == (-v if s else v)


def test_e2m1_roundtrip_all_16_codes():
    codes = np.arange(16, dtype=np.uint8)
    back = O.e2m1_round_code(O.e2m1_decode(codes))
    assert np.array_equal(back, codes)  # includes -0 -> 0x8


def test_e2m1_rounding_hand_worked_cases():
    for val, code, *_ in _rows("e2m1_rounding_cases.txt"):
        got = int(O.e2m1_round_code(np.array([float(val)]))[0])
        assert got == int(code, 16), (val, hex(got), code)


def test_e2m1_rounding_threshold_table():
    """Independent statement of RNE as interval tests on |u|."""
    def ref(u):
        a = abs(u)
        if a <= 0.25: c = 0
        elif a < 0.75: c = 1
        elif a <= 1.25: c = 2
        elif a < 1.75: c = 3
        elif a <= 2.5: c = 4
        elif a < 3.5: c = 5
        elif a <= 5.0: c = 6
        else: c = 7
        return c | (8 if np.signbit(u) else 0)
    grid = np.concatenate([np.linspace(-9, 9, 7201), np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]),
                           np.nextafter(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]), 10),
                           np.nextafter(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]), -10)])
    got = O.e2m1_round_code(grid)
    assert [int(c) for c in got] == [ref(float(u)) for u in grid]


def test_e2m1_rounding_is_nearest_and_monotone_and_idempotent():
    rng = np.random.default_rng(0)
    u = rng.uniform(-8, 8, 20000)
    q = O.e2m1_decode(O.e2m1_round_code(u))
    # nearest: no grid value is strictly closer (brute force over all 15 values)
    allv = np.unique(O.e2m1_decode(np.arange(16)))
    assert np.all(np.abs(q - u)[:, None] <= np.abs(allv[None, :] - u[:, None]) + 0.0)
    us = np.sort(u)
    assert np.all(np.diff(O.e2m1_decode(O.e2m1_round_code(us))) >= 0)
    assert np.array_equal(O.e2m1_round_code(q), O.e2m1_round_code(u))


# ---------------------------------------------------------------- MX scale
def test_mx_scale_hand_worked_cases():
    for amax, e, byte, code in _rows("mx_scale_cases.txt"):
        v = np.zeros((1, 32)); v[0, 5] = float(amax)
        codes, sb = O.mxfp4_quantize(v)
        assert int(O.mx_scale_exponent(np.array(float(amax)))) == int(e)
        assert int(sb[0, 0]) == int(byte)
        assert int(codes[0, 5]) == int(code, 16)
        assert not codes[0, np.arange(32) != 5].any()


def test_mx_scale_closed_form_and_invariant():
    rng = np.random.default_rng(1)
    amax = np.exp2(rng.uniform(-100, 100, 5000))
    e = O.mx_scale_exponent(amax)
    r = amax / np.exp2(e.astype(float))
    assert np.all((r >= 4) & (r < 8))          # amax / 2^e in [4, 8)
    # exact powers of two and their neighbours
    for p in range(-120, 121):
        x = 2.0 ** p
        assert O.mx_scale_exponent(np.array(x)) == p - 2
        assert O.mx_scale_exponent(np.nextafter(x, 0)) == p - 3
        assert O.mx_scale_exponent(np.nextafter(x, np.inf)) == p - 2
    # clamping to the UE8M0 range
    assert O.mx_scale_exponent(np.array(2.0 ** -140)) == -127
    assert O.mx_scale_exponent(np.array(2.0 ** 200)) == 127
    assert O.mx_scale_exponent(np.array(0.0)) == -127


def test_zero_block_and_sign_of_zero():
    v = np.zeros((1, 64)); v[0, 3] = -0.0
    codes, sb = O.mxfp4_quantize(v)
    assert sb[0, 0] == 0 and sb[0, 1] == 0
    assert codes[0, 3] == 8 and codes[0, 0] == 0


def test_quantize_dequantize_error_bound():
    """Within a block no element is off by more than half the largest grid step
    (1 at |u| in [4,6]) times the scale, except saturated ones (|u| in (6,8))."""
    rng = np.random.default_rng(2)
    V = rng.standard_normal((50, 128)) * np.exp2(rng.integers(-20, 20, (50, 1)))
    codes, sb = O.mxfp4_quantize(V)
    D = O.dequantize(codes, sb)
    scale = np.repeat(np.exp2(sb.astype(float) - 127), 32, axis=1)
    assert np.all(np.abs(D - V) <= 2.0 * scale + 1e-300)
    u = np.abs(V) / scale
    ok = u <= 6
    assert np.all(np.abs(D - V)[ok] <= 1.0 * scale[ok])


def test_pack_order_low_nibble_is_even_element():
    c = np.array([[1, 2, 0xF, 0x8]], dtype=np.uint8)
    p = O.pack_codes(c)
    assert list(p[0]) == [0x21, 0x8F]
    assert np.array_equal(O.unpack_codes(p), c)


# ---------------------------------------------------------------- transform
def _rand_factors(k, seed, geometry):
    t = synth.make_transform(32 * k, seed, geometry)
    return t


@pytest.mark.parametrize("geometry", ["baseline", "paper", "naive"])
def test_fast_form_equals_dense_kronecker(geometry):
    k = 5
    t = _rand_factors(k, 11, geometry)
    rng = np.random.default_rng(3)
    X = rng.standard_normal((7, 32 * k))
    dense = O.transform_dense(X, O.block_matrices(t.left, t.right, k))
    fast = O.transform_fast(X, t.left, t.right)
    assert np.allclose(dense, fast, rtol=0, atol=1e-12)


def test_kron_dense_matches_numpy_kron_and_index_order():
    rng = np.random.default_rng(4)
    L, R = rng.standard_normal((4, 4)), rng.standard_normal((8, 8))
    assert np.array_equal(O.kron_dense(L, R), np.kron(L, R))
    # element (r,c) of the block is index r*8+c: a right factor that shifts the
    # contiguous index by one moves element e to e+1 inside each run of 8
    shift = np.roll(np.eye(8), 1, axis=1)
    P = O.kron_dense(np.eye(4), shift)
    x = np.arange(32.0)[None, :]
    y = O.transform_dense(x, P[None])
    assert y[0, 1] == 0.0 and y[0, 0] == 7.0 and y[0, 9] == 8.0
    # a left factor that shifts the slow index moves element e to e+8
    P = O.kron_dense(np.roll(np.eye(4), 1, axis=1), np.eye(8))
    y = O.transform_dense(x, P[None])
    assert y[0, 8] == 0.0 and y[0, 0] == 24.0


def test_vec_identity_of_the_paper():
    """vec(V)(B (x) A) = vec(B^T V A) with row-major vec, for V g2 x g1."""
    rng = np.random.default_rng(5)
    B, A, V = rng.standard_normal((4, 4)), rng.standard_normal((8, 8)), rng.standard_normal((4, 8))
    lhs = V.reshape(1, 32) @ np.kron(B, A)
    rhs = (B.T @ V @ A).reshape(1, 32)
    assert np.allclose(lhs, rhs, atol=1e-13)
    assert np.allclose(O.transform_fast(V.reshape(1, 32), B[None], A[None]), rhs, atol=1e-13)


def test_block_isolation_bitwise():
    k = 6
    t = _rand_factors(k, 12, "baseline")
    P = O.block_matrices(t.left, t.right, k)
    rng = np.random.default_rng(6)
    X = rng.standard_normal((4, 32 * k))
    base = O.transform_dense(X, P)
    X2 = X.copy(); X2[:, 64:96] += 1000.0 * rng.standard_normal((4, 32))
    pert = O.transform_dense(X2, P)
    same = np.ones(32 * k, bool); same[64:96] = False
    assert np.array_equal(base[:, same], pert[:, same])
    assert not np.array_equal(base[:, ~same], pert[:, ~same])


def test_inverse_recovers_input():
    k = 4
    for geometry in ("baseline", "paper"):
        t = _rand_factors(k, 13, geometry)
        P = O.block_matrices(t.left, t.right, k)
        Pinv = O.invert_blocks(P)
        for j in range(k):
            assert np.allclose(Pinv[j] @ P[j], np.eye(32), atol=1e-12)
        rng = np.random.default_rng(7)
        X = rng.standard_normal((9, 32 * k))
        assert np.allclose(O.transform_dense(O.transform_dense(X, P), Pinv), X, rtol=0, atol=1e-12)


def test_table1_parameter_counts():
    want = {name: int(v) for name, v in _rows("table1_param_counts.txt")}
    N, g, g1, g2 = 4096, 32, 8, 4
    k = N // g
    paper = synth.make_transform(N, 1, "paper", clip=False)
    naive = synth.make_transform(N, 1, "naive", clip=False)
    assert paper.left.size + paper.right.size == want["gpk"] == g1 * g1 + k * g2 * g2
    assert naive.left.size + naive.right.size == want["naive_kronecker"]
    assert O.block_matrices(paper.left, paper.right, k).size == want["block_diag_no_decomposition"]
    assert 2 * N == want["flatquant_kronecker"]


def test_identity_transform_is_plain_mxfp4():
    xb = synth.make_activations(16, 256, 5)
    t = synth.make_transform(256, 5, identity=True, clip=False)
    a = O.quantize_act(xb, t.left, t.right)
    b = O.quantize_act(xb, None, None)
    c = O.mxfp4_quantize(O.bf16_bits_to_f64(xb))
    for u, v, w in zip(a, b, c):
        assert np.array_equal(u, v) and np.array_equal(v, w)


def test_bf16_decode_exact():
    bits = np.array([0x3F80, 0xBF80, 0x0000, 0x8000, 0x4049, 0x7F7F, 0x0080], dtype=np.uint16)
    want = [1.0, -1.0, 0.0, -0.0, 3.140625, 3.3895313892515355e38, 2.0 ** -126]
    got = O.bf16_bits_to_f64(bits)
    assert list(got) == want and np.signbit(got[3])
    # synth's rounding is nearest-even: 1 + 2^-8 is a tie -> 1.0; 1 + 3*2^-8 -> 1 + 2^-6
    r = synth.f32_to_bf16_bits(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20], np.float32))
    assert list(r) == [0x3F80, 0x3F82, 0x3F81]


# ---------------------------------------------------------------- clip
def test_clip_cases():
    k = 2
    V = np.zeros((1, 64))
    V[0, :32] = np.linspace(-4, 8, 32)       # mixed signs
    V[0, 32:] = np.linspace(0.9, 1.0, 32)    # all positive: lo > hi possible
    one = np.ones(k)
    assert np.array_equal(O.block_clip(V, one, one), V)       # ratio 1 = identity
    out = O.block_clip(V, np.array([0.5, 1.0]), np.array([0.75, 0.8]))
    assert out[0, :32].min() == -2.0 and out[0, :32].max() == 6.0
    inner = (V[0, :32] > -2) & (V[0, :32] < 6)
    assert np.array_equal(out[0, :32][inner], V[0, :32][inner])
    assert np.all(out[0, 32:] == 0.8)   # clamp order min(max(v,lo),hi): every element = hi
    # monotone in the ratio: tighter ratio never widens the range
    prev = np.inf
    for r in (1.0, 0.9, 0.8, 0.5):
        w = np.ptp(O.block_clip(V, np.full(k, r), np.full(k, r))[0, :32])
        assert w <= prev; prev = w
    # per-row ratios (weights): shape [S, k]
    V2 = np.vstack([V, V])
    out2 = O.block_clip(V2, np.array([[1, 1], [0.5, 1.0]]), np.array([[1, 1], [0.75, 0.8]]))
    assert np.array_equal(out2[0], V[0]) and np.array_equal(out2[1], out[0])


# ---------------------------------------------------------------- weights + whole pipeline
@pytest.mark.parametrize("geometry", ["baseline", "paper"])
def test_unquantized_pipeline_identity(geometry):
    """(X P)(W P^-T)^T = X W^T: catches every transpose / order error."""
    S, M, N = 6, 5, 128
    xb = synth.make_activations(S, N, 21)
    wb = synth.make_weight(M, N, 21)
    t = synth.make_transform(N, 21, geometry, clip=False)
    Xt = O.transform_clip(xb, t.left, t.right)
    Wt = O.transform_weight(wb, t.left, t.right)
    X, W = O.bf16_bits_to_f64(xb), O.bf16_bits_to_f64(wb)
    ref = X @ W.T
    got = Xt @ Wt.T
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-12 * np.abs(X) @ np.abs(W).T)
    # and a wrong reading (W P^-1 instead of W P^-T) must fail it
    k = N // 32
    Pinv = O.invert_blocks(O.block_matrices(t.left, t.right, k))
    wrong = O.transform_dense(W, Pinv)
    assert not np.allclose(Xt @ wrong.T, ref, rtol=1e-6)


def test_gemm_exact_integer_variant_and_unit_scales():
    rng = np.random.default_rng(8)
    S, M, N = 3, 4, 96
    cx = rng.integers(0, 16, (S, N)).astype(np.uint8)
    cw = rng.integers(0, 16, (M, N)).astype(np.uint8)
    sx = rng.integers(120, 135, (S, N // 32)).astype(np.uint8)
    sw = rng.integers(120, 135, (M, N // 32)).astype(np.uint8)
    Y, Sabs = O.gemm_mxfp4(cx, sx, cw, sw)
    Yi = O.gemm_mxfp4_exact_int(cx, sx, cw, sw)
    assert np.array_equal(Y, Yi)   # small exponents: fp64 sum is exact too
    assert np.all(np.abs(Y) <= Sabs)
    # Sabs pinned from both sides: with every sign bit cleared no product is negative, so the exact
    # contraction of the magnitudes *is* sum |a*b| (Python integers and fractions, no floating point)
    Sabs_exact = O.gemm_mxfp4_exact_int(cx & 7, sx, cw & 7, sw)
    assert np.array_equal(Sabs, Sabs_exact)
    assert np.all(Sabs_exact >= np.abs(Yi)) and np.any(Sabs_exact > np.abs(Yi))
    # all scales 2^0: plain integer dot product of doubled values / 4
    one = np.full((S, N // 32), 127, np.uint8)
    Y1, _ = O.gemm_mxfp4(cx, one, cw, np.full((M, N // 32), 127, np.uint8))
    ix = np.rint(2 * O.e2m1_decode(cx)).astype(int); iw = np.rint(2 * O.e2m1_decode(cw)).astype(int)
    assert np.array_equal(Y1, (ix @ iw.T) / 4.0)


def test_quantized_linear_is_close_to_fp():
    """Sanity of the whole oracle pipeline: W4A4 output correlates with the
    full-precision layer (not a paper number -- just guards gross errors)."""
    S, M, N = 32, 48, 256
    xb = synth.make_activations(S, N, 31)
    wb = synth.make_weight(M, N, 31)
    t = synth.make_transform(N, 31, "baseline")
    Y, Sabs, _, _ = O.linear_w4a4(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)
    ref = O.bf16_bits_to_f64(xb) @ O.bf16_bits_to_f64(wb).T
    rel = np.linalg.norm(Y - ref) / np.linalg.norm(ref)
    assert rel < 0.35


# ---------------------------------------------------------------- E4M3 / MXFP8
def test_e4m3_decode_against_the_format_definition():
    """1 sign / 4 exponent (bias 7) / 3 mantissa; the values the OCP format fixes."""
    d = O.e4m3_decode(np.arange(256, dtype=np.uint8))
    assert d[0] == 0.0 and d[1] == 2.0 ** -9 and d[7] == 7 * 2.0 ** -9      # subnormals
    assert d[8] == 2.0 ** -6 and d[0x38] == 1.0 and d[0x40] == 2.0          # normals
    assert d[0x7E] == 448.0 and np.isnan(d[0x7F]) and np.isnan(d[0xFF])     # largest finite, NaN
    assert np.array_equal(d[128:255], -d[0:127])
    assert np.all(np.diff(d[:127]) > 0)                                      # codes ordered like values


def test_e4m3_rounding_against_torch_float8():
    """An independent implementation of the same format: torch's float8_e4m3fn cast
    (round-to-nearest-even) inside the finite range."""
    import torch
    rng = np.random.default_rng(4)
    u = np.concatenate([rng.uniform(-448, 448, 20000), rng.standard_normal(20000) * 0.01,
                        rng.standard_normal(5000) * 2.0 ** -8, np.array([0.0, -0.0, 448.0, -448.0, 2.0 ** -10])])
    u = u.astype(np.float32).astype(np.float64)       # torch casts from fp32
    want = torch.from_numpy(u.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = O.e4m3_round_code(u)
    assert np.array_equal(got & 0x7F, want & 0x7F)
    nz = (got & 0x7F) != 0
    assert np.array_equal(got[nz], want[nz])          # signs (torch may drop the sign of a zero result)


def test_e4m3_rounding_properties():
    codes = np.arange(127, dtype=np.uint8)
    vals = O.e4m3_decode(codes)
    assert np.array_equal(O.e4m3_round_code(vals), codes)                    # grid points are fixed points
    mids = (vals[:-1] + vals[1:]) / 2                                         # exact ties
    tie = O.e4m3_round_code(mids)
    assert np.all(tie % 2 == 0) and np.all((tie == codes[:-1]) | (tie == codes[1:]))
    assert O.e4m3_round_code(np.array([1e9]))[0] == 0x7E and O.e4m3_round_code(np.array([-500.0]))[0] == 0xFE
    assert O.e4m3_round_code(np.array([-0.0]))[0] == 0x80
    rng = np.random.default_rng(5)
    u = np.sort(rng.uniform(-500, 500, 5000))
    assert np.all(np.diff(O.e4m3_decode(O.e4m3_round_code(u))) >= 0)          # monotone


def test_mxfp8_scale_rule_and_error_bound():
    rng = np.random.default_rng(6)
    V = rng.standard_normal((40, 128)) * np.exp2(rng.integers(-30, 30, (40, 1)))
    codes, sb = O.mxfp8_quantize(V)
    amax = np.abs(V).reshape(40, 4, 32).max(axis=2)
    r = amax / np.exp2(sb.astype(float) - 127)
    assert np.all((r >= 256) & (r < 512))            # amax / 2^e in [2^8, 2^9): e = floor(log2 amax) - 8
    D = O.dequantize_mxfp8(codes, sb)
    scale = np.repeat(np.exp2(sb.astype(float) - 127), 32, axis=1)
    u = np.abs(V) / scale
    ok = u <= 448
    assert np.all(np.abs(D - V)[ok] <= np.maximum(2.0 ** -4 * np.abs(V)[ok], 2.0 ** -10 * scale[ok]))  # half an ulp
    assert np.all(np.abs(D)[~ok] == 448 * scale[~ok])                          # (448, 512) saturates
    z = np.zeros((1, 32)); z[0, 3] = -0.0
    c, s_ = O.mxfp8_quantize(z)
    assert s_[0, 0] == 0 and c[0, 3] == 0x80 and c[0, 0] == 0


def test_w4a8_gemm_exact_rational_variant_and_sabs():
    """MXFP8 x MXFP4 contraction: fp64 equals the exact rational evaluation on tiny shapes, Sabs
    equals the exact contraction of the magnitudes, and with unit scales the result is the integer
    dot product of (512 * e4m3) and (2 * e2m1) over 1024."""
    rng = np.random.default_rng(18)
    S, M, N = 3, 4, 96
    cx = rng.integers(0, 256, (S, N)).astype(np.uint8)
    cx[(cx & 0x7F) == 0x7F] = 0x7E                      # no NaN codes
    cw = rng.integers(0, 16, (M, N)).astype(np.uint8)
    sx = rng.integers(120, 135, (S, N // 32)).astype(np.uint8)
    sw = rng.integers(120, 135, (M, N // 32)).astype(np.uint8)
    Y, Sabs = O.gemm_mxfp8_mxfp4(cx, sx, cw, sw)
    assert np.array_equal(Y, O.gemm_mxfp8_mxfp4_exact(cx, sx, cw, sw))
    assert np.array_equal(Sabs, O.gemm_mxfp8_mxfp4_exact(cx & 0x7F, sx, cw & 7, sw))
    assert np.all(np.abs(Y) <= Sabs)
    one_x, one_w = np.full((S, N // 32), 127, np.uint8), np.full((M, N // 32), 127, np.uint8)
    Y1, _ = O.gemm_mxfp8_mxfp4(cx, one_x, cw, one_w)
    ix = np.rint(512 * O.e4m3_decode(cx)).astype(np.int64)
    iw = np.rint(2 * O.e2m1_decode(cw)).astype(np.int64)
    assert np.array_equal(Y1, (ix @ iw.T) / 1024.0)


def test_w4a8_layer_is_closer_to_fp_than_w4a4():
    """The 8-bit activation format loses less than the 4-bit one (the paper's W4A8 rows sit above
    its W4A4 rows): on the same layer the W4A8 oracle output is nearer the full-precision product."""
    S, M, N = 32, 48, 256
    xb = synth.make_activations(S, N, 33)
    wb = synth.make_weight(M, N, 33)
    t = synth.make_transform(N, 33, "baseline")
    ref = O.bf16_bits_to_f64(xb) @ O.bf16_bits_to_f64(wb).T
    y8 = O.linear_w4a8(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)[0]
    y4 = O.linear_w4a4(xb, wb, t.left, t.right, t.clip_lo, t.clip_hi)[0]
    assert np.linalg.norm(y8 - ref) < np.linalg.norm(y4 - ref)
    # unquantised activations would leave only the weight error: W4A8 must sit between the two
    assert np.linalg.norm(y8 - ref) / np.linalg.norm(ref) < 0.35


def test_round_to_bf16_against_torch_and_the_format():
    """An independent implementation of the same rounding: torch's float32 -> bfloat16 cast."""
    import torch
    rng = np.random.default_rng(21)
    v = np.concatenate([rng.standard_normal(50000) * np.exp2(rng.integers(-40, 40, 50000)),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -257.0, 255.5])])
    v = v.astype(np.float32).astype(np.float64)
    want = torch.from_numpy(v.astype(np.float32)).bfloat16().float().numpy().astype(np.float64)
    got = O.round_to_bf16(v)
    assert np.array_equal(got, want)
    assert np.array_equal(O.round_to_bf16(got), got)                         # idempotent
    assert O.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0            # tie -> even mantissa
    assert O.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    bits = synth.f32_to_bf16_bits(v.astype(np.float32))                       # the input generator's own rounding agrees
    assert np.array_equal(O.bf16_bits_to_f64(bits), got)


def test_bf16_intermediate_transform_properties():
    """With values that need no rounding (small integers, integer factors) the BF16 form equals the
    exact transform; in general it differs from it by at most the two roundings (2^-8 relative each,
    propagated through the second contraction)."""
    rng = np.random.default_rng(22)
    S, N = 5, 96
    X = rng.integers(-3, 4, (S, N)).astype(np.float64)
    L = rng.integers(-1, 2, (1, 4, 4)).astype(np.float64)
    R = rng.integers(-1, 2, (3, 8, 8)).astype(np.float64)
    assert np.array_equal(O.transform_fast_bf16(X, L, R), O.transform_fast(X, L, R))
    t = synth.make_transform(N, 23, "baseline")
    Xr = O.bf16_bits_to_f64(synth.make_activations(S, N, 23))
    exact = O.transform_fast(Xr, t.left, t.right)
    got = O.transform_fast_bf16(Xr, t.left, t.right)
    assert np.array_equal(O.round_to_bf16(got), got)                          # the output is a bf16 tensor
    Vb = np.abs(Xr).reshape(S, 3, 4, 8)
    bound = np.zeros_like(Vb)
    for j in range(3):
        U = Vb[:, j] @ np.abs(t.right[j].astype(np.float64))
        bound[:, j] = np.einsum("ra,src->sac", np.abs(t.left[0].astype(np.float64)), U)
    assert np.all(np.abs(got - exact) <= 2.0 ** -7 * bound.reshape(S, N) + 1e-300)
    assert np.any(got != exact)
