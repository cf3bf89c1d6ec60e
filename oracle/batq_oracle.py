"""CPU oracle for the BATQuant W4A4 linear hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 / exact-integer numpy statement of what the path computes,
written from the paper's definitions.  It shares no code with the CUDA path
and must never be imported by the product package: only the tests, the smoke
check and the benchmark's ``cpu_baseline`` / ``--impl reference`` legs use it.

Notation (paper Sec. 3.1 and Algorithm 1).  A row vector of N = k*32 channels
is cut into k blocks of g = 32.  A block x is viewed as a matrix V[r][c] with
element index e = r*gc + c, r < gr, c < gc, gr*gc = 32 (the reshape
[-1, k, g2, g1] of Algorithm 1: the last, contiguous index has the size of the
factor multiplied from the right).  The block matrix is the Kronecker product
P_j = L_j (x) R_j (Eq. 2, written B_i (x) A there), a dense 32x32 matrix with
P[(r,c),(r',c')] = L[r][r'] * R[c][c'], and the transform of a row vector is
x~ = x P_j (Eq. 1, "XP" of the arg-min objective).

Parity status of each function is given in its docstring; everything here is
pinned by tests/test_oracle_*.py except where it says "parity unpinned".
Unpinned: nothing numeric.  (The behaviour of *learned* parameters and the
paper's accuracy tables cannot be pinned -- they need weights and datasets --
but no function in this file depends on them.)
"""
from __future__ import annotations

import numpy as np

GROUP = 32  # MX block size g (Sec. 2: the MX formats share one scale per 32 elements)

# The E2M1 magnitudes by code 0..7 (Sec. 2: 7 positive values + zero); bit 3
# of a code is the sign.
E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)
E2M1_EMAX = 2  # 6 = 1.5 * 2**2: exponent of the largest E2M1 magnitude


# ----------------------------------------------------------------------------
# Input decoding
# ----------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the exact real values, as fp64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------
# Block transform: Eq. 1 / Eq. 2 / Algorithm 1
# ----------------------------------------------------------------------------
def kron_dense(L: np.ndarray, R: np.ndarray) -> np.ndarray:
    """Dense P = L (x) R from the definition P[(r,c),(r',c')] = L[r,r'] R[c,c']
    (Eq. 2 with the index order of Algorithm 1).  L is gr x gr, R is gc x gc."""
    L = np.asarray(L, dtype=np.float64)
    R = np.asarray(R, dtype=np.float64)
    gr, gc = L.shape[0], R.shape[0]
    P = np.zeros((gr * gc, gr * gc), dtype=np.float64)
    for r in range(gr):
        for c in range(gc):
            for r2 in range(gr):
                for c2 in range(gc):
                    P[r * gc + c, r2 * gc + c2] = L[r, r2] * R[c, c2]
    return P


def _factor_for_block(F: np.ndarray, j: int) -> np.ndarray:
    """F is [1, n, n] (shared across blocks, the 'global' factor) or
    [k, n, n] (one per block, the 'private' factors)."""
    return F[0] if F.shape[0] == 1 else F[j]


def block_matrices(L: np.ndarray, R: np.ndarray, k: int) -> np.ndarray:
    """The k dense 32x32 blocks P_1..P_k of the block-diagonal P (Eq. 1)."""
    L = np.asarray(L, dtype=np.float64)
    R = np.asarray(R, dtype=np.float64)
    return np.stack([kron_dense(_factor_for_block(L, j), _factor_for_block(R, j))
                     for j in range(k)])


def transform_dense(X: np.ndarray, P: np.ndarray) -> np.ndarray:
    """x~ = x P_j on every block j of every row (Eq. 1).  X is [S, N] fp64,
    P is [k, 32, 32]."""
    S, N = X.shape
    k = N // GROUP
    Xb = X.reshape(S, k, GROUP)
    out = np.empty_like(Xb)
    for j in range(k):
        out[:, j, :] = Xb[:, j, :] @ P[j]
    return out.reshape(S, N)


def transform_fast(X: np.ndarray, L: np.ndarray, R: np.ndarray) -> np.ndarray:
    """The factored form of the same transform: V~ = L_j^T V R_j per block
    (the vec identity stated after Eq. 2; the two contractions of Algorithm 1).
    A second, independent routine; tests check it against transform_dense."""
    L = np.asarray(L, dtype=np.float64)
    R = np.asarray(R, dtype=np.float64)
    S, N = X.shape
    k = N // GROUP
    gr, gc = L.shape[1], R.shape[1]
    V = X.reshape(S, k, gr, gc)
    out = np.empty_like(V)
    for j in range(k):
        Lj = _factor_for_block(L, j)
        Rj = _factor_for_block(R, j)
        U = V[:, j] @ Rj                          # right factor on the contiguous index
        out[:, j] = np.einsum("ra,src->sac", Lj, U)  # L^T from the left
    return out.reshape(S, N)


def round_to_bf16(v: np.ndarray) -> np.ndarray:
    """Round real values (fp64) to the nearest bf16 value (8 significant bits, ties to even), as
    fp64.  Written from the format: v = m * 2**e with m in [0.5, 1); keep 8 bits of m."""
    v = np.asarray(v, dtype=np.float64)
    m, e = np.frexp(v)
    return np.ldexp(np.rint(m * 256.0) / 256.0, e)     # np.rint rounds halves to even


def transform_fast_bf16(X: np.ndarray, L: np.ndarray, R: np.ndarray) -> np.ndarray:
    """The two contractions of Algorithm 1 as the paper runs them (Sec. 3.2 keeps the
    pre-quantization transforms in BF16): the result of each contraction is a bf16 tensor, i.e.
    V R is rounded to bf16 before L^T is applied, and the output is rounded to bf16 again.  Each
    contraction itself is exact here (a BF16 matmul accumulates wider than it stores)."""
    L = np.asarray(L, dtype=np.float64)
    R = np.asarray(R, dtype=np.float64)
    S, N = X.shape
    k = N // GROUP
    gr, gc = L.shape[1], R.shape[1]
    V = X.reshape(S, k, gr, gc)
    out = np.empty_like(V)
    for j in range(k):
        U = round_to_bf16(V[:, j] @ _factor_for_block(R, j))
        out[:, j] = round_to_bf16(np.einsum("ra,src->sac", _factor_for_block(L, j), U))
    return out.reshape(S, N)


# ----------------------------------------------------------------------------
# Block-wise clipping: Eq. 3 / Eq. 4
# ----------------------------------------------------------------------------
def block_clip(V: np.ndarray, c_lo: np.ndarray, c_hi: np.ndarray) -> np.ndarray:
    """Per (row, block): lo = c_lo*min(v), hi = c_hi*max(v), v^ = min(max(v,lo),hi).
    c_lo / c_hi are the post-sigmoid ratios of Eq. 4, shape [k] (one pair per
    channel block, shared by all rows) or [S, k] (one pair per row and block,
    used for weights)."""
    S, N = V.shape
    k = N // GROUP
    Vb = V.reshape(S, k, GROUP)
    lo = np.asarray(c_lo, dtype=np.float64).reshape(-1, k)[:, :, None] * Vb.min(axis=2, keepdims=True)
    hi = np.asarray(c_hi, dtype=np.float64).reshape(-1, k)[:, :, None] * Vb.max(axis=2, keepdims=True)
    return np.minimum(np.maximum(Vb, lo), hi).reshape(S, N)


# ----------------------------------------------------------------------------
# MXFP4 quantizer Q(.): shared UE8M0 scale + E2M1 elements (Sec. 2)
# ----------------------------------------------------------------------------
def mx_scale_exponent(amax: np.ndarray) -> np.ndarray:
    """OCP MX shared-scale rule: e = floor(log2(amax)) - emax_elem, clamped to
    the UE8M0 range [-127, 127]; amax == 0 gives -127.  floor(log2) is taken
    exactly from the binary exponent (frexp), never from a floating log."""
    amax = np.asarray(amax, dtype=np.float64)
    mant, ex = np.frexp(amax)            # amax = mant * 2**ex, mant in [0.5, 1)
    floor_log2 = ex.astype(np.int64) - 1
    e = floor_log2 - E2M1_EMAX
    e = np.where(amax == 0.0, -127, e)
    return np.clip(e, -127, 127).astype(np.int64)


def e2m1_round_code(u: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even of u onto the E2M1 grid, saturating at +-6.
    Returns 4-bit codes (bit 3 = sign of u, so -0 keeps its sign).  Written as
    the definition: nearest representable magnitude; on a tie the candidate
    with the even code (even mantissa bit) wins."""
    u = np.asarray(u, dtype=np.float64)
    mag = np.abs(u)
    dist = np.abs(mag[..., None] - E2M1_VALUES)          # [..., 8]
    best = dist.min(axis=-1, keepdims=True)
    is_best = dist == best
    even = (np.arange(8) % 2) == 0
    # prefer an even code among the tied candidates, else the (unique) nearest
    pick_even = is_best & even
    code_even = np.argmax(pick_even, axis=-1)
    code_any = np.argmax(is_best, axis=-1)
    code = np.where(pick_even.any(axis=-1), code_even, code_any).astype(np.uint8)
    sign = np.signbit(u).astype(np.uint8)
    return (code | (sign << 3)).astype(np.uint8)


def e2m1_decode(code: np.ndarray) -> np.ndarray:
    """4-bit code -> real value (fp64)."""
    code = np.asarray(code, dtype=np.uint8)
    mag = E2M1_VALUES[code & 7]
    return np.where((code & 8) != 0, -mag, mag)


def mxfp4_quantize(V: np.ndarray):
    """Q(V) for V [S, N] fp64: per 32-block scale byte (e + 127) and one 4-bit
    code per element.  Returns (codes uint8 [S, N], scale_bytes uint8 [S, k])."""
    S, N = V.shape
    k = N // GROUP
    Vb = V.reshape(S, k, GROUP)
    amax = np.abs(Vb).max(axis=2)
    e = mx_scale_exponent(amax)
    u = Vb / np.exp2(e.astype(np.float64))[:, :, None]   # exact: power-of-two divisor
    codes = e2m1_round_code(u).reshape(S, N)
    return codes, (e + 127).astype(np.uint8)


# ----------------------------------------------------------------------------
# MXFP8 quantizer (E4M3 elements, the MXFP8 element type Sec. 2 settles on), used for
# 8-bit activations (W4A8) and the 8-bit KV cache
# ----------------------------------------------------------------------------
E4M3_EMAX = 8  # 448 = 1.75 * 2**8: exponent of the largest E4M3 magnitude


def e4m3_decode(code: np.ndarray) -> np.ndarray:
    """8-bit code -> real value: 1 sign, 4 exponent (bias 7), 3 mantissa bits;
    E = 0 holds the subnormals M/8 * 2**-6; E = 15, M = 7 is NaN (no infinities)."""
    code = np.asarray(code, dtype=np.uint8).astype(np.int64)
    sgn, E, M = code >> 7, (code >> 3) & 15, code & 7
    mag = np.where(E == 0, M / 8.0 * 2.0 ** -6, (1.0 + M / 8.0) * np.exp2((E - 7).astype(np.float64)))
    mag = np.where((E == 15) & (M == 7), np.nan, mag)
    return np.where(sgn == 1, -mag, mag)


def e4m3_round_code(u: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even of u onto the E4M3 grid, saturating at +-448.  Written as the
    definition: the nearest of the 127 finite magnitudes; on a tie the one with the even code."""
    u = np.asarray(u, dtype=np.float64)
    grid = e4m3_decode(np.arange(127, dtype=np.uint8))   # magnitudes of codes 0..126, increasing
    mag = np.minimum(np.abs(u), grid[-1])
    hi = np.clip(np.searchsorted(grid, mag, side="left"), 0, 126)   # first grid point >= mag
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = grid[hi] - mag, mag - grid[lo]
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return (code | (np.signbit(u).astype(np.uint8) << 7)).astype(np.uint8)


def mxfp8_quantize(V: np.ndarray):
    """Q(V) with E4M3 elements: per 32-block scale byte (e + 127, e = floor(log2 amax) - 8) and
    one 8-bit code per element.  Returns (codes uint8 [S, N], scale_bytes uint8 [S, k])."""
    S, N = V.shape
    k = N // GROUP
    Vb = V.reshape(S, k, GROUP)
    amax = np.abs(Vb).max(axis=2)
    mant, ex = np.frexp(amax)
    e = np.where(amax == 0.0, -127, ex.astype(np.int64) - 1 - E4M3_EMAX)
    e = np.clip(e, -127, 127).astype(np.int64)
    u = Vb / np.exp2(e.astype(np.float64))[:, :, None]
    return e4m3_round_code(u).reshape(S, N), (e + 127).astype(np.uint8)


def quantize_act_mxfp8(x_bits, L, R, c_lo=None, c_hi=None):
    """Stages 1+2 with 8-bit elements (transform -> clip -> MXFP8)."""
    return mxfp8_quantize(transform_clip(x_bits, L, R, c_lo, c_hi))


def dequantize_mxfp8(codes: np.ndarray, scale_bytes: np.ndarray) -> np.ndarray:
    S, N = codes.shape
    k = N // GROUP
    scale = np.exp2(scale_bytes.astype(np.float64) - 127.0)
    return (e4m3_decode(codes).reshape(S, k, GROUP) * scale[:, :, None]).reshape(S, N)


def gemm_mxfp8_mxfp4(codes_x8, scales_x, codes_w, scales_w):
    """Stage 3 of the W4A8 configuration (MXFP8-E4M3 activations x MXFP4 weights, the W4A8
    settings of Sec. 4): Y[s,m] = sum_e deq8_x[s,e] * deq4_w[m,e] in fp64 and
    Sabs[s,m] = sum_e |deq8_x * deq4_w|.  Returns (Y, Sabs)."""
    dx = dequantize_mxfp8(codes_x8, scales_x)
    dw = dequantize(codes_w, scales_w)
    return dx @ dw.T, np.abs(dx) @ np.abs(dw).T


def gemm_mxfp8_mxfp4_exact(codes_x8, scales_x, codes_w, scales_w):
    """The same contraction in exact rational arithmetic, for tiny shapes: every finite E4M3 value
    is an integer multiple of 2**-9 and every E2M1 value of 2**-1, so a block contributes
    2**(ex + ew - 10) times an integer dot product.  Returns fp64 after the exact evaluation."""
    from fractions import Fraction
    S, N = codes_x8.shape
    M = codes_w.shape[0]
    k = N // GROUP
    ix = np.rint(512 * e4m3_decode(codes_x8)).astype(np.int64)
    iw = np.rint(2 * e2m1_decode(codes_w)).astype(np.int64)
    Y = np.zeros((S, M), dtype=np.float64)
    for s in range(S):
        for m in range(M):
            acc = Fraction(0)
            for j in range(k):
                blk = int(np.dot(ix[s, j * GROUP:(j + 1) * GROUP], iw[m, j * GROUP:(j + 1) * GROUP]))
                ex = int(scales_x[s, j]) - 127 + int(scales_w[m, j]) - 127
                acc += Fraction(blk, 1024) * (Fraction(2) ** ex)
            Y[s, m] = float(acc)
    return Y


def linear_w4a8(x_bits, w_bits, L, R, c_lo=None, c_hi=None):
    """The W4A8 layer: Q8(XP) Q4(P^{-1} W^T), activations in MXFP8 (E4M3), weights in MXFP4.
    Returns (Y, Sabs, (codes_x8, scales_x), (codes_w, scales_w))."""
    qx = quantize_act_mxfp8(x_bits, L, R, c_lo, c_hi)
    qw = prepare_weight(w_bits, L, R)
    Y, Sabs = gemm_mxfp8_mxfp4(qx[0], qx[1], qw[0], qw[1])
    return Y, Sabs, qx, qw


def pack_codes(codes: np.ndarray) -> np.ndarray:
    """Two codes per byte: element 2i in bits 0-3, element 2i+1 in bits 4-7."""
    c = np.asarray(codes, dtype=np.uint8)
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    p = np.asarray(packed, dtype=np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = p & 0xF
    out[..., 1::2] = p >> 4
    return out


def dequantize(codes: np.ndarray, scale_bytes: np.ndarray) -> np.ndarray:
    """codes [S, N] (unpacked) and scale bytes [S, k] -> real values fp64."""
    S, N = codes.shape
    k = N // GROUP
    scale = np.exp2(scale_bytes.astype(np.float64) - 127.0)
    return (e2m1_decode(codes).reshape(S, k, GROUP) * scale[:, :, None]).reshape(S, N)


# ----------------------------------------------------------------------------
# The three stages
# ----------------------------------------------------------------------------
def transform_clip(x_bits, L, R, c_lo=None, c_hi=None, round_intermediate_bf16=False) -> np.ndarray:
    """Stage 1 in fp64: x~ = x P (dense form), then the block clip.  L / R may
    be None for the identity transform (plain MXFP4 of X).  round_intermediate_bf16: the
    transform as the paper's BF16 implementation computes it (transform_fast_bf16)."""
    X = bf16_bits_to_f64(x_bits)
    k = X.shape[1] // GROUP
    if L is not None and round_intermediate_bf16:
        X = transform_fast_bf16(X, L, R)
    elif L is not None:
        X = transform_dense(X, block_matrices(L, R, k))
    if c_lo is not None:
        X = block_clip(X, c_lo, c_hi)
    return X


def quantize_act(x_bits, L, R, c_lo=None, c_hi=None, round_intermediate_bf16=False):
    """Stages 1+2 (transform -> clip -> Q, the order of the paper's algorithm
    flow).  Returns (codes [S, N] unpacked, scale_bytes [S, k])."""
    return mxfp4_quantize(transform_clip(x_bits, L, R, c_lo, c_hi, round_intermediate_bf16))


def invert_blocks(P: np.ndarray) -> np.ndarray:
    """P_j^{-1} by Gauss-Jordan elimination with partial pivoting on the dense
    32x32 block, in fp64."""
    out = np.empty_like(P)
    for j in range(P.shape[0]):
        n = P.shape[1]
        aug = np.concatenate([P[j].copy(), np.eye(n)], axis=1)
        for col in range(n):
            piv = col + int(np.argmax(np.abs(aug[col:, col])))
            if aug[piv, col] == 0.0:
                raise ValueError("singular block matrix")
            if piv != col:
                aug[[col, piv]] = aug[[piv, col]]
            aug[col] /= aug[col, col]
            for row in range(n):
                if row != col and aug[row, col] != 0.0:
                    aug[row] -= aug[row, col] * aug[col]
        out[j] = aug[:, n:]
    return out


def transform_weight(w_bits, L, R) -> np.ndarray:
    """W~ = W P^{-T}: each 32-block of each weight row times P_j^{-T}, the only
    reading of "P^{-1} W^T" for which X~ W~^T = X W^T.  fp64."""
    W = bf16_bits_to_f64(w_bits)
    if L is None:
        return W
    k = W.shape[1] // GROUP
    Pinv = invert_blocks(block_matrices(L, R, k))
    return transform_dense(W, np.transpose(Pinv, (0, 2, 1)))


def prepare_weight(w_bits, L, R, w_c_lo=None, w_c_hi=None):
    """Offline weight fusion: transform with the inverse, optional block clip,
    Q.  Returns (codes [M, N] unpacked, scale_bytes [M, k])."""
    Wt = transform_weight(w_bits, L, R)
    if w_c_lo is not None:
        Wt = block_clip(Wt, w_c_lo, w_c_hi)
    return mxfp4_quantize(Wt)


def gemm_mxfp4(codes_x, scales_x, codes_w, scales_w):
    """Stage 3: Y[s,m] = sum_e deq_x[s,e] * deq_w[m,e] in fp64 over the
    dequantized values, and Sabs[s,m] = sum_e |deq_x * deq_w| (the tolerance
    normaliser).  Returns (Y, Sabs)."""
    dx = dequantize(codes_x, scales_x)
    dw = dequantize(codes_w, scales_w)
    return dx @ dw.T, np.abs(dx) @ np.abs(dw).T


def gemm_mxfp4_exact_int(codes_x, scales_x, codes_w, scales_w):
    """The same contraction in exact integer arithmetic (Python ints), for tiny
    shapes: E2M1 values are half-integers, so 2*value is a small integer; each
    block contributes 2^(ex+ew) * (sum of integer products) / 4.  Returned as
    fp64 after an exact rational evaluation."""
    from fractions import Fraction
    S, N = codes_x.shape
    M = codes_w.shape[0]
    k = N // GROUP
    ix = np.rint(2 * e2m1_decode(codes_x)).astype(np.int64)
    iw = np.rint(2 * e2m1_decode(codes_w)).astype(np.int64)
    Y = np.zeros((S, M), dtype=np.float64)
    for s in range(S):
        for m in range(M):
            acc = Fraction(0)
            for j in range(k):
                blk = int(np.dot(ix[s, j * GROUP:(j + 1) * GROUP], iw[m, j * GROUP:(j + 1) * GROUP]))
                ex = int(scales_x[s, j]) - 127 + int(scales_w[m, j]) - 127
                acc += Fraction(blk, 4) * (Fraction(2) ** ex)
            Y[s, m] = float(acc)
    return Y


def linear_w4a4(x_bits, w_bits, L, R, c_lo=None, c_hi=None):
    """The whole quantized linear layer Y ~ Q(XP) Q(P^{-1} W^T).  Returns
    (Y, Sabs, (codes_x, scales_x), (codes_w, scales_w))."""
    qx = quantize_act(x_bits, L, R, c_lo, c_hi)
    qw = prepare_weight(w_bits, L, R)
    Y, Sabs = gemm_mxfp4(qx[0], qx[1], qw[0], qw[1])
    return Y, Sabs, qx, qw
