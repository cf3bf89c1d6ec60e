"""Test-side helpers (no method arithmetic shared with the CUDA path or the oracle)."""
import numpy as np

E2M1_TIE_POINTS = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])


def sf_mma_to_rowmajor(buf: np.ndarray, rows: int, k: int) -> np.ndarray:
    """Undo the BATQ_SF_MMA layout as documented in include/batq.h:
    byte (row, j) at ((row/128)*KA + j/4)*512 + (row%32)*16 + ((row%128)/32)*4 + j%4,
    KA = 2*ceil(k/8)."""
    ka = 2 * ((k + 7) // 8)
    r = np.arange(rows)[:, None]
    j = np.arange(k)[None, :]
    off = ((r // 128) * ka + j // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + j % 4
    return np.asarray(buf).reshape(-1)[off]


def near_rounding_boundary(u_abs: np.ndarray, rel: float) -> np.ndarray:
    """True where |u| lies within a relative distance `rel` of an E2M1 tie point."""
    d = np.abs(u_abs[..., None] - E2M1_TIE_POINTS) / E2M1_TIE_POINTS
    return (d <= rel).any(axis=-1)


def fp32_transform_bound(x_abs_blocks: np.ndarray, p_abs: np.ndarray, rel: float) -> np.ndarray:
    """rel * sum_e |x_e| |P_ef| per output f: the a-priori bound on the fp32 transform error.
    x_abs_blocks [S, k, 32], p_abs [k, 32, 32]; returns [S, k*32]."""
    S, k, _ = x_abs_blocks.shape
    return rel * np.einsum("sje,jef->sjf", x_abs_blocks, p_abs).reshape(S, k * 32)


def code_mismatch_report(gc, gs, oc, os_, V, bound):
    """Compares GPU codes / scale bytes (gc [S, N], gs [S, k]) with the oracle's (oc, os_) computed
    from the fp64 transform output V, given the a-priori bound on |v^ - V| per element.

    Returns a dict of counts:
      scale_mismatch        blocks whose scale byte differs
      scale_unexplained     ... of which amax does NOT lie within the bound of a power of two
      code_mismatch         elements (in blocks with equal scale bytes) whose code differs
      strict                ... of which |u| lies within 1 fp32 ulp (2^-22 relative) of a rounding boundary
      bound_only            ... of which only the a-priori bound explains the difference
      unexplained           ... explained by neither
      not_neighbour         mismatching codes that are not the neighbouring code
    """
    S, N = gc.shape
    k = N // 32
    sdiff = gs != os_
    rep = {"elements": int(S) * int(N), "blocks": int(S) * k, "scale_mismatch": int(sdiff.sum()), "scale_unexplained": 0}
    if sdiff.any():
        amax = np.abs(V).reshape(S, k, 32).max(axis=2)
        bmax = bound.reshape(S, k, 32).max(axis=2)
        a, b = amax[sdiff], bmax[sdiff]
        p2 = np.exp2(np.round(np.log2(np.maximum(a, 1e-300))))
        rep["scale_unexplained"] = int((np.abs(a - p2) > b).sum())
    cdiff = (gc != oc) & np.repeat(~sdiff, 32, axis=1)
    rep["code_mismatch"] = int(cdiff.sum())
    rep["strict"] = rep["bound_only"] = rep["unexplained"] = rep["not_neighbour"] = 0
    if cdiff.any():
        scale = np.repeat(np.exp2(os_.astype(np.float64) - 127), 32, axis=1)
        u = (np.abs(V) / scale)[cdiff]
        du = (bound / scale)[cdiff]                       # the bound in units of the grid
        strict = near_rounding_boundary(u, 2.0 ** -22)
        dist = np.abs(u[:, None] - E2M1_TIE_POINTS).min(axis=1)
        by_bound = dist <= du
        rep["strict"] = int(strict.sum())
        rep["bound_only"] = int((by_bound & ~strict).sum())
        rep["unexplained"] = int((~by_bound & ~strict).sum())
        rep["not_neighbour"] = int((np.abs((gc[cdiff] & 7).astype(int) - (oc[cdiff] & 7).astype(int)) > 1).sum())
    return rep
