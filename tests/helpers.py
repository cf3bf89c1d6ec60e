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
