"""Host logic of the CTA-pair GEMM: its work distribution, checked without a GPU.

Tiles are numbered column of tiles after column and pair p of P takes tiles p, p + P, ...  The
columns come in a few segments, each all equally wide or alternately 256 and 192 wide.  The tiles
of all pairs together must cover the s x m output exactly once, every column must start at a
multiple of 64 features (the MMA cannot take weight scales from an odd 32-row group), only the
last column may be ragged, and no pair may have more than one tile more than another."""
import numpy as np
import pytest

from paper_2603_16590_b200 import binding as B

SHAPES = [(2048, 4096, 4096), (2048, 6144, 4096), (2048, 28672, 4096), (2048, 4096, 14336), (2048, 4096 + 8, 512),
          (300, 520, 3584), (129, 257, 2080), (260, 1000, 512), (8192, 3584, 3584), (8192, 18944, 3584),
          (8192, 4608, 3584), (257, 192, 256), (1000, 1100, 768), (4096, 64, 1024), (256, 100000, 256)]


def _check(sched, s, m):
    rows = -(-s // 256)
    cover = np.zeros((rows, -(-m // 64)), dtype=np.int32)
    cols = {}
    for p, tiles in enumerate(sched):
        for i, (mp, n0, bn) in enumerate(tiles):
            assert n0 % 64 == 0 and bn % 64 == 0 and 64 <= bn <= 256 and 0 <= mp < rows
            cols.setdefault(n0, set()).add(bn)
            cover[mp, n0 // 64:(n0 + bn) // 64] += 1
    assert np.all(cover == 1)
    starts = sorted(cols)
    assert all(len(v) == 1 for v in cols.values())
    widths = [next(iter(cols[c])) for c in starts]
    # column-major round robin: tile number = column index * rows + row block
    index = {c: k for k, c in enumerate(starts)}
    for p, tiles in enumerate(sched):
        for i, (mp, n0, bn) in enumerate(tiles):
            assert index[n0] * rows + mp == p + i * len(sched)
    body = widths[:-1]
    assert all(w in (64, 128, 192, 256) for w in body)
    # a handful of segments: the width pattern changes rarely
    changes = sum(1 for k in range(2, len(body)) if body[k] != body[k - 2])
    assert changes <= 8
    assert starts[-1] + widths[-1] >= m > starts[-1] + widths[-1] - 64
    counts = [len(t) for t in sched]
    assert max(counts) - min(counts) <= 1
    return widths


@pytest.mark.parametrize("s,m,n", SHAPES)
@pytest.mark.parametrize("sm_count", [148, 132, 2])
def test_tiles_cover_the_output_once(s, m, n, sm_count):
    sched = B.batq_debug_pair_schedule(s, m, n, sm_count)
    assert 1 <= len(sched) <= max(1, sm_count // 2)
    _check(sched, s, m)


@pytest.mark.parametrize("bn", [64, 128, 192, 256, 448])
def test_forced_widths(bn):
    for s, m, n in SHAPES[:8]:
        B.batq_debug_force_tile_width(bn)
        try:
            sched = B.batq_debug_pair_schedule(s, m, n)
        finally:
            B.batq_debug_force_tile_width(0)
        widths = _check(sched, s, m)
        if len(widths) > 2:
            assert set(widths[:-1]) == ({256, 192} if bn == 448 else {bn})


def test_bad_arguments():
    lib = B.load()
    assert lib.batq_debug_pair_schedule(0, 128, 128, 148, -1, None, 0) == -1
    assert lib.batq_debug_pair_schedule(128, 128, 128, 1, -1, None, 0) == -1
    assert lib.batq_debug_pair_schedule(256, 128, 128, 148, 999, None, 0) == 0


def test_forced_single_pattern():
    """Width 1 = the automatic choice among single-pattern schedules (all columns equally wide, or 256
    and 192 alternating)."""
    B.batq_debug_force_tile_width(1)
    try:
        for s, m, n in SHAPES[:8]:
            widths = _check(B.batq_debug_pair_schedule(s, m, n), s, m)
            body = widths[:-1]
            assert len(set(body)) <= 1 or all(w == (256 if k % 2 == 0 else 192) for k, w in enumerate(body))
    finally:
        B.batq_debug_force_tile_width(0)


def test_schedule_ends_the_pairs_together():
    """Llama-8B prefill shapes at 2048 tokens on 74 pairs: 6144 features are cut so that no pair has
    more than three tiles (four 192-wide ones otherwise) and none works on two 256-wide tiles in a
    row (they would share one accumulator slot)."""
    sched = B.batq_debug_pair_schedule(2048, 6144, 4096)
    assert max(len(t) for t in sched) == 3
    for tiles in sched:
        assert all(not (a[2] == 256 and b[2] == 256) for a, b in zip(tiles, tiles[1:]))
    assert sum(t[2] for tiles in sched for t in tiles) == 8 * 6144


# ---------------------------------------------------------------------------- wide tiles (one accumulator of up to 448 columns)
def _check_wide(sched, s, m):
    rows = -(-s // 256)
    cover = np.zeros((rows, -(-m // 64)), dtype=np.int32)
    cols = {}
    for p, tiles in enumerate(sched):
        for i, (mp, n0, bn) in enumerate(tiles):
            assert n0 % 64 == 0 and bn % 64 == 0 and 64 <= bn <= 448 and 0 <= mp < rows
            cols.setdefault(n0, set()).add(bn)
            cover[mp, n0 // 64:(n0 + bn) // 64] += 1
    assert np.all(cover == 1)
    starts = sorted(cols)
    assert all(len(v) == 1 for v in cols.values())
    widths = [next(iter(cols[c])) for c in starts]
    index = {c: k for k, c in enumerate(starts)}
    for p, tiles in enumerate(sched):
        for i, (mp, n0, bn) in enumerate(tiles):
            assert index[n0] * rows + mp == p + i * len(sched)
    # at most two widths before the ragged last column
    assert len(set(widths[:-1])) <= 2
    assert starts[-1] + widths[-1] >= m > starts[-1] + widths[-1] - 64
    counts = [len(t) for t in sched]
    assert max(counts) - min(counts) <= 1
    return widths


@pytest.mark.parametrize("s,m,n", SHAPES)
@pytest.mark.parametrize("sm_count", [148, 132, 2])
def test_wide_tiles_cover_the_output_once(s, m, n, sm_count):
    sched = B.batq_debug_wide_schedule(s, m, n, sm_count)
    assert 1 <= len(sched) <= max(1, sm_count // 2)
    _check_wide(sched, s, m)


@pytest.mark.parametrize("bn", [64, 128, 192, 256, 320, 384, 448])
def test_wide_forced_widths(bn):
    for s, m, n in SHAPES[:8]:
        B.batq_debug_force_tile_width(bn)
        try:
            sched = B.batq_debug_wide_schedule(s, m, n)
        finally:
            B.batq_debug_force_tile_width(0)
        widths = _check_wide(sched, s, m)
        assert all(w == bn for w in widths[:-1])


def test_wide_schedule_of_the_gate_up_projection():
    """28672 features at 2048 tokens on 74 pairs: 64 columns of 448 give every pair 6 or 7 tiles."""
    sched = B.batq_debug_wide_schedule(2048, 28672, 4096)
    cols = [sum(t[2] for t in tiles) for tiles in sched]
    assert max(cols) <= 3200 and len(sched) == 74
