"""Host-side audit of the address arithmetic of the bulk-copy mix kernel's form for parameter counts that are not multiples
of 4 (no GPU): every row piece is fetched from the 16-byte boundary below its first element in whole 16-byte units.  The
formulas of the producer (copy start, length, the plain-load tail at the end of a buffer), of the host planner (staged row
stride, the per-slice shift folded into the table offsets) and of the consumer (shared-memory index of a tile's element)
are restated here and checked against one another and against the buffer bounds over a sweep of shapes."""
import itertools

import numpy as np


def plan(P, rows, budget_bytes):
    """Tile width as the planner picks it for P % 4 != 0: staged row = w + 4 floats, w a multiple of 4 (128 / 32 / 4)."""
    w = budget_bytes // (rows * 4) - 4
    if w >= 128:
        w = min(1024, w // 128 * 128)
    elif w >= 32:
        w = w // 32 * 32
    else:
        w = w // 4 * 4
    assert w >= 4
    return min(w, (P + 3) // 4 * 4)


def piece(base_floats, row, P, c0, wd, n_rows):
    """Producer: (first float fetched, floats by bulk copy, floats by plain loads, shift of element 0 in the staged row),
    all relative to a buffer of n_rows * P floats whose base is 16-byte aligned (base_floats % 4 == 0)."""
    src = base_floats + row * P + c0
    a = src & 3
    src0 = src - a
    n = (a + wd + 3) & ~3
    end = base_floats + n_rows * P
    tail = 0
    if src0 + n > end:
        n -= 4
        tail = end - (src0 + n)
    return src0, n, tail, a


def test_every_fetch_stays_inside_its_buffer_and_its_staged_row():
    checked = 0
    for P, n_rows, rows_staged in itertools.product([1, 2, 3, 5, 7, 33, 130, 257, 1023, 4097, 4999, 10001, 10002, 10003],
                                                    [1, 2, 3, 6, 20], [1, 3, 40, 226]):
        if P % 4 == 0:
            continue
        w = plan(P, rows_staged, 110 * 1024)
        ws = w + 4
        tiles = (P + w - 1) // w
        for base in (0, 4, 64):
            for row in range(n_rows):
                shift_host = (row * P) & 3                           # what the planner folds into the table offsets
                for tile in sorted({0, 1, tiles // 2, tiles - 1} & set(range(tiles))):
                    c0 = tile * w
                    wd = min(w, P - c0)
                    src0, n, tail, a = piece(base, row, P, c0, wd, n_rows)
                    assert src0 % 4 == 0 and n % 4 == 0                              # 16-byte aligned source, 16-byte units
                    assert src0 >= base                                              # never below the buffer
                    assert src0 + n + tail <= base + n_rows * P                      # never past its end
                    assert 0 <= tail < 4 and (tail == 0 or (row == n_rows - 1 or src0 + n + tail == base + n_rows * P))
                    assert n + tail >= a + wd                                        # the whole piece is covered ...
                    assert a + wd <= ws and n + tail <= ws                           # ... and fits the staged row
                    assert a == shift_host                                           # same shift for every tile (w % 4 == 0)
                    # consumer: element c of the tile sits at staged index shift + c
                    for c in (0, wd - 1):
                        assert src0 + (shift_host + c) == base + row * P + c0 + c
                    checked += 1
    assert checked > 5000


def test_transaction_bytes_of_a_warp_add_up():
    """The producer warp posts the sum of its lanes' byte counts once per tile; plain-load tails carry no bytes."""
    rng = np.random.default_rng(0)
    for _ in range(200):
        P = int(rng.integers(1, 5000)) | 1
        n_rows = int(rng.integers(1, 9))
        w = plan(P, 8, 64 * 1024)
        tile = int(rng.integers(0, (P + w - 1) // w))
        c0, wd = tile * w, min(w, P - tile * w)
        total = sum(piece(0, r, P, c0, wd, n_rows)[1] * 4 for r in range(n_rows))
        covered = sum((lambda s0, n, t, a: n + t - a)(*piece(0, r, P, c0, wd, n_rows)) for r in range(n_rows))
        assert total % 16 == 0 and covered >= n_rows * wd
