"""CPU pins of the oracle's rejection islands (Sec. 3.4, Eq. 8: 8-connected components of R_X)."""
import itertools

import numpy as np
import pytest
from scipy import ndimage

import oracle


def canonical(labels):
    """Renumbers a labelling by the raster index of each label's first cell."""
    out = np.zeros_like(labels)
    nxt = 0
    seen = {}
    for v, t in zip(labels.ravel(), range(labels.size)):
        if v == 0:
            continue
        if v not in seen:
            nxt += 1
            seen[v] = nxt
        out.flat[t] = seen[v]
    return out, nxt


def closure_partition(mask):
    """Islands by the definition alone: transitive closure of the 8-adjacency matrix."""
    H, W = mask.shape
    cells = [(i, j) for i in range(H) for j in range(W) if mask[i, j]]
    n = len(cells)
    A = np.eye(n, dtype=bool)
    for a, b in itertools.combinations(range(n), 2):
        if abs(cells[a][0] - cells[b][0]) <= 1 and abs(cells[a][1] - cells[b][1]) <= 1:
            A[a, b] = A[b, a] = True
    for _ in range(max(1, int(np.ceil(np.log2(max(n, 2)))))):
        A = (A.astype(np.int32) @ A.astype(np.int32)) > 0
    labels = np.zeros((H, W), np.int32)
    nxt = 0
    for a in range(n):
        if labels[cells[a]] == 0:
            nxt += 1
            for b in range(n):
                if A[a, b]:
                    labels[cells[b]] = nxt
    return labels, nxt


def check_stats(labels, M, rows, size):
    assert rows.shape == (M, 2) and size.shape == (M,)
    for m in range(1, M + 1):
        ii, _ = np.nonzero(labels == m)
        assert size[m - 1] == ii.size > 0
        assert rows[m - 1, 0] == ii.min() and rows[m - 1, 1] == ii.max()


@pytest.mark.parametrize("shape", [(1, 1), (1, 7), (5, 1), (3, 4), (8, 8), (17, 33), (64, 64), (40, 70)])
@pytest.mark.parametrize("density", [0.02, 0.2, 0.45, 0.7])
def test_against_scipy_label(shape, density):
    rng = np.random.default_rng(hash((shape, density)) % (1 << 32))
    mask = (rng.random(shape) < density).astype(np.uint8)
    labels, M, rows, size = oracle.islands(mask)
    ref, n_ref = ndimage.label(mask, structure=np.ones((3, 3), np.int32))
    ref_c, n_c = canonical(ref.astype(np.int32))
    assert M == n_ref == n_c
    np.testing.assert_array_equal(labels, ref_c)
    np.testing.assert_array_equal((labels > 0), mask.astype(bool))
    check_stats(labels, M, rows, size)


def test_every_mask_of_a_3x4_grid_against_the_closure():
    for bits in range(1 << 12):
        mask = np.array([(bits >> t) & 1 for t in range(12)], np.uint8).reshape(3, 4)
        labels, M, rows, size = oracle.islands(mask)
        ref, n_ref = closure_partition(mask)
        assert M == n_ref, bits
        np.testing.assert_array_equal(labels, ref)


def test_numbering_follows_the_first_raster_position():
    mask = np.zeros((6, 9), np.uint8)
    mask[0, 7] = 1                 # island 1: first in raster order although far right
    mask[1, 0:3] = 1               # island 2
    mask[3, 4] = mask[4, 5] = 1    # island 3 (diagonal step)
    mask[5, 0] = 1                 # island 4
    labels, M, rows, size = oracle.islands(mask)
    assert M == 4
    assert labels[0, 7] == 1 and labels[1, 1] == 2 and labels[3, 4] == 3 and labels[4, 5] == 3
    assert labels[5, 0] == 4
    np.testing.assert_array_equal(rows, [[0, 0], [1, 1], [3, 4], [5, 5]])
    np.testing.assert_array_equal(size, [1, 3, 2, 1])


def test_diagonals_join_and_gaps_separate():
    n = 9
    anti = np.fliplr(np.eye(n, dtype=np.uint8))
    labels, M, _, size = oracle.islands(anti)
    assert M == 1 and size[0] == n            # 4-connectivity would give n islands
    labels, M, _, _ = oracle.islands(np.eye(n, dtype=np.uint8))
    assert M == 1
    checker = (np.add.outer(np.arange(8), np.arange(8)) % 2 == 0).astype(np.uint8)
    assert oracle.islands(checker)[1] == 1
    dots = np.zeros((8, 10), np.uint8)
    dots[::2, ::2] = 1                         # no two dots touch, not even at a corner
    labels, M, rows, size = oracle.islands(dots)
    assert M == 4 * 5 and (size == 1).all()
    np.testing.assert_array_equal(labels[::2, ::2].ravel(), np.arange(1, 21))
    two = np.zeros((3, 5), np.uint8)
    two[:, 0] = two[:, 2] = 1                  # neighbouring columns 0 and 2: a one-cell gap
    assert oracle.islands(two)[1] == 2
    two[1, 1] = 1
    assert oracle.islands(two)[1] == 1


def test_empty_full_and_late_merges():
    assert oracle.islands(np.zeros((5, 6), np.uint8))[1] == 0
    labels, M, rows, size = oracle.islands(np.ones((5, 6), np.uint8))
    assert M == 1 and size[0] == 30 and tuple(rows[0]) == (0, 4)
    u = np.zeros((6, 7), np.uint8)             # a "U": two arms that meet only in the last row
    u[:, 0] = u[:, 6] = 1
    u[5, :] = 1
    labels, M, _, _ = oracle.islands(u)
    assert M == 1 and labels[0, 6] == 1
    spiral = np.array([[1, 1, 1, 1, 1, 1, 1],
                       [0, 0, 0, 0, 0, 0, 1],
                       [1, 1, 1, 1, 1, 0, 1],
                       [1, 0, 0, 0, 1, 0, 1],
                       [1, 0, 1, 0, 0, 0, 1],
                       [1, 0, 0, 0, 0, 0, 1],
                       [1, 1, 1, 1, 1, 1, 1]], np.uint8)
    labels, M, _, _ = oracle.islands(spiral)
    assert M == 2 and labels[4, 2] == 2 and (labels[spiral == 1] > 0).all()
    ring = np.zeros((7, 7), np.uint8)
    ring[1, 1:6] = ring[5, 1:6] = ring[1:6, 1] = ring[1:6, 5] = 1
    ring[3, 3] = 1                              # a dot inside the ring, two cells from it
    assert oracle.islands(ring)[1] == 2


def test_islands_never_touch_and_are_connected():
    rng = np.random.default_rng(7)
    mask = (rng.random((24, 31)) < 0.35).astype(np.uint8)
    labels, M, _, _ = oracle.islands(mask)
    H, W = mask.shape
    for i in range(H):
        for j in range(W):
            if not mask[i, j]:
                assert labels[i, j] == 0
                continue
            for di in (-1, 0, 1):
                for dj in (-1, 0, 1):
                    a, b = i + di, j + dj
                    if 0 <= a < H and 0 <= b < W and mask[a, b]:
                        assert labels[a, b] == labels[i, j]
    for m in range(1, M + 1):   # each island alone is one component
        assert ndimage.label(labels == m, structure=np.ones((3, 3), np.int32))[1] == 1
