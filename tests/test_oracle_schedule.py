"""CPU pins of the oracle's island schedule (Sec. 3.4: islands concurrently, a ZipAR-style row window
inside an island)."""
import numpy as np
import pytest

import oracle


def simulate(labels, window):
    """Time-stepped simulation of the rule itself: in every step, every position whose requirements were met
    BEFORE the step is decoded -- its predecessors in the island's row, and the island's positions of the
    row above up to `window - 1` columns beyond it."""
    H, W = labels.shape
    done = np.zeros((H, W), bool)
    step = np.zeros((H, W), np.int32)
    todo = int((labels > 0).sum())
    t = 0
    while todo:
        t += 1
        ready = []
        for i in range(H):
            for j in range(W):
                m = labels[i, j]
                if m <= 0 or done[i, j]:
                    continue
                ok = all(done[i, jj] for jj in range(j) if labels[i, jj] == m)
                if ok and i > 0:
                    ok = all(done[i - 1, jj] for jj in range(min(W, j + window)) if labels[i - 1, jj] == m)
                if ok:
                    ready.append((i, j))
        assert ready, "the rule can always advance"
        for i, j in ready:
            done[i, j] = True
            step[i, j] = t
        todo -= len(ready)
    return step, t


@pytest.mark.parametrize("window", [1, 2, 4, 16])
@pytest.mark.parametrize("density", [0.15, 0.4, 0.8])
def test_against_the_simulation(window, density):
    rng = np.random.default_rng(window * 10 + int(density * 100))
    mask = (rng.random((12, 19)) < density).astype(np.uint8)
    labels, M, _, _ = oracle.islands(mask)
    step, nfe = oracle.island_schedule(labels, window)
    want, t = simulate(labels, window)
    np.testing.assert_array_equal(step, want)
    assert nfe == t == step.max()
    assert ((step > 0) == (mask > 0)).all()


@pytest.mark.parametrize("H,W,window", [(4, 9, 1), (6, 10, 3), (8, 8, 8), (5, 32, 16), (3, 7, 2)])
def test_full_grid_closed_form(H, W, window):
    """One island covering the grid: row i starts `window` steps after row i - 1: W + (H - 1) w steps."""
    labels = np.ones((H, W), np.int32)
    step, nfe = oracle.island_schedule(labels, window)
    assert nfe == W + (H - 1) * window
    np.testing.assert_array_equal(step, np.add.outer(np.arange(H) * window, np.arange(W) + 1))


def test_window_spanning_the_row_is_raster_order_inside_an_island():
    rng = np.random.default_rng(5)
    mask = (rng.random((10, 14)) < 0.45).astype(np.uint8)
    labels, M, _, size = oracle.islands(mask)
    step, nfe = oracle.island_schedule(labels, 14 + 1)
    for m in range(1, M + 1):
        s = step[labels == m]                     # raster order of the island's positions
        assert s.max() <= size[m - 1]
        assert (np.diff(s) > 0).all()             # strictly later along the raster
    solid = np.zeros((6, 8), np.uint8)
    solid[1:5, 2:7] = 1
    labels, M, _, size = oracle.islands(solid)
    step, nfe = oracle.island_schedule(labels, 100)
    assert nfe == size[0] == 20
    np.testing.assert_array_equal(step[1:5, 2:7], np.arange(1, 21).reshape(4, 5))


def test_islands_run_concurrently_and_empty_grid():
    labels = np.zeros((5, 12), np.int32)
    assert oracle.island_schedule(labels, 4)[1] == 0
    labels[0, 0:3] = 1
    labels[3, 5:11] = 2
    labels[4, 5:11] = 2
    step, nfe = oracle.island_schedule(labels, 2)
    np.testing.assert_array_equal(step[0, 0:3], [1, 2, 3])
    np.testing.assert_array_equal(step[3, 5:11], [1, 2, 3, 4, 5, 6])
    np.testing.assert_array_equal(step[4, 5:11], [3, 4, 5, 6, 7, 8])     # column 5 waits for columns <= 6 above
    assert nfe == 8                                                     # not 3 + 12: the islands overlap in time
