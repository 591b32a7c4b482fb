"""Pins of the oracle's step-by-step redraw of R_X (Sec. 3.4, Algorithm 1 Step 6): with a window as
wide as the grid the schedule is raster order and the loop is a plain sequential redraw; the number of
target-model calls is the schedule's step count; the tokens it draws follow the target distribution."""
import numpy as np
import pytest

import oracle as orc


def _logits(rng, n_steps, H, W, V):
    return [rng.normal(0.0, 2.0, (H, W, V)).astype(np.float32) for _ in range(n_steps)]


def _params(H, W, V, **kw):
    return orc.make_params(H, W, V, 1, orc.F32, **kw)


def _target_row(P, cond_row, uncond_row):
    z = orc.preprocess_row(cond_row, uncond_row, cfg_scale=P.cfg_scale, temperature=P.temperature)
    p, _, _ = orc.softmax_masked(z, orc.topk_threshold(z, P.top_k))
    return p


def test_wide_window_is_a_raster_order_redraw():
    """One island covering the grid, window >= W: step(t) = t + 1, so call s redraws exactly position
    s - 1 -- the loop must equal redrawing the positions one after the other in raster order, each from the
    logits of its own call and with its own uniform."""
    H, W, V = 4, 6, 64
    rng = np.random.default_rng(5)
    labels = np.ones((H, W), np.int32)
    step, nfe = orc.island_schedule(labels, window=W)
    assert np.array_equal(step.ravel(), np.arange(1, H * W + 1)) and nfe == H * W
    P = _params(H, W, V, top_k=20, temperature=0.8, cfg_scale=2.0, seed=77, round=3, image=2)
    cond, unc = _logits(rng, nfe, H, W, V), _logits(rng, nfe, H, W, V)
    start = rng.integers(0, V, (H, W)).astype(np.int32)
    got, calls = orc.redraw_loop(P, step, cond, unc, start)
    assert calls == nfe
    want = start.copy().ravel()
    for t in range(H * W):          # sequential: call t + 1 decodes position t
        p = _target_row(P, cond[t][t // W, t % W], unc[t][t // W, t % W])
        u = orc.position_uniforms(77, 2, t, 3, tag=1 + (t + 1))[0]
        want[t] = orc.inverse_cdf(p, u)[0]
    assert np.array_equal(got.ravel(), want)


def test_calls_equal_schedule_steps_and_positions_outside_keep_their_token():
    H, W, V = 8, 10, 32
    rng = np.random.default_rng(6)
    rx = np.zeros((H, W), np.uint8)
    rx[1:4, 2:7] = 1
    rx[6:8, 0:3] = 1
    rx[5, 9] = 1
    labels, n, _, _ = orc.islands(rx)
    assert n == 3
    for window in (1, 2, 16):
        step, nfe = orc.island_schedule(labels, window=window)
        # the islands run concurrently: the image needs as many calls as its slowest island has steps
        assert nfe == step.max() and nfe < rx.sum()
        P = _params(H, W, V, seed=9, image=0)
        cond = _logits(rng, nfe, H, W, V)
        start = rng.integers(0, V, (H, W)).astype(np.int32)
        got, calls = orc.redraw_loop(P, step, cond, None, start)
        assert calls == nfe
        assert np.array_equal(got[rx == 0], start[rx == 0])
        # every position of R_X took its token from the call its step names (and from no other)
        for (i, j) in np.argwhere(rx == 1):
            s = int(step[i, j])
            p = _target_row(P, cond[s - 1][i, j], None)
            u = orc.position_uniforms(9, 0, i * W + j, 0, tag=1 + s)[0]
            assert got[i, j] == orc.inverse_cdf(p, u)[0]
    # a wider window makes a position wait for more of the row above: never fewer calls
    n1 = orc.island_schedule(labels, window=1)[1]
    n16 = orc.island_schedule(labels, window=16)[1]
    assert n1 <= n16 <= rx.sum()


def test_redrawn_tokens_follow_the_target_distribution():
    """Chi-square of the token drawn at one position over many rounds against its target distribution."""
    H, W, V = 1, 2, 12
    rng = np.random.default_rng(7)
    step = np.array([[1, 2]], np.int32)
    cond = _logits(rng, 2, H, W, V)
    counts = np.zeros(V)
    n = 6000
    P0 = _params(H, W, V, top_k=8, seed=123, image=4)
    p = _target_row(P0, cond[1][0, 1], None)
    for rnd in range(n):
        P = _params(H, W, V, top_k=8, seed=123, image=4, round=rnd)
        got, _ = orc.redraw_loop(P, step, cond, None, np.zeros((H, W), np.int32))
        counts[got[0, 1]] += 1
    live = p > 0
    assert counts[~live].sum() == 0 and live.sum() == 8
    chi2 = float((((counts[live] - n * p[live]) ** 2) / (n * p[live])).sum())
    assert chi2 < 29.9          # 99.99 % point of chi-square with 7 degrees of freedom
    # the two positions use different uniforms (different position and step words)
    assert orc.position_uniforms(123, 4, 0, 0, tag=2)[0] != orc.position_uniforms(123, 4, 1, 0, tag=3)[0]
