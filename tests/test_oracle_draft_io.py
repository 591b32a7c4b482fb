"""CPU pins of the oracle's Step 1 (draft sampling on given logits) and Step 7 stand-in
(majority down-sampler)."""
import numpy as np
import pytest
from scipy import stats

import oracle


def _params(H, W, V, r, **kw):
    return oracle.make_params(H, W, V, r, oracle.F32, **kw)


def test_sampler_is_the_pinned_primitives_in_step_1_order():
    """cell -> (1/T) -> top-k -> softmax -> inverse CDF at word 0 of the tag-1 stream."""
    rng = np.random.default_rng(3)
    H = W = 8
    r, V = 2, 96
    draft = (rng.standard_normal((H // r, W // r, V)) * 2).astype(np.float32)
    P = _params(H, W, V, r, temperature=0.8, top_k=20, seed=0x1234567890ABCDEF, round=5, image=9)
    tok, edge = oracle.sample_draft_tokens(P, draft, with_edge=True)
    for cell in range((H // r) * (W // r)):
        z = oracle.preprocess_row(draft.reshape(-1, V)[cell], None, 0.0, 0.8)
        q, _, _ = oracle.softmax_masked(z, oracle.topk_threshold(z, 20))
        u = oracle.position_uniforms(0x1234567890ABCDEF, 9, cell, 5, tag=1)[0]
        want, _, gap = oracle.inverse_cdf(q, u)
        assert tok.ravel()[cell] == want
        assert edge.ravel()[cell] == (gap < 1e-6)
        assert q[want] > 0            # never a token outside the top-k set
    # the tag matters: the tag-0 stream (acceptance uniforms) gives other draws
    other = [oracle.inverse_cdf(oracle.softmax_masked(
        oracle.preprocess_row(draft.reshape(-1, V)[c], None, 0.0, 0.8),
        oracle.topk_threshold(oracle.preprocess_row(draft.reshape(-1, V)[c], None, 0.0, 0.8), 20))[0],
        oracle.position_uniforms(0x1234567890ABCDEF, 9, c, 5, tag=0)[0])[0] for c in range(16)]
    assert list(tok.ravel()) != other


def test_sampler_frequencies_follow_q():
    rng = np.random.default_rng(11)
    V = 12
    row = (rng.standard_normal(V) * 1.5).astype(np.float32)
    draft = np.broadcast_to(row, (4, 4, V)).copy()       # 16 cells with the same distribution
    z = oracle.preprocess_row(row, None, 0.0, 1.0)
    q, _, _ = oracle.softmax_masked(z, oracle.topk_threshold(z, 6))
    counts = np.zeros(V)
    rounds = 400
    for rnd in range(rounds):
        P = _params(4, 4, V, 1, top_k=6, seed=77, round=rnd)
        counts += np.bincount(oracle.sample_draft_tokens(P, draft).ravel(), minlength=V)
    assert (counts[q == 0] == 0).all()
    keep = q > 0
    chi2 = ((counts[keep] - 16 * rounds * q[keep]) ** 2 / (16 * rounds * q[keep])).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-6, keep.sum() - 1)
    # greedy limit: a very low temperature always returns the arg max
    P = _params(4, 4, V, 1, temperature=1e-3, seed=1)
    assert (oracle.sample_draft_tokens(P, draft) == int(np.argmax(row))).all()


@pytest.mark.parametrize("r", [1, 2, 3, 4])
def test_downsampler_inverts_replication(r):
    rng = np.random.default_rng(r)
    y = rng.integers(0, 1000, (5, 7)).astype(np.int32)
    x = np.repeat(np.repeat(y, r, axis=0), r, axis=1)       # U_r: replication
    np.testing.assert_array_equal(oracle.downsample_majority(x, r), y)
    # a minority of changed tokens per block does not change the answer
    if r >= 2:
        x2 = x.copy()
        x2[::r, ::r] = 1000 + rng.integers(0, 5, y.shape)    # one of r*r tokens per block
        if r * r - 1 > 1:
            np.testing.assert_array_equal(oracle.downsample_majority(x2, r), y)


@pytest.mark.parametrize("r", [2, 3, 4])
def test_downsampler_against_scipy_mode_when_the_majority_is_unique(r):
    rng = np.random.default_rng(100 + r)
    h, w = 6, 9
    x = rng.integers(0, 4, (h * r, w * r)).astype(np.int32)
    y = oracle.downsample_majority(x, r)
    checked = 0
    for a in range(h):
        for c in range(w):
            block = x[a * r:(a + 1) * r, c * r:(c + 1) * r].ravel()
            counts = np.bincount(block)
            if (counts == counts.max()).sum() == 1:
                assert y[a, c] == stats.mode(block, keepdims=False).mode
                checked += 1
            else:
                assert counts[y[a, c]] == counts.max()
    assert checked > 10


def test_downsampler_ties_go_to_the_first_in_raster_order():
    blocks = {
        (5, 5, 7, 7): 5, (7, 5, 5, 7): 7, (1, 2, 2, 3): 2, (4, 3, 2, 1): 4, (9, 8, 9, 8): 9, (8, 9, 9, 8): 8,
    }
    for block, want in blocks.items():
        x = np.array(block, np.int32).reshape(2, 2)
        assert oracle.downsample_majority(x, 2)[0, 0] == want
    x = np.array([[3, 1, 2], [2, 1, 3], [0, 0, 6]], np.int32)     # 3, 1, 2, 0 twice each: 3 comes first
    assert oracle.downsample_majority(x, 3)[0, 0] == 3
    x[2, 2] = 1                                                   # now 1 three times
    assert oracle.downsample_majority(x, 3)[0, 0] == 1
