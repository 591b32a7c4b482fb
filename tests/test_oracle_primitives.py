"""Pins for the oracle's building blocks (CPU only).

Each test checks the oracle against something other than itself: published
known answers, torch/numpy/scipy library routines, closed forms, brute force.
"""
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Philox

def test_philox_known_answers(orc):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        v = [int(x, 16) for x in row]
        assert orc.philox4x32_10(v[0:4], v[4:6]) == tuple(v[6:10])


def test_uniforms_are_24_bit_and_keyed(orc):
    seen = set()
    us = []
    for pos in range(2000):
        u = orc.position_uniforms(seed=(5 << 32) | 9, image=3, position=pos, round=2)
        for x in u:
            assert 0.0 <= x < 1.0
            assert x * (1 << 24) == int(x * (1 << 24))          # top-24-bit grid
            assert np.float32(x) == x                            # exact in fp32
        seen.add(u)
        us.extend(u)
    assert len(seen) == 2000
    us = np.array(us)
    # uniformity: mean 1/2, variance 1/12, chi-square over 16 bins
    assert abs(us.mean() - 0.5) < 4 * np.sqrt(1 / 12 / us.size)
    assert abs(us.var() - 1 / 12) < 0.01
    hist = np.histogram(us, bins=16, range=(0, 1))[0]
    chi2 = ((hist - us.size / 16) ** 2 / (us.size / 16)).sum()
    assert chi2 < 45.0   # df=15, p ~ 1e-4
    # every key / counter part changes the stream
    base = orc.position_uniforms(1, 2, 3, 4)
    assert base != orc.position_uniforms(2, 2, 3, 4)
    assert base != orc.position_uniforms(1 | (1 << 32), 2, 3, 4)
    assert base != orc.position_uniforms(1, 3, 3, 4)
    assert base != orc.position_uniforms(1, 2, 4, 4)
    assert base != orc.position_uniforms(1, 2, 3, 5)
    assert base != orc.position_uniforms(1, 2, 3, 4, tag=1)
    # counter layout: (position, image, round, tag), key = (seed lo, seed hi)
    w = orc.philox4x32_10([3, 2, 4, 0], [1, 0])
    assert base == tuple((x >> 8) / 2 ** 24 for x in w[:3])


# ------------------------------------------------- pre-processing / softmax

def _bf16_bits(t):
    return t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_preprocess_matches_fp32_definition(orc):
    g = torch.Generator().manual_seed(1)
    c = torch.randn(512, generator=g) * 2
    u = c + torch.randn(512, generator=g)
    cb, ub = _bf16_bits(c), _bf16_bits(u)
    cf = c.to(torch.bfloat16).float()
    uf = u.to(torch.bfloat16).float()
    # no CFG: bf16 -> fp32 exactly, times 1/T in fp32
    z = orc.preprocess_row(cb, None, temperature=0.7)
    want = cf.numpy() * np.float32(1.0 / np.float32(0.7))
    assert np.array_equal(z, want.astype(np.float32))
    # CFG identities: s = 1 -> cond, s = 0 -> uncond, equal rows -> identity
    assert np.array_equal(orc.preprocess_row(cb, ub, cfg_scale=1.0), cf.numpy())
    assert np.array_equal(orc.preprocess_row(cb, ub, cfg_scale=0.0), uf.numpy())
    assert np.array_equal(orc.preprocess_row(cb, cb, cfg_scale=3.0), cf.numpy())
    # general s: u + s (c - u), fused multiply-add => compare with float64 math
    z = orc.preprocess_row(cb, ub, cfg_scale=3.0)
    d = (cf - uf).double()           # exact here or one fp32 rounding
    d32 = (cf - uf).double()
    want = (3.0 * d32 + uf.double()).float().numpy()
    assert np.array_equal(z, want)
    # fp32 inputs pass through
    zf = orc.preprocess_row(c.numpy(), None)
    assert np.array_equal(zf, c.numpy())


@pytest.mark.parametrize("T", [1.0, 0.5, 2.0])
def test_softmax_matches_torch_fp64(orc, T):
    g = torch.Generator().manual_seed(2)
    x = torch.randn(4096, generator=g) * 3
    z = orc.preprocess_row(x.numpy(), None, temperature=T)
    p, m, Z = orc.softmax_masked(z)
    want = torch.softmax(torch.from_numpy(z).double(), dim=0).numpy()
    assert np.allclose(p, want, rtol=1e-12, atol=0)
    assert abs(p.sum() - 1) < 1e-12
    assert m == z.max()


@pytest.mark.parametrize("k", [1, 7, 100, 1000])
def test_topk_matches_torch_topk(orc, k):
    g = torch.Generator().manual_seed(3)
    x = (torch.randn(2048, generator=g) * 2).to(torch.bfloat16).float()   # many ties
    theta = orc.topk_threshold(x.numpy(), k)
    assert theta == torch.topk(x, k).values[-1].item()
    p, m, Z = orc.softmax_masked(x.numpy(), theta)
    keep = x >= torch.topk(x, k).values[-1]
    assert keep.sum() >= k
    want = torch.softmax(x.double().masked_fill(~keep, float("-inf")), dim=0).numpy()
    assert np.allclose(p, want, rtol=1e-12, atol=0)
    assert np.all((p > 0) == keep.numpy())


def test_topk_off_and_one_hot(orc):
    x = np.array([0.5, 2.0, -1.0, 2.0, 1.0, 0.0, -3.0, 0.25], np.float32)
    assert orc.topk_threshold(x, 0) == -np.inf
    assert orc.topk_threshold(x, 8) == -np.inf
    assert orc.topk_threshold(x, 100) == -np.inf
    th = orc.topk_threshold(x, 1)
    p, _, _ = orc.softmax_masked(x, th)
    assert np.allclose(p, [0, .5, 0, .5, 0, 0, 0, 0])        # ties kept
    assert orc.topk_threshold(x, 3) == 1.0


# ------------------------------------------------------------- inverse CDF

def test_inverse_cdf_matches_searchsorted(orc):
    rng = np.random.default_rng(4)
    for trial in range(50):
        V = int(rng.integers(1, 200))
        w = rng.random(V) * (rng.random(V) < 0.6)
        if w.sum() == 0:
            w[rng.integers(V)] = 1.0
        cs = np.cumsum(w)
        for u in rng.random(40):
            tok, Z, gap = orc.inverse_cdf(w, float(u))
            assert Z == pytest.approx(cs[-1], rel=1e-14)
            want = int(np.searchsorted(cs, u * cs[-1], side="right"))
            assert tok == want
            assert w[tok] > 0
            lo = cs[tok] - w[tok]
            assert gap == pytest.approx(min(u - lo / Z, cs[tok] / Z - u), abs=1e-12)


def test_inverse_cdf_special_cases(orc):
    w = np.zeros(16)
    assert orc.inverse_cdf(w, 0.3)[0] == -1                      # no mass
    w[5] = 2.0
    for u in (0.0, 0.25, 0.999999):
        assert orc.inverse_cdf(w, u)[0] == 5                     # one-hot
    n = 10
    w = np.zeros(32)
    active = np.arange(3, 3 + 2 * n, 2)
    w[active] = 0.125                                            # uniform over n tokens
    for u in np.linspace(0, 0.9999, 57):
        assert orc.inverse_cdf(w, float(u))[0] == active[int(np.floor(u * n))]
    # u = 0 never picks a leading zero-weight token
    w = np.array([0.0, 0.0, 1.0, 1.0])
    assert orc.inverse_cdf(w, 0.0)[0] == 2


# ---------------------------------------------------------------- dilation

def _brute_expand(rej, l, clip):
    H, W = rej.shape
    out = np.zeros_like(rej)
    idx = np.flatnonzero(rej.ravel())
    t0 = int(idx[0]) if idx.size else H * W
    for t in idx:
        it, jt = divmod(int(t), W)
        for u in range(H * W):
            iu, ju = divmod(u, W)
            if abs(iu - it) <= l and abs(ju - jt) <= l and (not clip or u >= t0):
                out[iu, ju] = 1
    return out, t0


@pytest.mark.parametrize("shape", [(1, 1), (4, 4), (8, 5), (16, 16), (7, 40)])
@pytest.mark.parametrize("l", [0, 1, 2, 3, 5])
def test_expand_vs_scipy_and_brute_force(orc, shape, l):
    from scipy.ndimage import binary_dilation
    rng = np.random.default_rng(hash((shape, l)) % 2 ** 32)
    for density in (0.0, 0.02, 0.2, 1.0):
        rej = (rng.random(shape) < density).astype(np.uint8)
        out0, t0 = orc.expand(rej, l, clip_before_first=0)
        want = binary_dilation(rej.astype(bool), structure=np.ones((2 * l + 1, 2 * l + 1), bool))
        assert np.array_equal(out0.astype(bool), want)
        out1, t0b = orc.expand(rej, l, clip_before_first=1)
        b1, bt0 = _brute_expand(rej, l, True)
        assert t0 == t0b == bt0
        assert np.array_equal(out1, b1)
        # nesting: R_T subset R_X(clip) subset R_X(no clip); R_X(clip) subset {u >= t0}
        assert np.all(rej <= out1) and np.all(out1 <= out0)
        assert not out1.ravel()[:t0].any()
        if l == 0:
            assert np.array_equal(out1, rej)


def test_expand_counts_and_composition(orc):
    rej = np.zeros((16, 16), np.uint8)
    rej[8, 8] = 1
    for l in (1, 2, 3):
        out, _ = orc.expand(rej, l, clip_before_first=0)
        assert out.sum() == (2 * l + 1) ** 2
    rej[:] = 0
    rej[0, 0] = 1
    for l in (1, 2, 3):
        assert orc.expand(rej, l, 0)[0].sum() == (l + 1) ** 2
    # e rounds of radius 1 == one round of radius e (box elements compose), and
    # the clip mask of the ORIGINAL t0 commutes with it
    rng = np.random.default_rng(9)
    rej = (rng.random((20, 24)) < 0.03).astype(np.uint8)
    cur = rej
    for e in (1, 2, 3):
        cur = orc.expand(cur, 1, 0)[0]
        assert np.array_equal(cur, orc.expand(rej, e, 0)[0])
        clipped = cur.copy().ravel()
        t0 = orc.expand(rej, e, 1)[1]
        clipped[:t0] = 0
        assert np.array_equal(clipped.reshape(rej.shape), orc.expand(rej, e, 1)[0])
    # monotone in l
    prev = rej
    for l in range(0, 6):
        out = orc.expand(rej, l, 1)[0]
        assert np.all(prev <= out) or l == 0
        prev = out


# ----------------------------------------------------------------- pooling

def test_pool_invariants_and_brute_force(orc):
    rng = np.random.default_rng(5)
    V = 8
    for trial in range(200):
        p = rng.random(V) ** 3
        p /= p.sum()
        tok = int(rng.integers(V))
        others = [x for x in rng.permutation(V) if x != tok]
        k = int(rng.integers(2, V + 1))
        nn_row = np.array([tok] + others[:k - 1], np.uint16)
        delta = float(rng.choice([0.0, 0.05, 0.1, 0.4, 2.0]))
        P, pp, J, gap = orc.pool(p, nn_row, k, delta, tok)
        # brute force over every prefix length: the longest prefix with all
        # partial sums < delta
        best = 0
        for j in range(1, k):
            if all(p[nn_row[1:m + 1]].sum() < delta for m in range(1, j + 1)):
                best = j
        assert J == best
        moved = p[nn_row[1:J + 1]].sum()
        assert P == pytest.approx(p[tok] + moved, abs=1e-15)
        assert moved < delta or J == 0                         # Eq. 4: TVD = moved mass < delta
        assert 0.5 * np.abs(pp - p).sum() == pytest.approx(moved, abs=1e-15)
        assert pp.sum() == pytest.approx(1.0, abs=1e-14)
        assert P >= p[tok]
        if delta == 0.0:
            assert J == 0 and P == p[tok] and np.array_equal(pp, p)
        if delta > 1.0 and k == V:
            assert P == pytest.approx(1.0, abs=1e-14)
    # pooling off
    P, pp, J, gap = orc.pool(p, None, 1, 0.1, 3)
    assert P == p[3] and J == 0 and np.array_equal(pp, p)


# -------------------------------------------------------------- acceptance

def test_accept_threshold_closed_form(orc):
    assert orc.accept_threshold(0.2, 0.4) == 0.5
    assert orc.accept_threshold(0.5, 0.25) == 1.0
    assert orc.accept_threshold(0.3, 0.3) == 1.0
    assert orc.accept_threshold(0.0, 0.3) == 0.0
    assert orc.accept_threshold(0.1, 0.0) == 1.0     # q = 0: accept iff P > 0
    assert orc.accept_threshold(0.0, 0.0) == 0.0


def test_residual_is_normalised_tvd(orc):
    rng = np.random.default_rng(6)
    for trial in range(50):
        V = 64
        p = rng.random(V) ** 4
        p /= p.sum()
        q = rng.random(V) ** 4
        q /= q.sum()
        w = orc.residual_weights(p, q, 1.0)
        assert np.array_equal(w, np.maximum(0.0, p - q))
        assert w.sum() == pytest.approx(1 - np.minimum(p, q).sum(), abs=1e-14)
        assert w.sum() == pytest.approx(0.5 * np.abs(p - q).sum(), abs=1e-14)
        assert np.all((w > 0) <= (p > q))
        assert (w / w.sum()).sum() == pytest.approx(1.0, abs=1e-14)
        assert np.array_equal(orc.residual_weights(p, q, 0.0), p)
        for u in rng.random(20):
            tok = orc.inverse_cdf(w, float(u))[0]
            assert p[tok] > q[tok]                               # never a zero-weight token
