"""Pins for the oracle's whole round (CPU only): the invariants the method must
satisfy, exhaustive enumeration on tiny vocabularies, and a chi-square test."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2601_05149_b200 import synth


def _params(orc, cfg, image=0, **over):
    kw = dict(temperature=cfg.temperature, top_k=cfg.top_k, cfg_scale=cfg.cfg_scale,
              accept_mode=cfg.accept_mode, tau=cfg.tau, pool_k=cfg.pool_k,
              pool_delta=cfg.pool_delta, radius=cfg.radius,
              clip_before_first=cfg.clip_before_first, resample_mode=cfg.resample_mode,
              seed=cfg.seed, round=cfg.round, image=image)
    kw.update(over)
    return orc.make_params(cfg.H, cfg.W, cfg.V, cfg.r, orc.BF16 if cfg.dtype == "bf16" else orc.F32,
                           **kw)


def _image(cfg, b=0):
    import oracle
    img = synth.make_image(cfg, b)
    draft = synth.to_numpy_logits(img["draft_lo"])
    tok = oracle.sample_draft_tokens(_params(oracle, cfg, b), draft)
    return (synth.to_numpy_logits(img["cond"]),
            None if img["uncond"] is None else synth.to_numpy_logits(img["uncond"]),
            draft, tok)


SMALL = synth.RoundConfig("small", B=1, H=8, W=8, V=256, dtype="f32", sigma=0.7, radius=1, seed=11)


def test_a_residual_with_next_to_no_mass_is_flagged_borderline(orc):
    """Target one ulp away from the draft in a single logit: the residual max(0, p - q) holds about 1e-8 of
    mass, so its normalised CDF means nothing at the tolerance of the probabilities -- every residual draw
    there carries the CDF-edge flag.  With the target equal to the draft the residual is exactly empty, the
    draw falls back to the target weights (mass 1) and is flagged only by the usual edge test."""
    cfg = dataclasses.replace(SMALL, dtype="f32", sigma=0.0, resample_mode=orc.RESAMPLE_RESIDUAL_ALL, radius=8,
                              clip_before_first=0)
    cond, uncond, draft, tok = _image(cfg)
    cond = cond.copy()
    cond[:, :, 5] = np.nextafter(cond[:, :, 5], np.float32(np.inf))
    # force one rejection so that R_X (radius 8, no clipping) covers the grid
    cond[0, 0, :] = -30.0
    cond[0, 0, (int(tok[0, 0]) + 1) % cfg.V] = 30.0
    out = orc.round_image(_params(orc, cfg), cond, None, draft, tok)
    assert out["reject"][0, 0] == 1 and out["expand"].all()
    near = np.ones((cfg.H, cfg.W), bool)
    near[0, 0] = False
    assert (out["flags"][near] & orc.FLAG_CDF_EDGE).all()
    assert not (out["flags"][0, 0] & orc.FLAG_CDF_EDGE)          # a residual with all the mass: decided
    same = orc.round_image(_params(orc, cfg), np.kron(draft, np.ones((2, 2, 1), np.float32)), None, draft, tok)
    assert same["reject"].sum() == 0


@pytest.mark.parametrize("dtype,top_k", [("f32", 0), ("bf16", 0), ("bf16", 40)])
def test_target_equal_to_draft_accepts_everything(orc, dtype, top_k):
    cfg = dataclasses.replace(SMALL, dtype=dtype, top_k=top_k, sigma=0.0)
    cond, uncond, draft, tok = _image(cfg)
    # sigma = 0: the conditional row is the up-sampled draft row, bit for bit
    assert np.array_equal(cond[::2, ::2], draft)
    out = orc.round_image(_params(orc, cfg), cond, None, draft, tok)
    assert out["reject"].sum() == 0 and out["expand"].sum() == 0
    assert np.array_equal(out["out_tok"], np.kron(tok, np.ones((2, 2), np.int32)))
    assert np.all(out["accept_prob"] == 1.0)
    assert np.allclose(out["p_tok"], out["q_tok"], rtol=1e-15)
    assert list(out["counts"]) == [0, 0, cfg.H * cfg.W]


def test_probabilities_against_torch(orc):
    cfg = dataclasses.replace(SMALL, dtype="bf16", top_k=50, cfg_scale=3.0, temperature=0.8)
    cond, uncond, draft, tok = _image(cfg)
    out = orc.round_image(_params(orc, cfg), cond, uncond, draft, tok)
    c = torch.from_numpy(cond.view(np.int16)).view(torch.bfloat16).float()
    u = torch.from_numpy(uncond.view(np.int16)).view(torch.bfloat16).float()
    d = torch.from_numpy(draft.view(np.int16)).view(torch.bfloat16).float()
    invT = np.float32(1.0) / np.float32(0.8)
    z = ((3.0 * (c - u).double() + u.double()).float() * invT)
    zq = d * invT

    def probs(z):
        kth = torch.topk(z, 50, dim=-1).values[..., -1:]
        return torch.softmax(z.double().masked_fill(z < kth, float("-inf")), dim=-1)

    p, q = probs(z), probs(zq)
    tok_hi = torch.from_numpy(np.kron(tok, np.ones((2, 2), np.int64)))
    q_hi = q.repeat_interleave(2, 0).repeat_interleave(2, 1)
    p_tok = p.gather(-1, tok_hi[..., None])[..., 0].numpy()
    q_tok = q_hi.gather(-1, tok_hi[..., None])[..., 0].numpy()
    assert np.allclose(out["p_tok"], p_tok, rtol=1e-12)
    assert np.allclose(out["q_tok"], q_tok, rtol=1e-12)
    assert np.allclose(out["accept_prob"], np.minimum(1.0, p_tok / q_tok), rtol=1e-12)
    # decisions follow u < thr with the position's first uniform
    for t in range(cfg.H * cfg.W):
        u0 = orc.position_uniforms(cfg.seed, 0, t, cfg.round)[0]
        assert out["reject"].ravel()[t] == (0 if u0 < out["accept_prob"].ravel()[t] else 1)


def test_acceptance_rate_is_sum_min_p_q(orc):
    """E_{x~ ~ q}[accept] = sum_x min(p(x), q(x)), checked per position in closed
    form and by Monte Carlo over rounds with fresh draft tokens."""
    cfg = dataclasses.replace(SMALL, H=4, W=4, V=64, sigma=1.0, seed=21)
    cond, _, draft, _ = _image(cfg)
    P0 = _params(orc, cfg)
    closed = np.zeros((cfg.H, cfg.W))
    for i in range(cfg.H):
        for j in range(cfg.W):
            q, p, pp, mass = orc.position_distributions(P0, cond[i, j], None, draft[i // 2, j // 2], 0)
            closed[i, j] = np.minimum(p, q).sum()
            # sum_x q(x) min(1, p/q) is the same number
            thr = np.array([orc.accept_threshold(p[x], q[x]) for x in range(cfg.V)])
            assert (q * thr).sum() == pytest.approx(closed[i, j], abs=1e-12)
    rounds = 4000
    acc = np.zeros((cfg.H, cfg.W))
    for rnd in range(rounds):
        Pr = _params(orc, cfg, round=rnd)
        tok = orc.sample_draft_tokens(Pr, draft)          # x~ ~ q, tag-1 stream
        out = orc.round_image(Pr, cond, None, draft, tok)
        acc += 1 - out["reject"]
    rate = acc / rounds
    sd = np.sqrt(closed * (1 - closed) / rounds)
    assert np.all(np.abs(rate - closed) < 4.5 * sd + 1e-9)


def _exact_output_pmf(orc, q, p_prime, P_of_tok, V):
    """Exact pmf of accept-then-resample when x~ ~ q, counting every one of the
    2^24 values each uniform can take."""
    N = 1 << 24
    out = np.zeros(V)
    for tok in range(V):
        if q[tok] == 0:
            continue
        thr = orc.accept_threshold(P_of_tok[tok], q[tok])
        n_acc = int(np.ceil(thr * N))                     # #{n : n/2^24 < thr}
        n_acc = min(n_acc, N)
        out[tok] += q[tok] * n_acc / N
        if n_acc < N:
            w = orc.residual_weights(p_prime[tok], q, 1.0)
            hist = orc.inverse_cdf_histogram(w)
            assert hist.sum() == N
            out += q[tok] * (1 - n_acc / N) * hist / N
    return out


@pytest.mark.parametrize("V,seed", [(4, 0), (8, 1), (8, 2)])
def test_exactness_by_enumeration(orc, V, seed):
    """Accept with min(1, p/q), else redraw from norm(max(0, p - q)): the output
    is distributed as p.  Enumerated exactly over all draft tokens and all 2^24
    values of both uniforms; the only slack is the 2^-24 grid."""
    rng = np.random.default_rng(seed)
    p = rng.random(V) ** 2
    p /= p.sum()
    q = rng.random(V) ** 2
    q /= q.sum()
    pmf = _exact_output_pmf(orc, q, [p] * V, p, V)
    assert np.abs(pmf - p).max() < V * 2.0 ** -24
    assert pmf.sum() == pytest.approx(1.0, abs=1e-12)
    # a dropped term shows up: using q as the redraw distribution is NOT exact
    bad = sum(q[t] * (orc.accept_threshold(p[t], q[t]) * np.eye(V)[t]
                      + (1 - orc.accept_threshold(p[t], q[t])) * q) for t in range(V))
    assert np.abs(bad - p).max() > 1e-3


@pytest.mark.parametrize("radius,mode", [(0, "MIXED"), (1, "ISOLATED_RESIDUAL")])
def test_round_output_distribution_chi_square(orc, radius, mode):
    """Whole-round check on a tiny grid with x~ ~ q: every position's output is a
    draw from its p.  That holds (a) without expansion, where the round is plain
    accept-then-residual, and (b) with expansion under the rule "residual only for
    a rejected position no other rejection covers, p for the rest of R_X".  Run
    with r = 1 so that every position has its own draft token (nearest-neighbour
    up-sampling makes the r*r siblings share one token, which ties a position's
    being swept in to its own token).  The default mixed rule is NOT exact for
    l > 0 (an accepted token survives only when no neighbour was rejected, which
    over-weights the residual): the last assertion shows the test sees that."""
    from scipy.stats import chi2
    cfg = dataclasses.replace(SMALL, H=4, W=4, V=8, r=1, sigma=1.0, radius=radius, seed=31,
                              resample_mode=getattr(orc, "RESAMPLE_" + mode))
    cond, _, draft, _ = _image(cfg)
    rounds = 20000
    counts = np.zeros((cfg.H, cfg.W, cfg.V))
    mixed = np.zeros_like(counts)
    ii, jj = np.meshgrid(np.arange(cfg.H), np.arange(cfg.W), indexing="ij")
    n_expanded_only = 0
    for rnd in range(rounds):
        Pr = _params(orc, cfg, round=rnd)
        tok = orc.sample_draft_tokens(Pr, draft)
        out = orc.round_image(Pr, cond, None, draft, tok)
        counts[ii, jj, out["out_tok"]] += 1
        n_expanded_only += int((out["expand"] & ~out["reject"] & 1).sum())
        if radius:
            out = orc.round_image(_params(orc, cfg, round=rnd, resample_mode=orc.RESAMPLE_MIXED),
                                  cond, None, draft, tok)
            mixed[ii, jj, out["out_tok"]] += 1
    assert (n_expanded_only > rounds) == (radius > 0)    # the expansion branch is exercised
    P0 = _params(orc, cfg)

    def worst_p(cnt):
        worst = 1.0
        for i in range(cfg.H):
            for j in range(cfg.W):
                q, p, _, _ = orc.position_distributions(P0, cond[i, j], None, draft[i, j], 0)
                stat = ((cnt[i, j] - rounds * p) ** 2 / (rounds * p)).sum()
                worst = min(worst, chi2.sf(stat, cfg.V - 1))
        return worst

    assert worst_p(counts) > 1e-3 / (cfg.H * cfg.W)    # Bonferroni over the 16 positions
    if radius:
        assert worst_p(mixed) < 1e-12


def test_modes_and_masks(orc):
    cfg = dataclasses.replace(SMALL, sigma=1.5, radius=2, seed=41)
    cond, _, draft, tok = _image(cfg)
    base = orc.round_image(_params(orc, cfg), cond, None, draft, tok)
    rej, exp = base["reject"].astype(bool), base["expand"].astype(bool)
    assert rej.any() and (exp & ~rej).any()
    tok_hi = np.kron(tok, np.ones((2, 2), np.int32))
    assert np.array_equal(base["out_tok"][~exp], tok_hi[~exp])
    assert np.array_equal(base["out_tok"][exp], base["cand_tok"][exp])
    assert list(base["counts"]) == [rej.sum(), exp.sum(), np.flatnonzero(rej.ravel())[0]]
    e2, t0 = orc.expand(base["reject"], cfg.radius, 1)
    assert np.array_equal(e2, base["expand"])
    # the forced modes agree with the mixed rule where their rule coincides
    res_all = orc.round_image(_params(orc, cfg, resample_mode=orc.RESAMPLE_RESIDUAL_ALL),
                              cond, None, draft, tok)
    tgt_all = orc.round_image(_params(orc, cfg, resample_mode=orc.RESAMPLE_TARGET_ALL),
                              cond, None, draft, tok)
    assert np.array_equal(res_all["reject"], base["reject"])
    assert np.array_equal(res_all["out_tok"][rej], base["out_tok"][rej])
    assert np.array_equal(tgt_all["out_tok"][exp & ~rej], base["out_tok"][exp & ~rej])
    # a residual draw always lands where p > q
    P0 = _params(orc, cfg)
    for (i, j) in zip(*np.nonzero(rej)):
        q, p, _, _ = orc.position_distributions(P0, cond[i, j], None, draft[i // 2, j // 2], 0)
        x = base["out_tok"][i, j]
        assert p[x] > q[x] and x != tok_hi[i, j]
    # radius 0 = naive local verification: R_X = R_T
    l0 = orc.round_image(_params(orc, cfg, radius=0), cond, None, draft, tok)
    assert np.array_equal(l0["expand"], l0["reject"])
    # the relaxed rule of Eq. 5: tau = 0 accepts all, tau > 1 rejects all
    a = orc.round_image(_params(orc, cfg, accept_mode=orc.ACCEPT_THRESHOLD, tau=0.0),
                        cond, None, draft, tok)
    assert a["reject"].sum() == 0
    b = orc.round_image(_params(orc, cfg, accept_mode=orc.ACCEPT_THRESHOLD, tau=1.5,
                                resample_mode=orc.RESAMPLE_TARGET_ALL), cond, None, draft, tok)
    assert b["reject"].all() and b["expand"].all() and b["counts"][2] == 0
    mid = orc.round_image(_params(orc, cfg, accept_mode=orc.ACCEPT_THRESHOLD, tau=1e-3),
                          cond, None, draft, tok)
    assert np.array_equal(mid["reject"].astype(bool), mid["p_tok"] < np.float32(1e-3))


def test_pooling_never_lowers_acceptance(orc):
    cfg = dataclasses.replace(SMALL, V=512, top_k=100, pool_k=64, pool_delta=0.1, sigma=1.0, seed=51,
                              dtype="bf16")
    cond, _, draft, tok = _image(cfg)
    nn = synth.neighbours_to_numpy(synth.codebook_neighbours(cfg.V, cfg.pool_k, cfg.seed))
    assert np.array_equal(nn[:, 0], np.arange(cfg.V))            # self first
    assert all(len(set(r)) == cfg.pool_k for r in nn[:16])
    off = orc.round_image(_params(orc, cfg, pool_k=1), cond, None, draft, tok)
    on = orc.round_image(_params(orc, cfg), cond, None, draft, tok, nn)
    assert np.all(on["accept_prob"] >= off["accept_prob"] - 1e-15)
    assert np.all(on["reject"] <= off["reject"])
    assert (on["accept_prob"] > off["accept_prob"]).any()
    assert np.array_equal(on["p_tok"], off["p_tok"])
    # the pooled mass never adds delta or more to p(x~)  (Eq. 4)
    ratio_gain = on["accept_prob"] * on["q_tok"] - on["p_tok"]
    assert np.all(ratio_gain[on["accept_prob"] < 1] < cfg.pool_delta)
