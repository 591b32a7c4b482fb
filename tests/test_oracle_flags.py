"""Pins for the two oracle parts every GPU parity test leans on (CPU only):

* ``upsample_pool_image`` (the checker of ``mulo_upsample_pool``) against a torch fp64
  restatement of the draft row statistics;
* the borderline flags of ``round_image``: which positions the comparison may excuse.  They are
  recomputed here, position by position, from primitives that have pins of their own
  (``position_uniforms``, ``accept_threshold``, ``pool``'s gap, ``inverse_cdf``'s gap), including
  which draw's flag a position carries under each resample mode, and on inputs built so that a
  uniform sits a known distance from its threshold.
"""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2601_05149_b200 import synth
from test_oracle_round import SMALL, _image, _params

EDGE = 1e-6            # "within 1e-6 of its decision threshold"
MIN_RESIDUAL_MASS = 1e-5   # a residual holding less mass than this decides nothing


def test_upsample_pool_image_against_torch(orc):
    cfg = dataclasses.replace(SMALL, H=6, W=10, V=384, dtype="bf16", top_k=37, temperature=0.7, seed=61)
    _, _, draft, tok = _image(cfg)
    got = orc.upsample_pool_image(_params(orc, cfg), draft, tok)
    d = torch.from_numpy(draft.view(np.int16)).view(torch.bfloat16).float()
    z = d * (np.float32(1.0) / np.float32(0.7))                     # fp32 multiply by fp32(1/T)
    kth = torch.topk(z, 37, dim=-1).values[..., -1]
    assert np.array_equal(got["stats"][..., 0], kth.double().numpy())   # theta: exact
    keep = z >= kth[..., None]
    m = z.masked_fill(~keep, float("-inf")).max(dim=-1).values.double()
    Z = (torch.exp(z.double() - m[..., None]) * keep).sum(dim=-1)
    assert np.array_equal(got["stats"][..., 1], m.numpy())
    assert np.allclose(got["stats"][..., 2], Z.numpy(), rtol=1e-13)
    q = torch.softmax(z.double().masked_fill(~keep, float("-inf")), dim=-1)
    q_tok_lo = q.gather(-1, torch.from_numpy(tok.astype(np.int64))[..., None])[..., 0].numpy()
    up = lambda a: np.kron(a, np.ones((cfg.r, cfg.r), a.dtype))
    assert np.array_equal(got["tok_hi"], up(tok))
    assert np.allclose(got["q_tok"], up(q_tok_lo), rtol=1e-12)
    # a token outside the draft's top-k set has q(x~) = 0 exactly
    low = z.argmin(dim=-1).numpy().astype(np.int32)
    assert np.all(orc.upsample_pool_image(_params(orc, cfg), draft, low)["q_tok"] == 0.0)
    # top-k off: theta = -inf, every entry counts
    off = orc.upsample_pool_image(_params(orc, cfg, top_k=0), draft, tok)
    assert np.all(np.isneginf(off["stats"][..., 0]))
    assert np.allclose(off["stats"][..., 2], torch.exp(z.double() - z.double().max(-1, keepdim=True).values).sum(-1).numpy(),
                       rtol=1e-13)


def _draw_flag(orc, w, u, residual):
    """CDF-edge flag of one draw over weights w: the uniform within EDGE of an edge of the chosen bin of
    the normalised CDF; a residual with next to no mass is always borderline."""
    tok, Zw, gap = orc.inverse_cdf(w, u)
    return tok, Zw, bool(gap < EDGE or (residual and Zw < MIN_RESIDUAL_MASS))


def _expected_flags(orc, cfg, cond, uncond, draft, tok, nn, out, **over):
    P = _params(orc, cfg, **over)
    H, W, r, l = cfg.H, cfg.W, cfg.r, P.radius
    rej = out["reject"].astype(bool)
    t0 = int(np.flatnonzero(rej.ravel())[0]) if rej.any() else H * W
    want = np.zeros((H, W), np.uint32)
    want_tok = np.zeros((H, W), np.int32)
    for i in range(H):
        for j in range(W):
            t = i * W + j
            x = int(tok[i // r, j // r])
            q, p, pp, mass = orc.position_distributions(P, cond[i, j], None if uncond is None else uncond[i, j],
                                                        draft[i // r, j // r], x, nn)
            u = orc.position_uniforms(P.seed, P.image, t, P.round)
            f = 0
            if P.pool_k > 1:
                _, _, _, gap = orc.pool(p, nn[x], P.pool_k, P.pool_delta, x)
                if gap < EDGE:
                    f |= orc.FLAG_POOL_EDGE
            if P.accept_mode == orc.ACCEPT_THRESHOLD:
                if abs(mass - np.float64(np.float32(P.tau))) < EDGE * abs(np.float64(np.float32(P.tau))):
                    f |= orc.FLAG_ACCEPT_EDGE
            elif abs(u[0] - orc.accept_threshold(mass, q[x])) < EDGE:
                f |= orc.FLAG_ACCEPT_EDGE
            # the draw this position would receive
            if P.resample_mode == orc.RESAMPLE_RESIDUAL_ALL:
                use_res = True
            elif P.resample_mode == orc.RESAMPLE_TARGET_ALL:
                use_res = False
            elif P.resample_mode == orc.RESAMPLE_ISOLATED_RESIDUAL:
                win = rej[max(0, i - l):i + l + 1, max(0, j - l):j + l + 1].sum() - int(rej[i, j])
                use_res = bool(rej[i, j]) and (win == 0 or (bool(P.clip_before_first) and t == t0))
            else:
                use_res = bool(rej[i, j])
            if use_res:
                w = orc.residual_weights(pp, q, 1.0)
                x_new, Zw, edge = _draw_flag(orc, w, u[1], True)
                if x_new < 0:      # residual without mass: the target weights, same uniform
                    x_new, Zw, edge = _draw_flag(orc, orc.residual_weights(pp, q, 0.0), u[1], True)
            else:
                x_new, Zw, edge = _draw_flag(orc, orc.residual_weights(pp, q, 0.0), u[2], False)
            if edge:
                f |= orc.FLAG_CDF_EDGE
            want[i, j] = f
            want_tok[i, j] = x_new
    return want, want_tok


@pytest.mark.parametrize("mode", ["MIXED", "RESIDUAL_ALL", "TARGET_ALL", "ISOLATED_RESIDUAL"])
def test_round_flags_follow_from_the_pinned_primitives(orc, mode):
    # few, heavy tokens: bins are wide, so only a handful of positions carry a flag -- scale the
    # logits down and the CDF gets ~V narrow bins; both regimes are run
    for scale, V, pool_k in ((1.0, 96, 12), (0.02, 4096, 1)):
        cfg = dataclasses.replace(SMALL, H=6, W=6, V=V, dtype="f32", top_k=V // 3, sigma=0.6, radius=1, seed=71,
                                  pool_k=pool_k, pool_delta=0.05, resample_mode=getattr(orc, "RESAMPLE_" + mode))
        cond, _, draft, tok = _image(cfg)
        cond, draft = (cond * np.float32(scale)), (draft * np.float32(scale))
        nn = synth.neighbours_to_numpy(synth.codebook_neighbours(V, pool_k, cfg.seed)) if pool_k > 1 else None
        out = orc.round_image(_params(orc, cfg), cond, None, draft, tok, nn)
        want, want_tok = _expected_flags(orc, cfg, cond, None, draft, tok, nn, out)
        assert np.array_equal(out["flags"], want)
        assert np.array_equal(out["cand_tok"], want_tok)
        if V == 4096:      # ~1300 bins of ~1e-3: a 2e-6 window per edge flags a fraction of a percent
            n = int((out["flags"] & orc.FLAG_CDF_EDGE != 0).sum())
            assert n <= 6, n


def test_flags_in_threshold_mode(orc):
    cfg = dataclasses.replace(SMALL, H=4, W=4, V=64, dtype="f32", sigma=0.8, seed=73, accept_mode=orc.ACCEPT_THRESHOLD,
                              resample_mode=orc.RESAMPLE_TARGET_ALL)
    cond, _, draft, tok = _image(cfg)
    base = orc.round_image(_params(orc, cfg, tau=1e-3), cond, None, draft, tok)
    # tau set to a position's own mass, then 5e-7 and 2e-6 (relative) away from it
    P_mass = float(base["accept_prob"][2, 1])
    for rel, expect in ((0.0, True), (5e-7, True), (2e-6, False)):
        tau = np.float32(P_mass * (1.0 + rel))
        out = orc.round_image(_params(orc, cfg, tau=float(tau)), cond, None, draft, tok)
        got = bool(out["flags"][2, 1] & orc.FLAG_ACCEPT_EDGE)
        true_rel = abs(P_mass - np.float64(tau)) / np.float64(tau)
        if abs(true_rel - EDGE) > 2e-7:      # fp32 tau: skip a case that rounding put on the line itself
            assert got == (true_rel < EDGE), (rel, true_rel)
        want, _ = _expected_flags(orc, cfg, cond, None, draft, tok, None, out, tau=float(tau))
        assert np.array_equal(out["flags"], want)


def _logit_for_ratio(target_thr):
    """fp32 logit d such that softmax([d, 0])[0] / 0.5 is as close as fp32 allows to target_thr."""
    p = target_thr / 2.0
    d0 = np.float32(np.log(p / (1.0 - p)))
    best = None
    d = d0
    for _ in range(64):
        d = np.nextafter(d, np.float32(-np.inf))
    for _ in range(129):
        thr = 2.0 / (1.0 + np.exp(-np.float64(d)))
        if best is None or abs(thr - target_thr) < abs(best[1] - target_thr):
            best = (d, thr)
        d = np.nextafter(d, np.float32(np.inf))
    return best


@pytest.mark.parametrize("offset,flagged", [(5e-7, True), (-5e-7, True), (2e-6, False), (-2e-6, False)])
def test_accept_edge_flag_at_a_known_distance(orc, offset, flagged):
    """Two tokens, a flat draft (q = 1/2 each), the target logit chosen so that thr = 2 p(x~) lands
    `offset` above the position's uniform: flagged at 5e-7, not flagged at 2e-6, and the accept bit
    is the sign of the offset."""
    cfg = dataclasses.replace(SMALL, H=2, W=2, V=2, r=1, dtype="f32", sigma=0.0, seed=97, radius=0)
    P = _params(orc, cfg)
    tok = np.zeros((2, 2), np.int32)
    draft = np.zeros((2, 2, 2), np.float32)
    cond = np.zeros((2, 2, 2), np.float32)
    # use a position whose uniform leaves room on both sides
    t = next(t for t in range(4) if 0.2 < orc.position_uniforms(P.seed, P.image, t, P.round)[0] < 0.8)
    u0 = orc.position_uniforms(P.seed, P.image, t, P.round)[0]
    d, thr = _logit_for_ratio(u0 + offset)
    assert abs(thr - (u0 + offset)) < 2e-7
    cond[t // 2, t % 2, 0] = d
    out = orc.round_image(P, cond, None, draft, tok)
    assert out["accept_prob"][t // 2, t % 2] == pytest.approx(thr, abs=1e-15)
    assert bool(out["flags"][t // 2, t % 2] & orc.FLAG_ACCEPT_EDGE) == flagged
    assert out["reject"][t // 2, t % 2] == (0 if offset > 0 else 1)


@pytest.mark.parametrize("offset,flagged", [(5e-7, True), (2e-6, False)])
def test_cdf_edge_flag_at_a_known_distance(orc, offset, flagged):
    """Target-distribution draw over two tokens with p(0) placed `offset` above the draw's uniform:
    token 0 is chosen, and the flag is up exactly when the uniform is within 1e-6 of the bin's edge."""
    cfg = dataclasses.replace(SMALL, H=2, W=2, V=2, r=1, dtype="f32", sigma=0.0, seed=99, radius=0,
                              accept_mode=orc.ACCEPT_THRESHOLD, tau=2.0, resample_mode=orc.RESAMPLE_TARGET_ALL)
    P = _params(orc, cfg)       # tau = 2: everything rejected, every position redrawn from p
    tok = np.zeros((2, 2), np.int32)
    draft = np.zeros((2, 2, 2), np.float32)
    cond = np.zeros((2, 2, 2), np.float32)
    t = next(t for t in range(4) if 0.2 < orc.position_uniforms(P.seed, P.image, t, P.round)[2] < 0.8)
    u2 = orc.position_uniforms(P.seed, P.image, t, P.round)[2]
    d, thr = _logit_for_ratio(2.0 * (u2 + offset))      # p(0) = thr / 2
    cond[t // 2, t % 2, 0] = d
    out = orc.round_image(P, cond, None, draft, tok)
    assert out["out_tok"][t // 2, t % 2] == 0
    assert abs(thr / 2.0 - u2 - offset) < 1e-7
    assert bool(out["flags"][t // 2, t % 2] & orc.FLAG_CDF_EDGE) == flagged
