"""GPU parity, through the C ABI, of the drafter's own sampling on given logits (Sec. 3.2 Step 1)
and of the majority down-sampler that stands in for D_r (Step 7)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2601_05149_b200 import binding, synth

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available()
    binding.lib()            # raises if the library was not built: no fallback
    c = binding.Context(0)
    c.set_workspace(torch.empty(1 << 16, dtype=torch.uint8, device="cuda"))
    yield c
    assert c.poll_device_status() & ~binding.DEV_DENSE_FALLBACK == 0
    c.close()


TINY = synth.RoundConfig("tiny", B=3, H=8, W=8, V=256, dtype="f32", sigma=1.0, radius=1, seed=301)


def sample_both(ctx, cfg, images=None, image_offset=0, rnd=0):
    batch = pu.build_batch(cfg)
    p = binding.params_from_config(cfg, image_offset=image_offset, round=rnd)
    tok = torch.full((cfg.B, cfg.h, cfg.w), -5, dtype=torch.int32, device="cuda")
    ctx.mulo_sample_draft(p, batch["draft_lo"], tok)
    torch.cuda.synchronize()
    tok = tok.cpu().numpy()
    images = range(cfg.B) if images is None else images
    excused = total = 0
    for b in images:
        want, edge = oracle.sample_draft_tokens(pu.orc_params(cfg, b + image_offset, round=rnd),
                                                synth.to_numpy_logits(batch["draft_lo"][b]), with_edge=True)
        differ = tok[b] != want
        assert not (differ & (edge == 0)).any(), (b, np.argwhere(differ & (edge == 0))[:5])
        excused += int(differ.sum())
        total += want.size
        assert (tok[b] >= 0).all() and (tok[b] < cfg.V).all()
    assert excused <= max(1, total // 1000)
    return tok


@pytest.mark.parametrize("cfg", [
    TINY,
    dataclasses.replace(TINY, dtype="bf16", seed=302),
    dataclasses.replace(TINY, dtype="bf16", top_k=40, temperature=0.7, seed=303),
    dataclasses.replace(TINY, V=264, H=6, W=10, r=1, top_k=17, seed=304),
    dataclasses.replace(TINY, V=8, H=4, W=4, top_k=3, seed=305),
    dataclasses.replace(TINY, B=1, V=16384, dtype="bf16", top_k=2000, seed=306),
    dataclasses.replace(TINY, B=1, V=65536, dtype="f32", top_k=0, seed=307),
], ids=lambda c: f"{c.dtype}-V{c.V}-k{c.top_k}-{c.H}x{c.W}r{c.r}")
def test_sample_draft_small(ctx, cfg):
    sample_both(ctx, cfg)


@pytest.mark.parametrize("cfg", [
    dataclasses.replace(TINY, B=2, H=16, W=16, V=16384, dtype="bf16", top_k=2000, seed=330),
    dataclasses.replace(TINY, B=2, H=16, W=16, V=4096, dtype="f32", top_k=500, temperature=0.8, seed=331),
    dataclasses.replace(TINY, B=1, H=8, W=8, V=4104, dtype="bf16", top_k=300, seed=332),     # ragged last chunk
    dataclasses.replace(TINY, B=1, H=8, W=8, V=65536, dtype="bf16", top_k=4000, seed=333),   # sixteen chunks per row
], ids=lambda c: f"{c.dtype}-V{c.V}-k{c.top_k}")
def test_sample_draft_fast_path(ctx, cfg):
    """Top-k on and V >= 1024: the streaming kernel in its sampling mode (two launches), same parity bar;
    switched off, the general kernel (one launch) meets it too."""
    ctx.ensure_workspace(binding.params_from_config(cfg))
    n0 = ctx.kernel_launches()
    sample_both(ctx, cfg)
    assert ctx.kernel_launches() - n0 == 2
    lost = ctx.poll_fallback_counts()[0]
    assert lost <= cfg.B * cfg.h * cfg.w // 4
    ctx.set_general_path_only(True)
    try:
        n0 = ctx.kernel_launches()
        sample_both(ctx, cfg)
        assert ctx.kernel_launches() - n0 == 1
    finally:
        ctx.set_general_path_only(False)


def test_sample_draft_fast_path_rows_that_are_not_normal(ctx):
    """Heavy-tailed rows defeat the pivot prediction now and then: those cells go through the list."""
    cfg = dataclasses.replace(TINY, B=2, H=32, W=32, V=4096, dtype="f32", top_k=400, seed=334)
    batch = pu.build_batch(cfg)
    batch["draft_lo"] = (batch["draft_lo"] ** 3).contiguous()
    p = binding.params_from_config(cfg)
    ctx.ensure_workspace(p)
    tok = torch.full((cfg.B, cfg.h, cfg.w), -5, dtype=torch.int32, device="cuda")
    ctx.mulo_sample_draft(p, batch["draft_lo"], tok)
    torch.cuda.synchronize()
    tok = tok.cpu().numpy()
    differ = 0
    for b in range(cfg.B):
        want, edge = oracle.sample_draft_tokens(pu.orc_params(cfg, b), synth.to_numpy_logits(batch["draft_lo"][b]),
                                                with_edge=True)
        bad = (tok[b] != want) & (edge == 0)
        assert not bad.any(), (b, np.argwhere(bad)[:5])
        differ += int((tok[b] != want).sum())
    assert differ <= 2


def test_sample_draft_streams(ctx):
    """Different rounds and image offsets draw different tokens; the same ones repeat exactly."""
    cfg = dataclasses.replace(TINY, B=2, dtype="bf16", top_k=40, seed=310)
    a = sample_both(ctx, cfg, rnd=0)
    b = sample_both(ctx, cfg, rnd=1)
    c = sample_both(ctx, cfg, rnd=0, image_offset=5)
    again = sample_both(ctx, cfg, rnd=0)
    np.testing.assert_array_equal(a, again)
    assert (a != b).any() and (a != c).any()


def test_sample_draft_full_size_sampled_images(ctx):
    cfg = dataclasses.replace(synth.CONFIGS["C4"], B=4, seed=311)
    sample_both(ctx, cfg, images=[0, 3])


def downsample_both(ctx, x, r):
    B, H, W = x.shape
    p = binding.make_params(B, H, W, 8, r, binding.F32)
    y = torch.full((B, H // r, W // r), -5, dtype=torch.int32, device="cuda")
    ctx.mulo_downsample(p, torch.from_numpy(x).cuda(), y)
    torch.cuda.synchronize()
    y = y.cpu().numpy()
    for b in range(B):
        np.testing.assert_array_equal(y[b], oracle.downsample_majority(x[b], r))
    return y


@pytest.mark.parametrize("r", [1, 2, 3, 4])
@pytest.mark.parametrize("alphabet", [3, 50000])
def test_downsample_random_tokens(ctx, r, alphabet):
    rng = np.random.default_rng(r * 7 + alphabet)
    x = rng.integers(0, alphabet, (3, 5 * r, 9 * r)).astype(np.int32)
    downsample_both(ctx, x, r)


def test_downsample_undoes_replication_and_follows_a_round(ctx):
    cfg = synth.RoundConfig("ds", B=3, H=16, W=24, V=512, r=2, dtype="bf16", top_k=64, sigma=0.15, radius=1,
                            seed=320)
    batch = pu.build_batch(cfg)
    g = pu.gpu_round(ctx, cfg, batch)
    tok_lo = batch["tok_lo"].cpu().numpy()
    up = np.repeat(np.repeat(tok_lo, cfg.r, axis=1), cfg.r, axis=2).astype(np.int32)
    np.testing.assert_array_equal(downsample_both(ctx, up, cfg.r), tok_lo)
    y = downsample_both(ctx, g["out_tok"].astype(np.int32), cfg.r)
    untouched = g["expand"].reshape(cfg.B, cfg.h, cfg.r, cfg.w, cfg.r).sum(axis=(2, 4)) == 0
    assert untouched.any()
    np.testing.assert_array_equal(y[untouched], tok_lo[untouched])   # blocks outside R_X keep the draft token


def test_limits_are_refused_before_launch(ctx):
    p = binding.make_params(1, 8, 8, 8, 2, binding.F32)
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_sample_draft(p, None, torch.zeros((1, 4, 4), dtype=torch.int32, device="cuda"))
    assert e.value.status == binding.ERR_INVALID_ARG
    p = binding.make_params(1, 34, 34, 8, 17, binding.F32)
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_downsample(p, torch.zeros((1, 34, 34), dtype=torch.int32, device="cuda"),
                            torch.zeros((1, 2, 2), dtype=torch.int32, device="cuda"))
    assert e.value.status == binding.ERR_UNSUPPORTED
