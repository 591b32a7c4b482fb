"""GPU parity on seeded random configurations: shapes, vocabularies, dtypes, top-k, CFG, temperature, accept and
resample modes, radii, pooling, and logits that are scaled, quantised (masses of ties), cubed (near one-hot) or
near-constant.  Every case goes through the C ABI and is compared with the CPU oracle element by element."""
import random

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
    c.close()


def random_config(rng, n):
    r = rng.choice([1, 2, 2, 2, 3, 4])
    h, w = rng.randint(1, 10), rng.randint(1, 16)
    V = rng.choice([1024, 1032, 2048, 4096, 4104, 8192, 16384])
    top_k = rng.choice([0, max(8, V // 64), max(8, V // 16), max(8, V // 8), V // 4, V // 3])
    pool_k = rng.choice([1, 1, 8, 64, 500, 1000])
    return synth.RoundConfig(
        f"rnd{n}", B=rng.randint(1, 2), H=h * r, W=w * r, V=V, r=r, dtype=rng.choice(["bf16", "bf16", "f32"]),
        top_k=top_k, cfg_scale=rng.choice([0.0, 0.0, 1.5, 3.0, 7.5]), temperature=rng.choice([1.0, 1.0, 0.7, 1.3]),
        sigma=rng.choice([0.1, 0.5, 1.0, 2.0]), radius=rng.randint(0, 3), seed=rng.randint(1, 10 ** 6),
        resample_mode=rng.randint(0, 3), clip_before_first=rng.randint(0, 1), accept_mode=rng.choice([0, 0, 0, 1]),
        tau=rng.choice([1e-3, 1e-4, 1e-2]), pool_k=min(pool_k, V), pool_delta=rng.choice([0.01, 0.1, 0.3, 0.9]))


def transform(batch, how, scale, step):
    def f(t):
        if t is None:
            return None
        x = t.float()
        if how == "scale":
            x = x * scale
        elif how == "quant":
            x = torch.round(x * step) / step
        elif how == "cube":
            x = x ** 3
        elif how == "const":
            x = torch.zeros_like(x) + 0.5 * (torch.arange(x.shape[-1], device=x.device) % 7 == 0)
        return x.to(t.dtype).contiguous()
    for key in ("cond", "uncond", "draft_lo"):
        batch[key] = f(batch[key])


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_random_rounds(ctx, seed):
    rng = random.Random(seed)
    fast = 0
    for n in range(40):
        cfg = random_config(rng, n)
        how = rng.choice(["none", "none", "scale", "quant", "cube", "const"])
        scale, step = rng.choice([0.05, 0.2, 4.0]), rng.choice([1.0, 2.0, 4.0])
        batch = pu.build_batch(cfg)
        p = binding.params_from_config(cfg)
        ctx.ensure_workspace(p)
        if how != "none":
            transform(batch, how, scale, step)
            # the draft tokens must have q > 0 under the new logits: redraw them (oracle's sampler)
            pu.redraw_tokens(cfg, batch)
        g = pu.gpu_round(ctx, cfg, batch)
        fast += ctx.round_kernel(p, cfg.has_uncond) != "general"
        o = pu.oracle_images(cfg, batch, list(range(cfg.B)))
        excused = 0
        for b in range(cfg.B):
            e, _ = pu.compare_image(cfg, g, b, o[b], 2e-3 if cfg.dtype == "bf16" else 1e-5)   # unflagged: exact
            excused += e
        if how == "none":   # the budget on excused positions is stated for the workloads' own logits
            total = cfg.B * cfg.H * cfg.W
            assert excused <= max(1, int(1e-4 * total)), (cfg, excused, total)
        assert ctx.poll_device_status() & ~(binding.DEV_DENSE_FALLBACK | binding.DEV_ZERO_DRAFT_PROB) == 0, cfg
    assert fast >= 10


@pytest.mark.parametrize("seed", [5, 6])
def test_random_draft_draws(ctx, seed):
    rng = random.Random(seed)
    for n in range(40):
        cfg = random_config(rng, n)
        cfg = synth.RoundConfig(cfg.name, B=cfg.B, H=cfg.H, W=cfg.W, V=rng.choice([cfg.V, 32768, 65536]), r=cfg.r,
                                dtype=cfg.dtype, top_k=cfg.top_k, temperature=cfg.temperature, seed=cfg.seed,
                                round=rng.randint(0, 5))
        how = rng.choice(["none", "scale", "quant", "cube", "const"])
        batch = pu.build_batch(cfg)
        transform(batch, how, rng.choice([0.05, 0.2, 4.0]), rng.choice([1.0, 2.0, 4.0]))
        off = rng.randint(0, 3)
        p = binding.params_from_config(cfg, image_offset=off)
        ctx.ensure_workspace(p)
        tok = torch.full((cfg.B, cfg.h, cfg.w), -5, dtype=torch.int32, device="cuda")
        ctx.mulo_sample_draft(p, batch["draft_lo"], tok)
        torch.cuda.synchronize()
        tok = tok.cpu().numpy()
        for b in range(cfg.B):
            want, edge = oracle.sample_draft_tokens(pu.orc_params(cfg, b + off),
                                                    synth.to_numpy_logits(batch["draft_lo"][b]), with_edge=True)
            bad = (tok[b] != want) & (edge == 0)
            assert not bad.any(), (cfg, how, np.argwhere(bad)[:4])
        assert ctx.poll_device_status() & ~binding.DEV_DENSE_FALLBACK == 0
