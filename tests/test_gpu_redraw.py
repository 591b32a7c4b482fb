"""GPU parity of the step-by-step redraw of R_X (Sec. 3.4): the device-side plan (positions sorted by
schedule step) and one launch per step, against the oracle's redraw loop on the same per-step logits."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2601_05149_b200 import binding, synth

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available()
    binding.lib()
    c = binding.Context(0)
    yield c
    c.close()


def _schedule(rng, B, H, W, window, density):
    """R_X masks, their islands and schedule by the ORACLE (the device gets them as inputs)."""
    steps = np.zeros((B, H, W), np.int32)
    for b in range(B):
        seeds = rng.random((H, W)) < density
        rx, _ = orc.expand(seeds.astype(np.uint8), 1, 0)
        labels, _, _, _ = orc.islands(rx)
        steps[b], _ = orc.island_schedule(labels, window)
    return steps


@pytest.mark.parametrize("case", [
    dict(B=2, H=12, W=16, V=512, dtype="bf16", top_k=64, cfg_scale=2.0, temperature=1.0, window=16, density=0.04),
    dict(B=3, H=8, W=8, V=256, dtype="f32", top_k=0, cfg_scale=0.0, temperature=0.7, window=2, density=0.10),
    dict(B=1, H=6, W=40, V=1032, dtype="bf16", top_k=100, cfg_scale=0.0, temperature=1.0, window=4, density=0.5),
], ids=lambda c: f"{c['dtype']}-V{c['V']}-{c['B']}x{c['H']}x{c['W']}-w{c['window']}")
def test_redraw_steps_against_oracle(ctx, case):
    B, H, W, V = case["B"], case["H"], case["W"], case["V"]
    rng = np.random.default_rng(41)
    cfg = synth.RoundConfig("redraw", B=B, H=H, W=W, V=V, r=1, dtype=case["dtype"], top_k=case["top_k"],
                            cfg_scale=case["cfg_scale"], temperature=case["temperature"], seed=4242, round=2)
    steps = _schedule(rng, B, H, W, case["window"], case["density"])
    n_steps = int(steps.max())
    assert n_steps >= 3
    g = torch.Generator(device="cuda").manual_seed(99)
    dt = cfg.torch_dtype
    cond = [(2.0 * torch.randn((B, H, W, V), generator=g, device="cuda")).to(dt) for _ in range(n_steps)]
    unc = [(c.float() + torch.randn((B, H, W, V), generator=g, device="cuda")).to(dt) for c in cond] \
        if cfg.has_uncond else None
    start = torch.from_numpy(rng.integers(0, V, (B, H, W)).astype(np.int32)).cuda()

    p = binding.params_from_config(cfg, image_offset=3)
    max_step = H * W                       # the bound a caller has without reading n_steps back
    guard = pu.Guarded("cuda")
    pos_list = guard.empty("pos_list", (B * H * W,), torch.int32)
    offsets = guard.empty("step_offsets", (2 * (max_step + 2),), torch.int32)
    out = guard.empty("out_tok", (B, H, W), torch.int32)
    out.copy_(start)
    d_steps = torch.from_numpy(steps).cuda()
    n0 = ctx.kernel_launches()
    ctx.mulo_redraw_plan(p, d_steps, max_step, pos_list, offsets)
    for s in range(1, n_steps + 1):
        ctx.mulo_redraw_step(p, s, max_step, pos_list, offsets, cond[s - 1], None if unc is None else unc[s - 1], out)
    torch.cuda.synchronize()
    guard.check()
    assert ctx.kernel_launches() - n0 == 3 + n_steps         # one launch per sequential step

    # the plan: slice s of the list holds exactly the positions of step s
    off = offsets.cpu().numpy()
    lst = pos_list.cpu().numpy()
    flat = steps.ravel()
    for s in range(1, n_steps + 1):
        assert sorted(lst[off[s]:off[s + 1]].tolist()) == np.flatnonzero(flat == s).tolist()
    assert off[n_steps + 1] == (flat > 0).sum() == off[max_step + 1]

    got = out.cpu().numpy()
    differ = flagged = 0
    for b in range(B):
        want, calls, edge = orc.redraw_loop(
            pu.orc_params(cfg, b + 3), steps[b], [synth.to_numpy_logits(c[b]) for c in cond],
            None if unc is None else [synth.to_numpy_logits(u[b]) for u in unc], start[b].cpu().numpy(), with_edge=True)
        assert calls == int(steps[b].max())
        bad = got[b] != want
        assert not (bad & (edge == 0)).any(), np.argwhere(bad & (edge == 0))[:5]
        assert np.array_equal(got[b][steps[b] == 0], start[b].cpu().numpy()[steps[b] == 0])
        differ += int(bad.sum())
        flagged += int(edge.sum())
    n_rx = int((steps > 0).sum())
    print(f"[redraw] {n_rx} positions over {n_steps} steps, flagged {flagged}, differing {differ}")
    assert differ <= max(1, int(1e-3 * n_rx))


def test_redraw_arguments_are_checked(ctx):
    p = binding.make_params(1, 8, 8, 256, 1, binding.F32)
    t = torch.zeros(64, dtype=torch.int32, device="cuda")
    off = torch.zeros(2 * 66, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_redraw_plan(p, t, 0, t, off)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_redraw_plan(p, t, 65, t, off)             # more steps than positions
    assert e.value.status == binding.ERR_INVALID_ARG
    logits = torch.zeros((1, 8, 8, 256), device="cuda")
    for s in (0, 65):
        with pytest.raises(binding.MuloError) as e:
            ctx.mulo_redraw_step(p, s, 64, t, off, logits, None, t)
        assert e.value.status == binding.ERR_INVALID_ARG
