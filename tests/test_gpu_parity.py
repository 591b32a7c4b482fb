"""GPU parity: the CUDA round, called through the C ABI, against the CPU oracle
on the same seeded inputs -- decisions, masks and tokens bit for bit (borderline
uniforms excepted and counted), probabilities within the stated tolerances."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2601_05149_b200 import binding, synth

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available()
    binding.lib()            # raises if the library was not built: no fallback
    c = binding.Context(0)
    c.set_workspace(torch.empty(1 << 16, dtype=torch.uint8, device="cuda"))   # so that status polls work from the start
    yield c
    assert c.poll_device_status() & ~binding.DEV_DENSE_FALLBACK == 0
    c.close()


TINY = synth.RoundConfig("tiny", B=2, H=8, W=8, V=256, dtype="f32", sigma=1.0, radius=1, seed=101)


def _run(ctx, cfg, images=None, **over):
    batch = pu.build_batch(cfg)
    g = pu.gpu_round(ctx, cfg, batch, **over)
    images = list(range(cfg.B)) if images is None else images
    o = pu.oracle_images(cfg, batch, images, **over)
    return batch, g, o


@pytest.mark.parametrize("cfg", [
    TINY,
    dataclasses.replace(TINY, dtype="bf16", seed=102),
    dataclasses.replace(TINY, dtype="bf16", top_k=40, seed=103),
    dataclasses.replace(TINY, dtype="f32", top_k=40, cfg_scale=3.0, temperature=0.7, seed=104),
    dataclasses.replace(TINY, dtype="bf16", top_k=40, cfg_scale=3.0, radius=2, seed=105),
    dataclasses.replace(TINY, V=264, H=6, W=10, r=1, top_k=17, seed=106),          # ragged sizes
    dataclasses.replace(TINY, V=8, H=4, W=4, top_k=3, seed=107),                    # tiny vocabulary
    dataclasses.replace(TINY, H=12, W=36, r=3, radius=3, dtype="bf16", seed=108),   # two mask words per row
    dataclasses.replace(TINY, V=2048, top_k=300, pool_k=128, pool_delta=0.1, dtype="bf16", sigma=2.0, seed=109),
    dataclasses.replace(TINY, V=2048, top_k=0, pool_k=64, pool_delta=0.3, dtype="f32", seed=110),
], ids=lambda c: f"{c.dtype}-V{c.V}-k{c.top_k}-cfg{c.cfg_scale}-pool{c.pool_k}-{c.H}x{c.W}r{c.r}l{c.radius}")
def test_round_small(ctx, cfg):
    batch, g, o = _run(ctx, cfg)
    pu.check_round(cfg, g, o)
    # something was rejected and something was swept in, or the case tests nothing
    assert g["n_reject"].sum() > 0 and g["n_expand"].sum() > g["n_reject"].sum()


@pytest.mark.parametrize("mode", [binding.RESAMPLE_MIXED, binding.RESAMPLE_RESIDUAL_ALL,
                                  binding.RESAMPLE_TARGET_ALL, binding.RESAMPLE_ISOLATED_RESIDUAL])
@pytest.mark.parametrize("clip", [0, 1])
def test_round_modes(ctx, mode, clip):
    cfg = dataclasses.replace(TINY, dtype="bf16", top_k=60, radius=2, seed=120 + mode,
                              resample_mode=mode, clip_before_first=clip)
    batch, g, o = _run(ctx, cfg)
    pu.check_round(cfg, g, o)


@pytest.mark.parametrize("tau", [0.0, 1e-3, 1e-4, 1.5])
def test_round_threshold_rule(ctx, tau):
    """The relaxed rule of Eq. 5 with redraws from the target distribution."""
    cfg = dataclasses.replace(TINY, dtype="bf16", V=2048, top_k=300, pool_k=64, pool_delta=0.1, seed=130,
                              accept_mode=binding.ACCEPT_THRESHOLD, tau=tau,
                              resample_mode=binding.RESAMPLE_TARGET_ALL)
    batch, g, o = _run(ctx, cfg)
    pu.check_round(cfg, g, o)
    if tau == 0.0:
        assert g["n_reject"].sum() == 0
    if tau > 1:
        assert g["reject"].all() and g["expand"].all()


def test_identity_target_equals_draft(ctx):
    cfg = dataclasses.replace(TINY, dtype="bf16", top_k=40, sigma=0.0, seed=140)
    batch, g, o = _run(ctx, cfg)
    assert g["n_reject"].sum() == 0 and g["n_expand"].sum() == 0
    assert np.all(g["accept_prob"] == 1.0)
    assert np.array_equal(g["out_tok"], batch["tok_lo"].cpu().numpy().repeat(2, 1).repeat(2, 2))
    assert np.all(g["first_reject"] == cfg.H * cfg.W)
    pu.check_round(cfg, g, o)


def test_stages_equal_fused(ctx):
    """upsample_pool -> verify -> local_reject_expand -> resample gives exactly
    the fused round of the general path; each stage is also checked against the oracle."""
    import oracle as orc
    for cfg in (dataclasses.replace(TINY, dtype="bf16", top_k=40, cfg_scale=3.0, radius=2, seed=150),
                dataclasses.replace(TINY, V=2048, top_k=300, pool_k=128, dtype="bf16", seed=151,
                                    resample_mode=binding.RESAMPLE_ISOLATED_RESIDUAL)):
        batch = pu.build_batch(cfg)
        # the stages run the general routines: bit for bit the fused round on the general path ...
        ctx.set_general_path_only(True)
        try:
            f = pu.gpu_round(ctx, cfg, batch)
        finally:
            ctx.set_general_path_only(False)
        s = pu.gpu_stages(ctx, cfg, batch)
        for k in ("out_tok", "reject_bits", "expand_bits", "n_reject", "n_expand", "first_reject",
                  "p_tok", "q_tok", "accept_prob"):
            assert np.array_equal(f[k], s[k]), k
        o = pu.oracle_images(cfg, batch, list(range(cfg.B)))
        pu.check_round(cfg, s, o)
        # ... and the fused round as it runs by default (the streaming kernel where it applies) meets
        # the same bar against the oracle
        pu.check_round(cfg, pu.gpu_round(ctx, cfg, batch), o)
        for b in range(cfg.B):
            up = orc.upsample_pool_image(pu.orc_params(cfg, b), synth.to_numpy_logits(batch["draft_lo"][b]),
                                         batch["tok_lo"][b].cpu().numpy())
            assert np.array_equal(s["tok_hi"][b], up["tok_hi"])
            assert np.array_equal(s["stats"][b][..., 0], up["stats"][..., 0].astype(np.float32))
            assert np.array_equal(s["stats"][b][..., 1], up["stats"][..., 1].astype(np.float32))
            Zq = s["stats"][b][..., 2].astype(np.float64) + s["stats"][b][..., 3]
            assert np.allclose(Zq, up["stats"][..., 2], rtol=1e-7)
            assert np.allclose(s["q_tok_hi"][b], up["q_tok"], rtol=2e-6)
            assert np.array_equal(s["q_tok_hi"][b], s["q_tok"][b])


def test_expand_stage_against_oracle(ctx):
    """mulo_local_reject_expand alone on random masks, all radii, clip on/off."""
    import oracle as orc
    rng = np.random.default_rng(7)
    for (H, W) in ((5, 7), (16, 16), (9, 70), (64, 64)):
        for l in (0, 1, 2, 3, 5, 9):
            for clip in (0, 1):
                B = 3
                rej = (rng.random((B, H, W)) < rng.choice([0.0, 0.01, 0.1])).astype(np.uint8)
                Ww = (W + 31) // 32
                padded = np.zeros((B, H, Ww * 32), np.uint8)
                padded[..., :W] = rej
                words = (padded.reshape(B, H, Ww, 32).astype(np.uint64) << np.arange(32, dtype=np.uint64)).sum(-1)
                words = words.astype(np.uint32)
                first = np.array([np.flatnonzero(r.ravel())[0] if r.any() else H * W for r in rej], np.int32)
                p = binding.make_params(B, H, W, 8, 1, binding.F32, radius=l, clip_before_first=clip)
                d_rej = torch.from_numpy(words.view(np.int32)).cuda()
                d_first = torch.from_numpy(first).cuda()
                d_exp = torch.empty_like(d_rej)
                d_n = torch.empty(B, dtype=torch.int32, device="cuda")
                ctx.mulo_local_reject_expand(p, d_rej, d_first, d_exp, d_n)
                got = binding.unpack_bits(d_exp, W).numpy()
                for b in range(B):
                    want, t0 = orc.expand(rej[b], l, clip)
                    assert np.array_equal(got[b], want), (H, W, l, clip, b)
                    assert int(d_n[b]) == want.sum()


def test_config_C1(ctx):
    cfg = synth.CONFIGS["C1"]
    batch, g, o = _run(ctx, cfg)
    pu.check_round(cfg, g, o)


def test_config_C2(ctx):
    cfg = synth.CONFIGS["C2"]
    batch = pu.build_batch(cfg, images=[0])
    g = pu.gpu_round(ctx, cfg, batch)
    o = pu.oracle_images(cfg, batch, [0])
    pu.check_round(cfg, g, o)


def test_config_C3_sampled_images(ctx):
    """Full-size batch on the GPU, first and last image against the oracle."""
    cfg = synth.CONFIGS["C3"]
    batch = pu.build_batch(cfg, images=[0, cfg.B - 1])
    g = pu.gpu_round(ctx, cfg, batch)
    o = pu.oracle_images(cfg, batch, [0, cfg.B - 1])
    pu.check_round(cfg, g, o)


def test_rounds_and_image_offset_change_the_draws(ctx):
    cfg = dataclasses.replace(TINY, dtype="bf16", top_k=40, seed=160)
    batch = pu.build_batch(cfg)
    a = pu.gpu_round(ctx, cfg, batch)
    b = pu.gpu_round(ctx, cfg, batch, round=1)
    assert not np.array_equal(a["reject"], b["reject"])
    # image_offset shifts the Philox image index: image 0 with offset 1 uses image 1's stream
    c = pu.gpu_round(ctx, cfg, batch, image_offset=5)
    o = pu.oracle_images(cfg, batch, [0, 1], image_offset=5)
    pu.check_round(cfg, c, o)
    # a repeated call is bit-identical
    a2 = pu.gpu_round(ctx, cfg, batch)
    for k in a:
        assert np.array_equal(a[k], a2[k])


def test_host_buffer_round(ctx):
    cfg = dataclasses.replace(TINY, dtype="bf16", top_k=40, cfg_scale=3.0, seed=170)
    batch = pu.build_batch(cfg)
    ref = pu.gpu_round(ctx, cfg, batch)
    p = binding.params_from_config(cfg)
    arena = torch.empty(binding.Context.round_host_arena_bytes(p, True), dtype=torch.uint8, device="cuda")
    host = {k: (None if v is None else v.cpu().pin_memory()) for k, v in batch.items()}
    o = binding.alloc_round_outputs(p, "cpu", True)
    c2 = binding.Context(0)
    c2.mulo_round_host(p, arena, host["cond"], host["uncond"], host["draft_lo"], host["tok_lo"], host["nn"],
                       o["out_tok"], o["reject_bits"], o["expand_bits"], o["p_tok"], o["q_tok"],
                       o["accept_prob"], o["n_reject"], o["n_expand"], o["first_reject"])
    for k in ("out_tok", "reject_bits", "expand_bits", "p_tok", "q_tok", "accept_prob", "n_reject",
              "n_expand", "first_reject"):
        assert np.array_equal(o[k].numpy(), ref[k]), k
    c2.close()


def test_device_status_reports_contract_violations(ctx):
    cfg = dataclasses.replace(TINY, dtype="bf16", top_k=4, seed=180)
    batch = pu.build_batch(cfg)
    assert ctx.poll_device_status() & ~binding.DEV_DENSE_FALLBACK == 0
    bad = dict(batch)
    bad["tok_lo"] = batch["tok_lo"].clone()
    bad["tok_lo"][0, 0, 0] = cfg.V + 5                 # outside the vocabulary
    pu.gpu_round(ctx, cfg, bad)
    assert ctx.poll_device_status() & binding.DEV_BAD_TOKEN
    # a token outside the draft top-k has q = 0
    worst = batch["draft_lo"][0, 0, 0].float().argmin().item()
    bad["tok_lo"] = batch["tok_lo"].clone()
    bad["tok_lo"][0, 0, 0] = worst
    pu.gpu_round(ctx, cfg, bad)
    assert ctx.poll_device_status() & binding.DEV_ZERO_DRAFT_PROB
    assert ctx.poll_device_status() & ~binding.DEV_DENSE_FALLBACK == 0      # reading clears


# ------------------------------------------------------------------ fast top-k path

BIG = synth.RoundConfig("big", B=2, H=8, W=8, V=16384, dtype="bf16", sigma=1.0, cfg_scale=3.0,
                        top_k=2000, radius=1, seed=201)


@pytest.mark.parametrize("cfg", [
    BIG,
    dataclasses.replace(BIG, V=4096, top_k=500, cfg_scale=0.0, seed=202),
    dataclasses.replace(BIG, V=8192, top_k=1000, dtype="f32", seed=203),
    dataclasses.replace(BIG, V=8192, top_k=1000, dtype="f32", cfg_scale=0.0, temperature=0.8, seed=204),
    dataclasses.replace(BIG, V=5000, top_k=600, seed=205),                         # ragged last chunk
    dataclasses.replace(BIG, V=65536, top_k=2000, cfg_scale=0.0, H=4, W=4, seed=206),   # largest vocabulary
    dataclasses.replace(BIG, V=2048, top_k=64, seed=207),                          # small k
    dataclasses.replace(BIG, V=4096, top_k=400, B=2, H=32, W=32, radius=2, seed=208),  # several parents per CTA
    dataclasses.replace(BIG, V=4096, top_k=500, r=1, H=6, W=6, seed=209),          # r = 1
    dataclasses.replace(BIG, V=4096, top_k=500, r=4, H=8, W=8, seed=210),          # r = 4 (16 children)
    dataclasses.replace(BIG, resample_mode=binding.RESAMPLE_ISOLATED_RESIDUAL, radius=2, seed=211),
    dataclasses.replace(BIG, resample_mode=binding.RESAMPLE_RESIDUAL_ALL, seed=212),
    dataclasses.replace(BIG, resample_mode=binding.RESAMPLE_TARGET_ALL, accept_mode=binding.ACCEPT_THRESHOLD,
                        tau=1e-4, seed=213),
], ids=lambda c: f"{c.dtype}-V{c.V}-k{c.top_k}-cfg{c.cfg_scale}-{c.B}x{c.H}x{c.W}r{c.r}-m{c.resample_mode}")
def test_round_fast_path(ctx, cfg):
    batch = pu.build_batch(cfg)
    assert ctx.poll_device_status() == 0
    g = pu.gpu_round(ctx, cfg, batch)
    # Gaussian rows: the pivot prediction must hold, no row may have left the fast path
    assert ctx.poll_device_status() == 0
    o = pu.oracle_images(cfg, batch, list(range(cfg.B)))
    pu.check_round(cfg, g, o)
    # and the general kernel gives the same decisions and tokens
    ctx.set_general_path_only(True)
    try:
        d = pu.gpu_round(ctx, cfg, batch)
    finally:
        ctx.set_general_path_only(False)
    pu.check_round(cfg, d, o)
    same = (g["out_tok"] == d["out_tok"]).mean()
    assert same > 0.999 and np.array_equal(g["reject_bits"], d["reject_bits"])


def test_fast_path_falls_back_on_rows_it_cannot_predict(ctx):
    """Rows of ties (all logits equal, or two values) defeat the pivot prediction;
    those rows must be redone by the general routines with identical results."""
    cfg = dataclasses.replace(BIG, V=4096, top_k=500, H=4, W=4, B=2, seed=220)
    batch = pu.build_batch(cfg)
    batch["draft_lo"][0, 0, 0] = 1.0                     # a constant draft row: top-k keeps everything
    batch["cond"][0, 0, 1] = 0.5                         # a constant target row
    batch["uncond"][0, 0, 1] = 0.25
    batch["cond"][1, 2, 2, ::2] = 3.0                    # two-valued target row
    batch["tok_lo"][0, 0, 0] = 17
    ctx.poll_device_status()
    g = pu.gpu_round(ctx, cfg, batch)
    st = ctx.poll_device_status()
    assert st & binding.DEV_DENSE_FALLBACK and not st & ~binding.DEV_DENSE_FALLBACK
    o = pu.oracle_images(cfg, batch, [0, 1])
    pu.check_round(cfg, g, o)


def test_identity_fast_path(ctx):
    cfg = dataclasses.replace(BIG, cfg_scale=0.0, sigma=0.0, seed=230)
    batch = pu.build_batch(cfg)
    g = pu.gpu_round(ctx, cfg, batch)
    assert ctx.poll_device_status() == 0
    # the two partition sums are added up in an order that depends on each row's own pivot, so
    # p / q may miss 1 by a rounding error of the fp32 segment sums
    assert g["n_reject"].sum() == 0 and np.all(np.abs(g["accept_prob"] - 1.0) <= 1e-6)
    assert np.array_equal(g["out_tok"], batch["tok_lo"].cpu().numpy().repeat(2, 1).repeat(2, 2))


def test_config_C4_sampled_images(ctx):
    """The benchmark's workload in its launch configuration (B = 32 on the device),
    first and last image against the oracle, radii 1..3."""
    cfg = synth.CONFIGS["C4"]
    batch = pu.build_batch(cfg, images=[0, cfg.B - 1])
    for radius in (3, 1, 2):
        c = dataclasses.replace(cfg, radius=radius)
        ctx.poll_fallback_counts()
        g = pu.gpu_round(ctx, c, batch, probs=(radius == 3))
        assert ctx.poll_device_status() == 0
        assert ctx.poll_fallback_counts()[0] == 0      # no row left the fast path
        if radius == 3:
            o = pu.oracle_images(c, batch, [0, cfg.B - 1])
        else:   # only the masks and the choice of draw depend on the radius
            o = pu.oracle_images(c, batch, [cfg.B - 1])
        pu.check_round(c, g, o)


def _sweep_picks():
    """Twelve points of the throughput sweep at its largest batch: every (grid, vocabulary) pair twice,
    every noise level three times."""
    pts = synth.sweep_points()
    picks = []
    for pair in range(6):               # (grid, V) pairs in the sweep's own order
        for s in ((2 * pair) % 4, (2 * pair + 1) % 4):
            picks.append((pair * 4 + 3) * 4 + s)     # batch index 3: B = 64
    return [pts[i] for i in picks]


@pytest.mark.parametrize("cfg", _sweep_picks(), ids=lambda c: f"{c.H}x{c.W}-V{c.V}-B{c.B}-s{c.sigma}")
def test_sweep_points_at_launch_size(ctx, cfg):
    """Points of the throughput sweep in the configuration the sweep times (B = 64 on the device): the
    first four images and the last against the oracle, no row redone by the general kernel."""
    assert cfg.B == 64
    batch = pu.build_batch(cfg, images=[0, 1, 2, 3, cfg.B - 1])
    ctx.poll_fallback_counts()
    g = pu.gpu_round(ctx, cfg, batch)
    counts = ctx.poll_fallback_counts()      # rows redone, then by reason: list full, too few, above range, crowded bin
    assert counts[0] == 0, counts
    assert ctx.poll_device_status() == 0
    o = pu.oracle_images(cfg, batch, [0, 1, 2, 3, cfg.B - 1])
    pu.check_round(cfg, g, o)


def test_fast_path_adapts_to_rows_that_are_not_normal(ctx):
    """Heavy-tailed logits (cubed normals) defeat the normal-shaped first guess of the pivot; the guess
    must adapt within a few rows, the rows it loses go to the general routines, results stay exact."""
    cfg = dataclasses.replace(BIG, V=4096, top_k=500, B=8, H=64, W=64, seed=240)
    batch = pu.build_batch(cfg)
    for k in ("cond", "uncond", "draft_lo"):
        x = batch[k].float()
        batch[k] = (x * x * x / 8.0).to(batch[k].dtype).contiguous()
    # draft tokens must have draft probability > 0 under the new logits: take each row's maximum
    batch["tok_lo"] = batch["draft_lo"].float().argmax(-1).to(torch.int32).contiguous()
    ctx.poll_device_status()
    ctx.poll_fallback_counts()
    g = pu.gpu_round(ctx, cfg, batch)
    assert ctx.poll_device_status() & ~binding.DEV_DENSE_FALLBACK == 0
    lost = ctx.poll_fallback_counts()[0]
    rows = cfg.B * cfg.H * cfg.W
    assert lost < 0.6 * rows, (lost, rows)      # every CTA loses its first few parents while it adapts
    o = pu.oracle_images(cfg, batch, [0, cfg.B - 1])
    pu.check_round(cfg, g, o)


@pytest.mark.parametrize("fast", [True, False])
def test_residual_for_all_with_near_one_hot_rows(ctx, fast):
    """Cubed logits make target and draft near one-hot; drawing EVERY position of R_X from the residual then
    asks, at accepted positions, for a draw from max(0, p - q) with next to no mass.  In fp32 that residual is
    empty (the draw falls back to the target weights), in fp64 it is rounding dust: the oracle flags such
    draws (edge test in units of probability mass), and the outputs may differ only there.  No budget on how
    many: the case is ill-posed by construction."""
    cfg = synth.RoundConfig("onehot", B=2, H=8, W=24, V=4096, r=2, dtype="bf16", top_k=64, cfg_scale=7.5,
                            sigma=2.0, radius=2, resample_mode=binding.RESAMPLE_RESIDUAL_ALL, seed=219012)
    batch = pu.build_batch(cfg)
    for k in ("cond", "uncond", "draft_lo"):
        batch[k] = (batch[k].float() ** 3).to(batch[k].dtype).contiguous()
    batch["tok_lo"] = batch["draft_lo"].float().argmax(-1).to(torch.int32).contiguous()
    ctx.set_general_path_only(not fast)
    try:
        g = pu.gpu_round(ctx, cfg, batch)
    finally:
        ctx.set_general_path_only(False)
    o = pu.oracle_images(cfg, batch, list(range(cfg.B)))
    differ = flagged = 0
    for b in range(cfg.B):
        e, f = pu.compare_image(cfg, g, b, o[b], 2e-3)     # raises where an unflagged position differs
        differ += e
        flagged += f
    assert flagged > 0


@pytest.mark.parametrize("scale,pool_k,delta", [(4.0, 2048, 0.01), (1.0, 1000, 0.1), (0.2, 500, 0.3)])
def test_pooling_on_the_streaming_path(ctx, scale, pool_k, delta):
    """Eq. 3-4 inside the streaming kernel (top-k on, V <= 16384).  With logits scaled up the row is peaked:
    the pooled prefix then adds masses of 1e-19 before an entry of 0.7, which the prefix sums must keep."""
    cfg = synth.RoundConfig("poolfast", B=2, H=8, W=12, V=4096, r=2, dtype="bf16", top_k=1024, cfg_scale=7.5,
                            sigma=1.0, radius=1, clip_before_first=0, pool_k=pool_k, pool_delta=delta,
                            resample_mode=binding.RESAMPLE_ISOLATED_RESIDUAL, seed=305057)
    batch = pu.build_batch(cfg)
    for k in ("cond", "uncond", "draft_lo"):
        batch[k] = (batch[k].float() * scale).to(batch[k].dtype).contiguous()
    pu.redraw_tokens(cfg, batch)                                      # draft tokens with q > 0 under the new logits
    n0 = ctx.kernel_launches()
    g = pu.gpu_round(ctx, cfg, batch)
    assert ctx.kernel_launches() - n0 == 3                            # streaming kernel, its list, the mask kernel
    o = pu.oracle_images(cfg, batch, list(range(cfg.B)))
    pu.check_round(cfg, g, o)
    pooled = sum(int((o[b]["accept_prob"] > o[b]["p_tok"] / np.maximum(o[b]["q_tok"], 1e-300) * (1 + 1e-9)).sum())
                 for b in range(cfg.B))
    assert pooled > 0                                                 # some position did gain pooled mass


def test_round_replays_from_a_cuda_graph(ctx):
    """The calls only enqueue work on the given stream, so a round can be captured once and replayed."""
    cfg = dataclasses.replace(synth.CONFIGS["C3"], name="graph", B=2, H=8, W=8, V=2048, top_k=250, radius=2,
                              sigma=1.0, seed=77)
    batch = pu.build_batch(cfg)
    p = binding.params_from_config(cfg)
    ctx.ensure_workspace(p)
    direct = binding.alloc_round_outputs(p, "cuda", probs=True)
    replay = binding.alloc_round_outputs(p, "cuda", probs=True)

    def call(o):
        ctx.mulo_round(p, batch["cond"], batch["uncond"], batch["draft_lo"], batch["tok_lo"], batch["nn"],
                       o["out_tok"], o["reject_bits"], o["expand_bits"], o["p_tok"], o["q_tok"], o["accept_prob"],
                       o["n_reject"], o["n_expand"], o["first_reject"])
    call(direct)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call(replay)                       # warm-up on the side stream, as graph capture wants
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call(replay)
    for v in replay.values():
        v.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for k in direct:
        assert torch.equal(direct[k], replay[k]), k
    assert int(direct["n_reject"].sum()) > 0


@pytest.mark.parametrize("fast", [True, False], ids=["fast-path", "general-path"])
def test_draft_token_without_draft_mass(ctx, fast):
    """q(x~) = 0: the drafter's token lies outside the draft row's own top-k set at a few cells (a
    contract violation the round must survive).  Eq. 1 then accepts iff p(x~) > 0; decisions, masks
    and tokens follow the oracle on both kernels, and the status bit is raised."""
    cfg = dataclasses.replace(BIG, V=4096, top_k=500, H=16, W=16, radius=2, seed=260)
    batch = pu.build_batch(cfg)
    tok = batch["tok_lo"].clone()
    cells = [(0, 0, 0), (0, 3, 5), (1, 7, 7), (1, 2, 0)]
    order = batch["draft_lo"].float().argsort(-1)
    for n, (b, i, j) in enumerate(cells):
        # the draft row's least likely id, and (last two cells) one just outside its top-k set
        tok[b, i, j] = order[b, i, j, 0] if n < 2 else order[b, i, j, cfg.V - cfg.top_k - 1 - n]
    batch["tok_lo"] = tok.contiguous()
    ctx.poll_device_status()
    ctx.set_general_path_only(not fast)
    try:
        n0 = ctx.kernel_launches()
        g = pu.gpu_round(ctx, cfg, batch)
        assert (ctx.kernel_launches() - n0 == 3) == fast
    finally:
        ctx.set_general_path_only(False)
    status = ctx.poll_device_status()
    assert status & binding.DEV_ZERO_DRAFT_PROB and status & ~(binding.DEV_ZERO_DRAFT_PROB | binding.DEV_DENSE_FALLBACK) == 0
    o = pu.oracle_images(cfg, batch, list(range(cfg.B)))
    pu.check_round(cfg, g, o)
    for (b, i, j) in cells:
        for di in range(cfg.r):
            for dj in range(cfg.r):
                y, x = i * cfg.r + di, j * cfg.r + dj
                assert g["q_tok"][b, y, x] == 0.0 and o[b]["q_tok"][y, x] == 0.0
                # accepted iff the target gives the token any mass; the threshold is then 1 or 0
                assert g["accept_prob"][b, y, x] == (1.0 if o[b]["p_tok"][y, x] > 0 else 0.0)
                assert g["reject"][b, y, x] == (0 if o[b]["p_tok"][y, x] > 0 else 1)


@pytest.mark.parametrize("name", ["C4", "C2x8", "P4x4"])
def test_round_is_bit_reproducible_at_launch_size(ctx, name):
    """The benchmark's workload (B = 32) on the lane kernel, a pooled top-k workload on the streaming
    kernel and the paper-default workload on the resident-row kernel: the same call twice, and once
    more from another stream, gives every output array bit for bit -- decisions depend on (seed,
    image, position, round) and the inputs only, not on how CTAs were scheduled."""
    cfg = {"C4": synth.CONFIGS["C4"], "C2x8": dataclasses.replace(synth.CONFIGS["C2"], B=8),
           "P4x4": dataclasses.replace(synth.CONFIGS["P4"], B=4)}[name]
    assert ctx.round_kernel(binding.params_from_config(cfg), cfg.has_uncond) == \
        {"C4": "lane", "C2x8": "stream", "P4x4": "full"}[name]
    batch = pu.build_batch(cfg, images=[])      # nothing here goes to the oracle
    p = binding.params_from_config(cfg)
    ctx.ensure_workspace(p)

    def run(stream):
        o, guard = pu.round_outputs(p, "cuda", True)
        ctx.mulo_round(p, batch["cond"], batch["uncond"], batch["draft_lo"], batch["tok_lo"], batch["nn"],
                       o["out_tok"], o["reject_bits"], o["expand_bits"], o["p_tok"], o["q_tok"], o["accept_prob"],
                       o["n_reject"], o["n_expand"], o["first_reject"], stream=stream)
        torch.cuda.synchronize()
        guard.check()
        return {k: v.cpu().numpy() for k, v in o.items()}

    first = run(None)
    second = run(None)
    side = torch.cuda.Stream()
    third = run(side)
    for k in first:
        assert first[k].tobytes() == second[k].tobytes(), k
        assert first[k].tobytes() == third[k].tobytes(), k
    assert ctx.poll_device_status() & ~binding.DEV_DENSE_FALLBACK == 0


# ------------------------------------------------------------------ rows without a top-k cut

@pytest.mark.parametrize("tau", [1e-3, 1e-4, 5e-5, 1e-5])
@pytest.mark.parametrize("accept_mode", [binding.ACCEPT_THRESHOLD, binding.ACCEPT_RATIO], ids=["eq5", "eq1"])
def test_paper_default_sampling(ctx, tau, accept_mode):
    """The paper's default sampling on the benchmark's shapes: no top-k cut, CFG 4.0, pooling over the
    1000 nearest codebook entries with delta = 0.1, l = 3; Eq. 5 (redraws from the target distribution)
    for four thresholds, and Eq. 1 with the same pooling (residual redraws at rejections).  64x64 at
    B = 2, both images against the oracle; the rows run on the resident-row kernel."""
    if accept_mode == binding.ACCEPT_RATIO and tau != 1e-3:
        pytest.skip("tau does not enter Eq. 1")
    cfg = dataclasses.replace(synth.CONFIGS["P4"], name=f"P4-{tau}", B=2, tau=tau, accept_mode=accept_mode,
                              resample_mode=binding.RESAMPLE_TARGET_ALL if accept_mode == binding.ACCEPT_THRESHOLD
                              else binding.RESAMPLE_MIXED)
    p = binding.params_from_config(cfg)
    assert ctx.round_kernel(p, True) == "full"
    batch = pu.build_batch(cfg)
    n0 = ctx.kernel_launches()
    g = pu.gpu_round(ctx, cfg, batch)
    assert ctx.kernel_launches() - n0 == 2          # the row kernel and the mask kernel: nothing was redone
    assert ctx.poll_device_status() == 0
    o = pu.oracle_images(cfg, batch, [0, 1])
    pu.check_round(cfg, g, o)
    assert g["n_reject"].sum() > 0


@pytest.mark.parametrize("cfg", [
    dataclasses.replace(BIG, top_k=0, V=4096, dtype="f32", cfg_scale=0.0, seed=270),
    dataclasses.replace(BIG, top_k=0, V=2048, seed=271),
    dataclasses.replace(BIG, top_k=0, V=6144, temperature=0.8, seed=272),                    # three pieces per thread
    dataclasses.replace(BIG, top_k=0, V=8192, pool_k=64, pool_delta=0.3, seed=273),
    dataclasses.replace(BIG, top_k=0, V=4096, pool_k=500, pool_delta=0.9, cfg_scale=0.0, seed=274),   # several list tiles
    dataclasses.replace(BIG, top_k=0, V=4096, r=1, H=6, W=6, seed=275),
    dataclasses.replace(BIG, top_k=0, V=4096, r=3, H=9, W=9, seed=276),
    dataclasses.replace(BIG, top_k=0, V=4096, resample_mode=binding.RESAMPLE_RESIDUAL_ALL, seed=277),
    dataclasses.replace(BIG, top_k=0, V=4096, resample_mode=binding.RESAMPLE_ISOLATED_RESIDUAL, radius=2, seed=278),
    dataclasses.replace(BIG, top_k=0, V=4096, accept_mode=binding.ACCEPT_THRESHOLD, tau=1e-3, seed=279),  # residual draws under Eq. 5
], ids=lambda c: f"{c.dtype}-V{c.V}-cfg{c.cfg_scale}-pool{c.pool_k}-r{c.r}-m{c.resample_mode}-a{c.accept_mode}")
def test_round_resident_rows(ctx, cfg):
    batch = pu.build_batch(cfg)
    assert ctx.round_kernel(binding.params_from_config(cfg), cfg.has_uncond) == "full"
    n0 = ctx.kernel_launches()
    g = pu.gpu_round(ctx, cfg, batch)
    assert ctx.kernel_launches() - n0 == 2
    assert ctx.poll_device_status() == 0
    o = pu.oracle_images(cfg, batch, list(range(cfg.B)))
    pu.check_round(cfg, g, o)
    # the general routines give the same decisions and tokens wherever the oracle did not flag the position
    ctx.set_general_path_only(True)
    try:
        d = pu.gpu_round(ctx, cfg, batch)
    finally:
        ctx.set_general_path_only(False)
    pu.check_round(cfg, d, o)
