"""GPU parity of the rejection islands (Sec. 3.4, Eq. 8) through the C ABI: labels, island
count and the per-island tables bit for bit against the CPU oracle."""
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
    yield c
    c.close()


def pack_bits(mask):
    """[B, H, W] 0/1 -> [B, H, ceil(W/32)] uint32, bit j % 32 of word j / 32."""
    B, H, W = mask.shape
    Ww = (W + 31) // 32
    padded = np.zeros((B, H, Ww * 32), np.uint64)
    padded[:, :, :W] = mask
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (padded.reshape(B, H, Ww, 32) * weights).sum(-1).astype(np.uint32)


def run_islands(ctx, mask, max_islands):
    B, H, W = mask.shape
    p = binding.make_params(B, H, W, 8, 1, binding.F32)
    bits = torch.from_numpy(pack_bits(mask).view(np.int32)).cuda()
    labels = torch.full((B, H, W), -7, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    rows = torch.full((B, max(max_islands, 1), 2), -7, dtype=torch.int32, device="cuda")
    size = torch.full((B, max(max_islands, 1)), -7, dtype=torch.int32, device="cuda")
    ctx.mulo_islands(p, bits, labels, n, rows if max_islands else None, size if max_islands else None,
                     max_islands=max_islands)
    torch.cuda.synchronize()
    return labels.cpu().numpy(), n.cpu().numpy(), rows.cpu().numpy(), size.cpu().numpy()


def check_against_oracle(ctx, mask, max_islands):
    labels, n, rows, size = run_islands(ctx, mask, max_islands)
    for b in range(mask.shape[0]):
        o_labels, M, o_rows, o_size = oracle.islands(mask[b])
        assert n[b] == M
        np.testing.assert_array_equal(labels[b], o_labels)
        k = min(M, max_islands)
        np.testing.assert_array_equal(rows[b, :k], o_rows[:k])
        np.testing.assert_array_equal(size[b, :k], o_size[:k])
        if max_islands:
            assert (rows[b, k:max_islands] == -1).all() and (size[b, k:max_islands] == 0).all()


@pytest.mark.parametrize("shape", [(3, 1, 1), (2, 1, 40), (2, 9, 1), (4, 8, 8), (3, 17, 33), (8, 64, 64),
                                   (2, 40, 70), (2, 128, 128), (1, 16, 1024)])
@pytest.mark.parametrize("density", [0.03, 0.3, 0.5])
def test_random_masks(ctx, shape, density):
    rng = np.random.default_rng(shape[1] * 1000 + shape[2] + int(density * 100))
    mask = (rng.random(shape) < density).astype(np.uint8)
    check_against_oracle(ctx, mask, max_islands=shape[1] * shape[2])


def test_shapes_with_long_chains_and_late_merges(ctx):
    H = W = 64
    m = np.zeros((6, H, W), np.uint8)
    m[0] = np.fliplr(np.eye(H, dtype=np.uint8))                      # anti-diagonal: one island
    m[1] = (np.add.outer(np.arange(H), np.arange(W)) % 2 == 0)       # checkerboard: one island
    m[2, ::2, ::2] = 1                                               # 1024 single positions
    m[3, :, 0] = m[3, :, W - 1] = m[3, H - 1, :] = 1                 # "U": the arms meet in the last row
    for i in range(0, H, 4):                                         # a serpentine: one long chain
        m[4, i, :] = 1
        m[4, i + 1: i + 4, (W - 1) if (i // 4) % 2 == 0 else 0] = 1
    m[5, ::2, :] = 1                                                 # 32 stripes
    labels, n, rows, size = run_islands(ctx, m, H * W)
    assert list(n) == [1, 1, (H // 2) * (W // 2), 1, 1, H // 2]
    check_against_oracle(ctx, m, max_islands=H * W)


def test_empty_full_and_small_tables(ctx):
    m = np.zeros((3, 12, 36), np.uint8)
    m[1] = 1
    m[2, ::2, ::2] = 1
    check_against_oracle(ctx, m, max_islands=16)   # image 2 has 108 islands: the tables hold the first 16
    check_against_oracle(ctx, m, max_islands=0)    # no tables at all
    labels, n, _, _ = run_islands(ctx, m, 0)
    assert list(n) == [0, 1, 108] and labels[0].max() == 0 and (labels[1] == 1).all()


def test_islands_of_a_real_round(ctx):
    cfg = synth.RoundConfig("islands", B=4, H=32, W=32, V=512, dtype="bf16", top_k=64, sigma=1.0, radius=1,
                            seed=4242)
    batch = pu.build_batch(cfg)
    g = pu.gpu_round(ctx, cfg, batch)
    mask = g["expand"].astype(np.uint8)
    assert 0 < mask.sum() < mask.size
    check_against_oracle(ctx, mask, max_islands=256)


def schedule_both(ctx, mask, window):
    B, H, W = mask.shape
    p = binding.make_params(B, H, W, 8, 1, binding.F32)
    labels, _, _, _ = run_islands(ctx, mask, 0)
    step = torch.full((B, H, W), -7, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ctx.mulo_island_schedule(p, torch.from_numpy(labels).cuda(), window, step, n)
    torch.cuda.synchronize()
    step, n = step.cpu().numpy(), n.cpu().numpy()
    for b in range(B):
        want, nfe = oracle.island_schedule(oracle.islands(mask[b])[0], window)
        np.testing.assert_array_equal(step[b], want)
        assert n[b] == nfe
    return step, n


@pytest.mark.parametrize("shape", [(2, 1, 1), (2, 1, 40), (2, 9, 1), (3, 17, 33), (4, 64, 64), (2, 40, 70),
                                   (1, 16, 1024), (1, 128, 128)])
@pytest.mark.parametrize("window", [1, 3, 16])
def test_schedule_random_masks(ctx, shape, window):
    rng = np.random.default_rng(shape[1] * 77 + shape[2] + window)
    for density in (0.1, 0.5, 0.9):
        mask = (rng.random(shape) < density).astype(np.uint8)
        schedule_both(ctx, mask, window)


def test_schedule_closed_forms(ctx):
    H, W = 32, 48
    mask = np.zeros((3, H, W), np.uint8)
    mask[0] = 1                      # one island covering the grid
    mask[1, 4:12, 10:30] = 1         # a solid block
    step, n = schedule_both(ctx, mask, 16)
    assert list(n) == [W + (H - 1) * 16, 20 + 7 * 16, 0]
    step, n = schedule_both(ctx, mask, 1000)          # window beyond the row: raster order inside an island
    assert list(n) == [H * W, 8 * 20, 0]


def test_schedule_of_a_real_round(ctx):
    cfg = synth.RoundConfig("sched", B=4, H=32, W=32, V=512, dtype="bf16", top_k=64, sigma=0.3, radius=1,
                            seed=4343)
    batch = pu.build_batch(cfg)
    g = pu.gpu_round(ctx, cfg, batch)
    mask = g["expand"].astype(np.uint8)
    step, n = schedule_both(ctx, mask, 16)
    assert (n <= mask.reshape(cfg.B, -1).sum(1)).all() and (n > 0).any()


def test_limits_are_refused_before_launch(ctx):
    p = binding.make_params(1, 129, 128, 8, 1, binding.F32)
    bits = torch.zeros((1, 129, 4), dtype=torch.int32, device="cuda")
    labels = torch.zeros((1, 129, 128), dtype=torch.int32, device="cuda")
    n = torch.zeros((1,), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_islands(p, bits, labels, n)
    assert e.value.status == binding.ERR_UNSUPPORTED
    p = binding.make_params(1, 8, 8, 8, 1, binding.F32)
    with pytest.raises(binding.MuloError) as e:
        ctx.mulo_islands(p, None, labels, n)
    assert e.value.status == binding.ERR_INVALID_ARG


def test_round_driver_chains_the_stages(ctx):
    """The host loop over rounds: every stage runs, the reports are consistent with the arrays behind them,
    and the prefix for the next draft is the draft itself wherever nothing was redrawn."""
    from paper_2601_05149_b200 import driver
    cfg = synth.RoundConfig("drv", B=3, H=32, W=32, V=2048, dtype="bf16", top_k=256, cfg_scale=3.0, sigma=0.3,
                            radius=1, seed=99)
    d = driver.RoundDriver(cfg, ctx, window=4)
    reports = d.run(3)
    assert [r.round for r in reports] == [0, 1, 2]
    assert len({r.acceptance_rate for r in reports}) > 1          # fresh logits every round
    last = reports[-1]
    assert 0.0 < last.acceptance_rate < 1.0 and last.redraw_fraction >= 1.0 - last.acceptance_rate
    assert last.draft_steps == 4 * (cfg.h - 1) + cfg.w
    labels, step = d.labels.cpu().numpy(), d.step.cpu().numpy()
    expand = binding.unpack_bits(d.out["expand_bits"], cfg.W).numpy().astype(bool)
    assert ((labels > 0) == expand).all() and ((step > 0) == expand).all()
    assert last.target_steps_per_image == step.reshape(cfg.B, -1).max(1).sum() / cfg.B
    untouched = expand.reshape(cfg.B, cfg.h, cfg.r, cfg.w, cfg.r).sum(axis=(2, 4)) == 0
    assert (d.prefix_lo.cpu().numpy()[untouched] == d.tok_lo.cpu().numpy()[untouched]).all()
