"""A host-side loop over speculative rounds on synthetic logits (argument marshalling only: every step
runs in the library's kernels).

One round = the drafter's own draw on the low-resolution grid (Sec. 3.2 Step 1), the fused draft-and-verify
round over the whole high-resolution grid (Steps 2-6 on given logits), the rejection islands of R_X and their
redraw schedule (Sec. 3.4), the redraw itself executed step by step (one launch per sequential target-model
step; the model call that would produce a step's logits is stood in for by the round's own target logits), and
the down-sampled prefix for the next low-resolution draft (Step 7 stand-in).
The model forwards that would produce the logits are not part of this repository: every round draws fresh
synthetic logits from the workload's recipe with a round-dependent seed.  The loop reports, per round, what
the paper's latency analysis is made of: acceptance rate, |R_X|, number of islands, sequential target steps
of the redraw under the row-window schedule, and the theoretical speed-up S_T = T_p / ((1 - a) T_p + T_q).
"""
from __future__ import annotations

import dataclasses

import torch

from . import binding, synth


@dataclasses.dataclass
class RoundReport:
    round: int
    acceptance_rate: float
    redraw_fraction: float          # |R_X| / N
    islands_per_image: float
    target_steps_per_image: float   # sequential steps of the redraw (islands concurrently, row window)
    draft_steps: int                # the low-resolution grid under the same row window
    speedup_theoretical: float      # S_T of the paper's latency analysis
    redraw_nfe: int = 0             # target-model calls of the executed redraw: the slowest image's step count
    redraw_us_per_step: float = 0.0  # device time of one redraw step (launch to launch), microseconds


class RoundDriver:
    def __init__(self, cfg: synth.RoundConfig, ctx: binding.Context | None = None, window: int = 16,
                 device="cuda"):
        self.cfg, self.window, self.device = cfg, window, torch.device(device)
        self.ctx = ctx or binding.Context(self.device.index or 0)
        self.p = binding.params_from_config(cfg)
        self.ctx.ensure_workspace(self.p)
        B, H, W, h, w = cfg.B, cfg.H, cfg.W, cfg.h, cfg.w
        i32 = dict(dtype=torch.int32, device=self.device)
        self.out = binding.alloc_round_outputs(self.p, self.device, probs=False)
        self.tok_lo = torch.empty((B, h, w), **i32)
        self.labels = torch.empty((B, H, W), **i32)
        self.n_islands = torch.empty((B,), **i32)
        self.step = torch.empty((B, H, W), **i32)
        self.n_steps = torch.empty((B,), **i32)
        self.prefix_lo = torch.empty((B, h, w), **i32)
        self.pos_list = torch.empty((B * H * W,), **i32)
        self.step_offsets = torch.empty((2 * (H * W + 2),), **i32)

    def run_round(self, rnd: int) -> RoundReport:
        cfg, p, ctx, out = self.cfg, self.p, self.ctx, self.out
        batch = synth.build_batch(dataclasses.replace(cfg, seed=cfg.seed + 7919 * rnd), self.device)
        p.round = rnd
        ctx.mulo_sample_draft(p, batch["draft_lo"], self.tok_lo)
        ctx.mulo_round(p, batch["cond"], batch["uncond"], batch["draft_lo"], self.tok_lo, batch["nn"],
                       out["out_tok"], out["reject_bits"], out["expand_bits"], None, None, None,
                       out["n_reject"], out["n_expand"], out["first_reject"])
        ctx.mulo_islands(p, out["expand_bits"], self.labels, self.n_islands)
        ctx.mulo_island_schedule(p, self.labels, self.window, self.step, self.n_steps)
        # the redraw, executed: one host read (how many steps the slowest image needs), then the plan and one
        # launch per step with nothing read back in between
        nfe = int(self.n_steps.max().item())
        us_per_step = 0.0
        if nfe > 0:
            max_step = cfg.H * cfg.W
            ctx.mulo_redraw_plan(p, self.step, max_step, self.pos_list, self.step_offsets)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for s in range(1, nfe + 1):
                ctx.mulo_redraw_step(p, s, max_step, self.pos_list, self.step_offsets, batch["cond"], batch["uncond"],
                                     out["out_tok"])
            e1.record()
            torch.cuda.synchronize(self.device)
            us_per_step = e0.elapsed_time(e1) * 1e3 / nfe
        ctx.mulo_downsample(p, out["out_tok"], self.prefix_lo)
        torch.cuda.synchronize(self.device)
        n = cfg.B * cfg.H * cfg.W
        acc = 1.0 - int(out["n_reject"].sum().item()) / n
        t_p, t_q = cfg.H * cfg.W, cfg.h * cfg.w
        return RoundReport(
            round=rnd, acceptance_rate=acc, redraw_fraction=int(out["n_expand"].sum().item()) / n,
            islands_per_image=int(self.n_islands.sum().item()) / cfg.B,
            target_steps_per_image=int(self.n_steps.sum().item()) / cfg.B,
            draft_steps=min(cfg.w, self.window) * (cfg.h - 1) + cfg.w,
            speedup_theoretical=t_p / ((1.0 - acc) * t_p + t_q), redraw_nfe=nfe, redraw_us_per_step=us_per_step)

    def run(self, rounds: int):
        return [self.run_round(r) for r in range(rounds)]
