"""Seeded synthetic inputs for the MuLo-SD draft-and-verify round.

This module only MAKES INPUTS (logit tensors, codebook neighbour lists).  It holds none of the round's arithmetic and is the one module that both
the CUDA tests/benchmark and the CPU oracle's tests draw their data from.

Recipe (per image ``b`` of a config with seed ``s``; generator seed
``s * 1_000_003 + b``):

1. draft logits on the low-res grid ``[h, w, V]``: ``2 * N(0,1)``, rounded to the
   logit dtype;
2. conditional target logits ``[H, W, V]``: nearest-neighbour up-sampled draft
   logits (as fp32) ``+ sigma * N(0,1)``, rounded to the logit dtype;
3. with classifier-free guidance: unconditional logits ``= fp32(cond) + N(0,1)``,
   rounded;
4. draft tokens ``[h, w]``: one draw per low-res cell from the draft distribution
   (temperature and top-k applied) -- the drafter's own sampling step, which the
   round takes as an input.  They are NOT drawn here: callers use the library's
   ``mulo_sample_draft`` or, where the tokens feed the oracle, the oracle's sampler;
5. with probability pooling: a synthetic codebook ``E ~ N(0,1)^{V x 8}`` and, per
   token, the ``k`` nearest codebook entries by L2 distance (self first, ties to
   the lower id) as ``uint16``.

These stand in for the logits of the paper's AR models on its evaluation prompts,
which need trained weights and datasets that are not available here.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class RoundConfig:
    name: str
    B: int
    H: int
    W: int
    V: int
    r: int = 2
    dtype: str = "bf16"          # "bf16" | "f32"
    sigma: float = 0.5           # target-vs-draft logit noise
    cfg_scale: float = 0.0       # 0: no unconditional tensor
    temperature: float = 1.0
    top_k: int = 0
    pool_k: int = 1
    pool_delta: float = 0.1
    radius: int = 1
    clip_before_first: int = 1
    accept_mode: int = 0
    tau: float = 1e-4
    resample_mode: int = 0
    seed: int = 0
    round: int = 0

    @property
    def h(self):
        return self.H // self.r

    @property
    def w(self):
        return self.W // self.r

    @property
    def has_uncond(self):
        return self.cfg_scale != 0.0

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_size(self):
        return 2 if self.dtype == "bf16" else 4

    def algorithmic_bytes_per_position(self) -> float:
        """Bytes the method itself must move per target position: the target
        row(s), the parent's draft row shared by r*r children, the neighbour list
        when pooling is on, and the per-position outputs."""
        v = self.V * self.elem_size
        # Eq. 5 with every redraw from the target distribution never looks at the draft row
        # (accept_mode 1 = threshold rule, resample_mode 2 = target for all)
        draft = 0.0 if (self.accept_mode == 1 and self.resample_mode == 2) else v / (self.r * self.r)
        return v * (2 if self.has_uncond else 1) + draft + \
            (2 * self.pool_k if self.pool_k > 1 else 0) + 24


# The workloads named by the build's baseline description.
CONFIGS = {
    "C1": RoundConfig("C1", B=1, H=16, W=16, V=4096, dtype="f32", sigma=0.5, radius=1, seed=0),
    "C2": RoundConfig("C2", B=1, H=32, W=32, V=16384, sigma=0.5, top_k=2000, pool_k=1000,
                      pool_delta=0.1, radius=1, seed=1),
    "C3": RoundConfig("C3", B=8, H=64, W=64, V=16384, sigma=0.5, cfg_scale=3.0, top_k=2000,
                      radius=1, seed=2),
    "C4": RoundConfig("C4", B=32, H=64, W=64, V=16384, sigma=1.0, cfg_scale=3.0, top_k=2000,
                      radius=3, seed=3),
    # C4's shapes under the paper's default sampling: no top-k cut, CFG 4.0, probability pooling over
    # the k = 1000 nearest codebook entries with delta = 0.1, the relaxed rule of Eq. 5 with tau = 1e-4,
    # every redraw from the target distribution, l = 3
    "P4": RoundConfig("P4", B=32, H=64, W=64, V=16384, sigma=1.0, cfg_scale=4.0, top_k=0, pool_k=1000,
                      pool_delta=0.1, radius=3, accept_mode=1, tau=1e-4, resample_mode=2, seed=5),
}


def sweep_points():
    """The throughput sweep: grids x vocabularies x batches x noise levels."""
    pts = []
    idx = 0
    for g in (32, 64, 96):
        for V in (8192, 16384):
            for B in (1, 4, 16, 64):
                for sigma in (0.1, 0.5, 1.0, 2.0):
                    pts.append(replace(CONFIGS["C4"], name=f"S{idx}", B=B, H=g, W=g, V=V,
                                       sigma=sigma, radius=1, seed=4 + idx))
                    idx += 1
    return pts


def _gen(cfg: RoundConfig, b: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + b)
    return g


def make_image(cfg: RoundConfig, b: int, device="cpu"):
    """Logits of image ``b``: dict(draft_lo [h,w,V], cond [H,W,V], uncond | None)."""
    g = _gen(cfg, b, device)
    dt = cfg.torch_dtype
    h, w, V, r = cfg.h, cfg.w, cfg.V, cfg.r
    draft = (2.0 * torch.randn((h, w, V), generator=g, device=device, dtype=torch.float32)).to(dt)
    up = draft.float().repeat_interleave(r, dim=0).repeat_interleave(r, dim=1)
    cond = (up + cfg.sigma * torch.randn((cfg.H, cfg.W, V), generator=g, device=device,
                                         dtype=torch.float32)).to(dt)
    del up
    uncond = None
    if cfg.has_uncond:
        uncond = (cond.float() + torch.randn((cfg.H, cfg.W, V), generator=g, device=device,
                                             dtype=torch.float32)).to(dt)
    return dict(draft_lo=draft.contiguous(), cond=cond.contiguous(),
                uncond=None if uncond is None else uncond.contiguous())


def codebook_neighbours(V: int, k: int, seed: int, device="cpu") -> torch.Tensor:
    """``[V, k]`` uint16-valued ids (returned as int32 holding 0..V-1, cast by the
    caller): the k nearest entries of a random 8-dim codebook, self first."""
    assert V <= 65536
    g = torch.Generator(device=device)
    g.manual_seed(seed * 7_368_787 + 11)
    E = torch.randn((V, 8), generator=g, device=device, dtype=torch.float32)
    out = torch.empty((V, k), dtype=torch.int32, device=device)
    ids = torch.arange(V, device=device)
    step = 1024
    for s in range(0, V, step):
        d = torch.cdist(E[s:s + step].double(), E.double())
        d[torch.arange(d.shape[0], device=device), ids[s:s + step]] = -1.0  # self first
        # stable sort => ties go to the lower id
        order = torch.sort(d, dim=1, stable=True).indices[:, :k]
        out[s:s + step] = order.to(torch.int32)
    return out


def to_numpy_logits(t: torch.Tensor) -> np.ndarray:
    """Host numpy view of a logit tensor: float32, or bf16 as raw uint16 bits."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def neighbours_to_numpy(nn: torch.Tensor) -> np.ndarray:
    return nn.detach().cpu().numpy().astype(np.uint16)


def build_batch(cfg: RoundConfig, device="cuda"):
    """The logits of one round as device tensors, and an UNFILLED ``tok_lo`` [B, h, w] int32: the
    drafter's tokens are the caller's to draw (this module holds none of the method's arithmetic) --
    with ``mulo_sample_draft`` in the benchmark and the round driver, with the oracle's sampler
    where the tokens feed the oracle."""
    dt = cfg.torch_dtype
    cond = torch.empty((cfg.B, cfg.H, cfg.W, cfg.V), dtype=dt, device=device)
    uncond = torch.empty_like(cond) if cfg.has_uncond else None
    draft = torch.empty((cfg.B, cfg.h, cfg.w, cfg.V), dtype=dt, device=device)
    tok = torch.zeros((cfg.B, cfg.h, cfg.w), dtype=torch.int32, device=device)
    for b in range(cfg.B):
        img = make_image(cfg, b, device)
        cond[b] = img["cond"]
        if uncond is not None:
            uncond[b] = img["uncond"]
        draft[b] = img["draft_lo"]
        del img
    nn = None
    if cfg.pool_k > 1:
        # uint16 ids, carried in an int16 tensor (same bit pattern)
        ids = neighbours_to_numpy(codebook_neighbours(cfg.V, cfg.pool_k, cfg.seed, device))
        nn = torch.from_numpy(ids.view(np.int16)).to(device).contiguous()
    return dict(cond=cond, uncond=uncond, draft_lo=draft, tok_lo=tok, nn=nn)
