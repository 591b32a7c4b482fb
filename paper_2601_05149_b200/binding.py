"""Thin ctypes binding of ``libmulo.so``: the same calls as ``include/mulo.h``.

Argument marshalling only -- every step of the round runs in the CUDA kernels.
Tensors are torch CUDA tensors (torch is used for device memory and streams);
there is no CPU fallback: a missing library raises ``RuntimeError``.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmulo.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1
ACCEPT_RATIO, ACCEPT_THRESHOLD = 0, 1
RESAMPLE_MIXED, RESAMPLE_RESIDUAL_ALL, RESAMPLE_TARGET_ALL, RESAMPLE_ISOLATED_RESIDUAL = 0, 1, 2, 3
DEV_ZERO_DRAFT_PROB, DEV_BAD_TOKEN, DEV_DENSE_FALLBACK, DEV_TIMEOUT = 1, 2, 4, 8

EXPORTS = (
    "mulo_create", "mulo_destroy", "mulo_status_string", "mulo_workspace_bytes",
    "mulo_set_workspace", "mulo_poll_device_status", "mulo_status_of_device_flags", "mulo_poll_fallback_counts",
    "mulo_kernel_launches",
    "mulo_set_timing", "mulo_read_timing", "mulo_set_general_path_only", "mulo_round_kernel",
    "mulo_upsample_pool", "mulo_verify", "mulo_local_reject_expand", "mulo_islands", "mulo_island_schedule", "mulo_sample_draft", "mulo_downsample", "mulo_resample",
    "mulo_redraw_plan", "mulo_redraw_step",
    "mulo_round", "mulo_round_host_arena_bytes", "mulo_round_host", "mulo_round_static",
)

STATIC_SCRATCH_BYTES = 1 << 20


class MuloParams(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("H", C.c_int32), ("W", C.c_int32), ("V", C.c_int32), ("r", C.c_int32),
        ("logit_dtype", C.c_int32),
        ("temperature", C.c_float),
        ("top_k", C.c_int32),
        ("cfg_scale", C.c_float),
        ("accept_mode", C.c_int32),
        ("tau", C.c_float),
        ("pool_k", C.c_int32),
        ("pool_delta", C.c_float),
        ("radius", C.c_int32),
        ("clip_before_first", C.c_int32),
        ("resample_mode", C.c_int32),
        ("seed", C.c_uint64),
        ("round", C.c_uint32),
        ("image_offset", C.c_uint32),
    ]


class MuloError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status_string(status)} (status {status})")
        self.status = status


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2601_05149_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.mulo_status_string.restype = C.c_char_p
        L.mulo_status_string.argtypes = [C.c_int]
        L.mulo_destroy.restype = None
        for name in EXPORTS:
            fn = getattr(L, name)
            if name not in ("mulo_status_string", "mulo_destroy"):
                fn.restype = C.c_int
        _lib = L
    return _lib


def status_of_device_flags(flags: int) -> int:
    """The status a set of MULO_DEV_* bits maps to (ERR_TIMEOUT or OK)."""
    return lib().mulo_status_of_device_flags(C.c_uint32(flags))


def status_string(status: int) -> str:
    return lib().mulo_status_string(int(status)).decode()


def make_params(B, H, W, V, r, dtype, *, temperature=1.0, top_k=0, cfg_scale=1.0,
                accept_mode=ACCEPT_RATIO, tau=1e-4, pool_k=1, pool_delta=0.1, radius=1,
                clip_before_first=1, resample_mode=RESAMPLE_MIXED, seed=0, round=0,
                image_offset=0) -> MuloParams:
    return MuloParams(B, H, W, V, r, dtype, temperature, top_k, cfg_scale, accept_mode, tau, pool_k,
                      pool_delta, radius, clip_before_first, resample_mode, seed, round, image_offset)


def params_from_config(cfg, **over) -> MuloParams:
    """MuloParams for a ``synth.RoundConfig``."""
    kw = dict(temperature=cfg.temperature, top_k=cfg.top_k, cfg_scale=cfg.cfg_scale,
              accept_mode=cfg.accept_mode, tau=cfg.tau, pool_k=cfg.pool_k, pool_delta=cfg.pool_delta,
              radius=cfg.radius, clip_before_first=cfg.clip_before_first,
              resample_mode=cfg.resample_mode, seed=cfg.seed, round=cfg.round)
    B = over.pop("B", cfg.B)
    kw.update(over)
    return make_params(B, cfg.H, cfg.W, cfg.V, cfg.r, BF16 if cfg.dtype == "bf16" else F32, **kw)


def _dev(t):
    if t is None:
        return C.c_void_p(None)
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensor arguments must be contiguous CUDA tensors")
    return C.c_void_p(t.data_ptr())


def _host(t):
    if t is None:
        return C.c_void_p(None)
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("host arguments must be contiguous CPU tensors")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(status, what):
    if status != OK:
        raise MuloError(status, what)


class Context:
    """A ``mulo_ctx`` plus the torch-allocated workspace it was handed."""

    def __init__(self, device: int | None = None):
        if device is None:
            device = torch.cuda.current_device()
        self.device = device
        self._ctx = C.c_void_p()
        _check(lib().mulo_create(C.byref(self._ctx), int(device)), "mulo_create")
        self._ws = None

    def close(self):
        if self._ctx:
            lib().mulo_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- workspace ---------------------------------------------------------
    @staticmethod
    def workspace_bytes(p: MuloParams) -> int:
        n = C.c_size_t()
        _check(lib().mulo_workspace_bytes(C.byref(p), C.byref(n)), "mulo_workspace_bytes")
        return n.value

    def set_workspace(self, t: torch.Tensor):
        _check(lib().mulo_set_workspace(self._ctx, _dev(t), C.c_size_t(t.numel() * t.element_size())),
               "mulo_set_workspace")
        self._ws = t

    def ensure_workspace(self, p: MuloParams):
        need = self.workspace_bytes(p)
        if self._ws is None or self._ws.numel() < need:
            self.set_workspace(torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}"))

    def poll_device_status(self, stream=None) -> int:
        """The MULO_DEV_* bits since the last poll; raises MuloError(ERR_TIMEOUT) if a kernel's
        bounded wait gave up (the bits are then in the exception's ``flags``)."""
        f = C.c_uint32()
        st = lib().mulo_poll_device_status(self._ctx, _stream(stream), C.byref(f))
        if st != OK:
            e = MuloError(st, "mulo_poll_device_status")
            e.flags = f.value
            raise e
        return f.value

    def poll_fallback_counts(self, stream=None):
        """[rows redone by the general routines, list full, too few candidates, k-th largest
        above the histogram, crowded bin] since the last poll."""
        c = (C.c_uint32 * 5)()
        _check(lib().mulo_poll_fallback_counts(self._ctx, _stream(stream), c), "mulo_poll_fallback_counts")
        return [int(x) for x in c]

    def kernel_launches(self) -> int:
        n = C.c_uint64()
        _check(lib().mulo_kernel_launches(self._ctx, C.byref(n)), "mulo_kernel_launches")
        return n.value

    def round_kernel(self, p: "MuloParams", has_uncond: bool) -> str:
        """The row kernel ``mulo_round`` launches for these parameters: "full", "lane", "stream" or "general"."""
        k = C.c_int()
        _check(lib().mulo_round_kernel(self._ctx, C.byref(p), int(has_uncond), C.byref(k)), "mulo_round_kernel")
        return ("general", "stream", "lane", "full")[k.value]

    def set_general_path_only(self, on: bool):
        _check(lib().mulo_set_general_path_only(self._ctx, int(bool(on))), "mulo_set_general_path_only")

    def set_timing(self, max_launches: int):
        _check(lib().mulo_set_timing(self._ctx, int(max_launches)), "mulo_set_timing")

    def read_timing(self):
        """(summed milliseconds, launches) of the fused row kernel since the last read."""
        ms, n = C.c_double(), C.c_uint64()
        _check(lib().mulo_read_timing(self._ctx, C.byref(ms), C.byref(n)), "mulo_read_timing")
        return ms.value, n.value

    # -- stages ------------------------------------------------------------
    def mulo_upsample_pool(self, p, draft_logits_lo, draft_tok_lo, nn, draft_tok_hi, draft_stats_lo,
                           q_tok_hi, stream=None):
        _check(lib().mulo_upsample_pool(self._ctx, C.byref(p), _dev(draft_logits_lo), _dev(draft_tok_lo),
                                        _dev(nn), _dev(draft_tok_hi), _dev(draft_stats_lo),
                                        _dev(q_tok_hi), _stream(stream)), "mulo_upsample_pool")

    def mulo_verify(self, p, tgt_cond, tgt_uncond, draft_logits_lo, draft_stats_lo, draft_tok_hi, nn,
                    p_tok, q_tok, accept_prob, reject_bits, n_reject, first_reject, stream=None):
        _check(lib().mulo_verify(self._ctx, C.byref(p), _dev(tgt_cond), _dev(tgt_uncond),
                                 _dev(draft_logits_lo), _dev(draft_stats_lo), _dev(draft_tok_hi),
                                 _dev(nn), _dev(p_tok), _dev(q_tok), _dev(accept_prob),
                                 _dev(reject_bits), _dev(n_reject), _dev(first_reject),
                                 _stream(stream)), "mulo_verify")

    def mulo_local_reject_expand(self, p, reject_bits, first_reject, expand_bits, n_expand, stream=None):
        _check(lib().mulo_local_reject_expand(self._ctx, C.byref(p), _dev(reject_bits),
                                              _dev(first_reject), _dev(expand_bits), _dev(n_expand),
                                              _stream(stream)), "mulo_local_reject_expand")

    def mulo_island_schedule(self, p, labels, window, step, n_steps, stream=None):
        _check(lib().mulo_island_schedule(self._ctx, C.byref(p), _dev(labels), C.c_int32(int(window)), _dev(step),
                                          _dev(n_steps), _stream(stream)), "mulo_island_schedule")

    def mulo_sample_draft(self, p, draft_logits_lo, draft_tok_lo, stream=None):
        _check(lib().mulo_sample_draft(self._ctx, C.byref(p), _dev(draft_logits_lo), _dev(draft_tok_lo),
                                       _stream(stream)), "mulo_sample_draft")

    def mulo_downsample(self, p, tok_hi, tok_lo, stream=None):
        _check(lib().mulo_downsample(self._ctx, C.byref(p), _dev(tok_hi), _dev(tok_lo), _stream(stream)),
               "mulo_downsample")

    def mulo_islands(self, p, expand_bits, labels, n_islands, island_rows=None, island_size=None,
                     max_islands=None, stream=None):
        if max_islands is None:
            max_islands = 0
            if island_rows is not None:
                max_islands = island_rows.shape[1]
            elif island_size is not None:
                max_islands = island_size.shape[1]
        _check(lib().mulo_islands(self._ctx, C.byref(p), _dev(expand_bits), _dev(labels), _dev(n_islands),
                                  C.c_int32(int(max_islands)), _dev(island_rows), _dev(island_size),
                                  _stream(stream)), "mulo_islands")

    def mulo_resample(self, p, tgt_cond, tgt_uncond, draft_logits_lo, draft_stats_lo, draft_tok_hi, nn,
                      reject_bits, expand_bits, out_tok, stream=None):
        _check(lib().mulo_resample(self._ctx, C.byref(p), _dev(tgt_cond), _dev(tgt_uncond),
                                   _dev(draft_logits_lo), _dev(draft_stats_lo), _dev(draft_tok_hi),
                                   _dev(nn), _dev(reject_bits), _dev(expand_bits), _dev(out_tok),
                                   _stream(stream)), "mulo_resample")

    def mulo_redraw_plan(self, p, step, max_step, pos_list, step_offsets, stream=None):
        _check(lib().mulo_redraw_plan(self._ctx, C.byref(p), _dev(step), int(max_step), _dev(pos_list),
                                      _dev(step_offsets), _stream(stream)), "mulo_redraw_plan")

    def mulo_redraw_step(self, p, s, max_step, pos_list, step_offsets, tgt_cond, tgt_uncond, out_tok, stream=None):
        _check(lib().mulo_redraw_step(self._ctx, C.byref(p), int(s), int(max_step), _dev(pos_list),
                                      _dev(step_offsets), _dev(tgt_cond), _dev(tgt_uncond), _dev(out_tok),
                                      _stream(stream)), "mulo_redraw_step")

    def mulo_round(self, p, tgt_cond, tgt_uncond, draft_logits_lo, draft_tok_lo, nn, out_tok,
                   reject_bits, expand_bits, p_tok=None, q_tok=None, accept_prob=None, n_reject=None,
                   n_expand=None, first_reject=None, stream=None):
        _check(lib().mulo_round(self._ctx, C.byref(p), _dev(tgt_cond), _dev(tgt_uncond),
                                _dev(draft_logits_lo), _dev(draft_tok_lo), _dev(nn), _dev(out_tok),
                                _dev(reject_bits), _dev(expand_bits), _dev(p_tok), _dev(q_tok),
                                _dev(accept_prob), _dev(n_reject), _dev(n_expand), _dev(first_reject),
                                _stream(stream)), "mulo_round")

    def mulo_round_static(self, p, tgt_cond, tgt_uncond, draft_logits_lo, draft_tok_lo, nn, out_tok,
                          reject_bits, expand_bits, p_tok=None, q_tok=None, accept_prob=None,
                          n_reject=None, n_expand=None, first_reject=None, device_status=None,
                          stream=None):
        """``mulo_round`` on the library's built-in scratch array: for hosts that cannot
        allocate device memory.  Needs no workspace; at most ``STATIC_SCRATCH_BYTES`` of
        scratch (``workspace_bytes(p)``), one call at a time per device.  ``device_status``
        is an optional one-element int32 CUDA tensor for the MULO_DEV_* bits."""
        _check(lib().mulo_round_static(self._ctx, C.byref(p), _dev(tgt_cond), _dev(tgt_uncond),
                                       _dev(draft_logits_lo), _dev(draft_tok_lo), _dev(nn),
                                       _dev(out_tok), _dev(reject_bits), _dev(expand_bits),
                                       _dev(p_tok), _dev(q_tok), _dev(accept_prob), _dev(n_reject),
                                       _dev(n_expand), _dev(first_reject), _dev(device_status),
                                       _stream(stream)), "mulo_round_static")

    @staticmethod
    def round_host_arena_bytes(p: MuloParams, has_uncond: bool) -> int:
        n = C.c_size_t()
        _check(lib().mulo_round_host_arena_bytes(C.byref(p), int(has_uncond), C.byref(n)),
               "mulo_round_host_arena_bytes")
        return n.value

    def mulo_round_host(self, p, arena, tgt_cond, tgt_uncond, draft_logits_lo, draft_tok_lo, nn,
                        out_tok, reject_bits, expand_bits, p_tok=None, q_tok=None, accept_prob=None,
                        n_reject=None, n_expand=None, first_reject=None, stream=None):
        """All tensor arguments except ``arena`` are HOST tensors."""
        self._ws = None     # the arena replaces the workspace
        _check(lib().mulo_round_host(self._ctx, C.byref(p), _dev(arena),
                                     C.c_size_t(arena.numel() * arena.element_size()),
                                     _host(tgt_cond), _host(tgt_uncond), _host(draft_logits_lo),
                                     _host(draft_tok_lo), _host(nn), _host(out_tok),
                                     _host(reject_bits), _host(expand_bits), _host(p_tok),
                                     _host(q_tok), _host(accept_prob), _host(n_reject),
                                     _host(n_expand), _host(first_reject), _stream(stream)),
               "mulo_round_host")


def alloc_round_outputs(p: MuloParams, device, probs: bool = True):
    """Output tensors of ``mulo_round`` for these parameters."""
    B, H, W = p.B, p.H, p.W
    Ww = (W + 31) // 32
    o = dict(
        out_tok=torch.empty((B, H, W), dtype=torch.int32, device=device),
        reject_bits=torch.empty((B, H, Ww), dtype=torch.int32, device=device),
        expand_bits=torch.empty((B, H, Ww), dtype=torch.int32, device=device),
        n_reject=torch.empty((B,), dtype=torch.int32, device=device),
        n_expand=torch.empty((B,), dtype=torch.int32, device=device),
        first_reject=torch.empty((B,), dtype=torch.int32, device=device),
    )
    if probs:
        for k in ("p_tok", "q_tok", "accept_prob"):
            o[k] = torch.empty((B, H, W), dtype=torch.float32, device=device)
    return o


def unpack_bits(bits: torch.Tensor, W: int) -> torch.Tensor:
    """[B,H,ceil(W/32)] int32 words -> [B,H,W] uint8 (host-side helper for tests/metrics)."""
    b = bits.detach().cpu().numpy().view("uint32")
    import numpy as np
    sh = (b[..., :, None] >> np.arange(32, dtype=np.uint32)) & 1
    out = sh.reshape(b.shape[0], b.shape[1], -1)[..., :W].astype("uint8")
    return torch.from_numpy(out)
