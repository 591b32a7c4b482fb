"""ctypes access to the CPU oracle (``mulo_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the CPU-baseline leg of
the benchmark import this package.  It knows nothing about the CUDA library and
imports nothing from it.  Arrays are numpy; logits are ``float32`` or raw bf16
bit patterns (``uint16``).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mulo_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libmulo_oracle.so")

F32, BF16 = 0, 1
ACCEPT_RATIO, ACCEPT_THRESHOLD = 0, 1
RESAMPLE_MIXED, RESAMPLE_RESIDUAL_ALL, RESAMPLE_TARGET_ALL, RESAMPLE_ISOLATED_RESIDUAL = 0, 1, 2, 3
FLAG_ACCEPT_EDGE, FLAG_CDF_EDGE, FLAG_POOL_EDGE = 1, 2, 4


class OrcParams(C.Structure):
    _fields_ = [
        ("H", C.c_int32), ("W", C.c_int32), ("V", C.c_int32), ("r", C.c_int32),
        ("dtype", C.c_int32),
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
        ("image", C.c_uint32),
    ]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no fp contraction)."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None
_lock = threading.Lock()


def lib() -> C.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            _lib = C.CDLL(build())
            _lib.orc_uniform24.restype = C.c_double
            _lib.orc_topk_threshold.restype = C.c_float
            _lib.orc_pool.restype = C.c_double
            _lib.orc_accept_threshold.restype = C.c_double
            _lib.orc_accept_threshold.argtypes = [C.c_double, C.c_double]
            _lib.orc_inverse_cdf.restype = C.c_int
            _lib.orc_expand.restype = C.c_int
            _lib.orc_islands.restype = C.c_int
            _lib.orc_island_schedule.restype = C.c_int
            _lib.orc_redraw_loop.restype = C.c_int
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"logits must be float32 or uint16 (bf16 bits), got {a.dtype}")


def make_params(H, W, V, r, dtype, *, temperature=1.0, top_k=0, cfg_scale=1.0,
                accept_mode=ACCEPT_RATIO, tau=1e-4, pool_k=1, pool_delta=0.1, radius=1,
                clip_before_first=1, resample_mode=RESAMPLE_MIXED, seed=0, round=0, image=0):
    return OrcParams(H, W, V, r, dtype, temperature, top_k, cfg_scale, accept_mode, tau, pool_k,
                     pool_delta, radius, clip_before_first, resample_mode, seed, round, image)


# ----------------------------------------------------------------- primitives

def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    out = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, out)
    return tuple(int(x) for x in out)


def position_uniforms(seed, image, position, round, tag=0):
    u = (C.c_double * 3)()
    lib().orc_position_uniforms(C.c_uint64(seed), C.c_uint32(image), C.c_uint32(position),
                                C.c_uint32(round), C.c_uint32(tag), u)
    return tuple(float(x) for x in u)


def preprocess_row(cond, uncond=None, cfg_scale=1.0, temperature=1.0):
    cond = np.ascontiguousarray(cond)
    V = cond.shape[0]
    z = np.empty(V, np.float32)
    if uncond is not None:
        uncond = np.ascontiguousarray(uncond)
        assert uncond.dtype == cond.dtype
    lib().orc_preprocess_row(_ptr(cond), _ptr(uncond), _dtype_code(cond), V, C.c_float(cfg_scale),
                             C.c_float(temperature), _ptr(z))
    return z


def topk_threshold(z, top_k):
    z = np.ascontiguousarray(z, np.float32)
    return float(lib().orc_topk_threshold(_ptr(z), z.shape[0], int(top_k)))


def softmax_masked(z, theta=-np.inf):
    z = np.ascontiguousarray(z, np.float32)
    p = np.empty(z.shape[0], np.float64)
    m, Z = C.c_double(), C.c_double()
    lib().orc_softmax_masked(_ptr(z), z.shape[0], C.c_float(theta), _ptr(p), C.byref(m), C.byref(Z))
    return p, m.value, Z.value


def pool(p, nn_row, pool_k, delta, tok):
    p = np.ascontiguousarray(p, np.float64)
    pp = np.empty_like(p)
    J, gap = C.c_int(), C.c_double()
    nn_row = None if nn_row is None else np.ascontiguousarray(nn_row, np.uint16)
    P = lib().orc_pool(_ptr(p), p.shape[0], _ptr(nn_row), int(pool_k), C.c_double(delta), int(tok),
                       _ptr(pp), C.byref(J), C.byref(gap))
    return float(P), pp, J.value, gap.value


def accept_threshold(P, q):
    return float(lib().orc_accept_threshold(P, q))


def inverse_cdf(w, u):
    w = np.ascontiguousarray(w, np.float64)
    Z, gap = C.c_double(), C.c_double()
    tok = lib().orc_inverse_cdf(_ptr(w), w.shape[0], C.c_double(u), C.byref(Z), C.byref(gap))
    return int(tok), Z.value, gap.value


def residual_weights(p_prime, q, lam):
    p_prime = np.ascontiguousarray(p_prime, np.float64)
    q = np.ascontiguousarray(q, np.float64)
    w = np.empty_like(q)
    lib().orc_residual_weights(_ptr(p_prime), _ptr(q), q.shape[0], C.c_double(lam), _ptr(w))
    return w


def inverse_cdf_histogram(w, n_begin=0, n_end=1 << 24):
    w = np.ascontiguousarray(w, np.float64)
    hist = np.zeros(w.shape[0], np.int64)
    lib().orc_inverse_cdf_histogram(_ptr(w), w.shape[0], C.c_uint32(n_begin), C.c_uint32(n_end),
                                    _ptr(hist))
    return hist


def expand(reject, radius, clip_before_first=1):
    reject = np.ascontiguousarray(reject, np.uint8)
    H, W = reject.shape
    out = np.empty_like(reject)
    t0 = lib().orc_expand(_ptr(reject), H, W, int(radius), int(clip_before_first), _ptr(out))
    return out, int(t0)


def islands(in_rx):
    """Eq. 8: labels [H, W] (0 outside R_X, islands 1..M numbered by their first raster
    position), and per island its first / last grid row and its number of positions."""
    in_rx = np.ascontiguousarray(in_rx, np.uint8)
    H, W = in_rx.shape
    labels = np.zeros((H, W), np.int32)
    rows = np.zeros((max(H * W, 1), 2), np.int32)
    size = np.zeros(max(H * W, 1), np.int32)
    M = int(lib().orc_islands(_ptr(in_rx), H, W, _ptr(labels), _ptr(rows), _ptr(size)))
    return labels, M, rows[:M].copy(), size[:M].copy()


def island_schedule(labels, window):
    """Step index of every position of R_X under the row-window rule (0 outside R_X) and the number of
    sequential steps of the image."""
    labels = np.ascontiguousarray(labels, np.int32)
    H, W = labels.shape
    step = np.zeros((H, W), np.int32)
    nfe = int(lib().orc_island_schedule(_ptr(labels), H, W, int(window), _ptr(step)))
    return step, nfe


def redraw_loop(params, step, cond_steps, uncond_steps, tok, with_edge=False):
    """The redraw of R_X, one target-model call per sequential step: ``cond_steps[s - 1]`` (and
    ``uncond_steps[s - 1]``, or None) are the [H, W, V] logits of call s.  Returns the grid's tokens
    after the redraw and the number of calls made."""
    H, W = params.H, params.W
    step = np.ascontiguousarray(step, np.int32)
    n_steps = int(step.max()) if step.size else 0
    assert len(cond_steps) >= n_steps
    conds = [np.ascontiguousarray(c) for c in cond_steps[:n_steps]]
    unconds = None if uncond_steps is None else [np.ascontiguousarray(u) for u in uncond_steps[:n_steps]]
    arr = (C.c_void_p * max(1, n_steps))(*[c.ctypes.data for c in conds])
    uarr = None if unconds is None else (C.c_void_p * max(1, n_steps))(*[u.ctypes.data for u in unconds])
    out = np.array(tok, np.int32, copy=True).reshape(H, W)
    edge = np.zeros((H, W), np.uint8)
    calls = int(lib().orc_redraw_loop(C.byref(params), _ptr(step), n_steps, arr, uarr, _ptr(out), _ptr(edge)))
    return (out, calls, edge) if with_edge else (out, calls)


def position_distributions(params, cond_row, uncond_row, draft_row, tok, nn=None):
    V = params.V
    q = np.empty(V, np.float64)
    p = np.empty(V, np.float64)
    pp = np.empty(V, np.float64)
    mass = C.c_double()
    lib().orc_position_distributions(C.byref(params), _ptr(np.ascontiguousarray(cond_row)),
                                     _ptr(None if uncond_row is None else np.ascontiguousarray(uncond_row)),
                                     _ptr(np.ascontiguousarray(draft_row)), int(tok), _ptr(nn),
                                     _ptr(q), _ptr(p), _ptr(pp), C.byref(mass))
    return q, p, pp, mass.value


def sample_draft_tokens(params, draft_lo, with_edge=False):
    h, w = params.H // params.r, params.W // params.r
    tok = np.empty((h, w), np.int32)
    edge = np.zeros((h, w), np.uint8)
    lib().orc_sample_draft_tokens(C.byref(params), _ptr(np.ascontiguousarray(draft_lo)), _ptr(tok), _ptr(edge))
    return (tok, edge) if with_edge else tok


def downsample_majority(x, r):
    """Step 7 stand-in: the most frequent token of every r x r block (ties: first in raster order)."""
    x = np.ascontiguousarray(x, np.int32)
    H, W = x.shape
    y = np.empty((H // r, W // r), np.int32)
    lib().orc_downsample_majority(_ptr(x), H, W, int(r), _ptr(y))
    return y


# --------------------------------------------------------------------- stages

def upsample_pool_image(params, draft_lo, draft_tok_lo):
    H, W, r = params.H, params.W, params.r
    h, w = H // r, W // r
    draft_lo = np.ascontiguousarray(draft_lo)
    draft_tok_lo = np.ascontiguousarray(draft_tok_lo, np.int32)
    tok_hi = np.empty((H, W), np.int32)
    stats = np.empty((h, w, 3), np.float64)
    q_tok = np.empty((H, W), np.float64)
    lib().orc_upsample_pool_image(C.byref(params), _ptr(draft_lo), _ptr(draft_tok_lo), _ptr(tok_hi),
                                  _ptr(stats), _ptr(q_tok))
    return dict(tok_hi=tok_hi, stats=stats, q_tok=q_tok)


def round_image(params, cond, uncond, draft_lo, draft_tok_lo, nn=None):
    """One speculative round for one image; returns a dict of numpy arrays."""
    H, W = params.H, params.W
    cond = np.ascontiguousarray(cond)
    uncond = None if uncond is None else np.ascontiguousarray(uncond)
    draft_lo = np.ascontiguousarray(draft_lo)
    draft_tok_lo = np.ascontiguousarray(draft_tok_lo, np.int32)
    nn = None if nn is None else np.ascontiguousarray(nn, np.uint16)
    assert _dtype_code(cond) == params.dtype == _dtype_code(draft_lo)
    out = dict(
        out_tok=np.empty((H, W), np.int32), reject=np.empty((H, W), np.uint8),
        expand=np.empty((H, W), np.uint8), p_tok=np.empty((H, W), np.float64),
        q_tok=np.empty((H, W), np.float64), accept_prob=np.empty((H, W), np.float64),
        flags=np.empty((H, W), np.uint32), cand_tok=np.empty((H, W), np.int32),
        counts=np.empty(3, np.int32))
    lib().orc_round_image(C.byref(params), _ptr(cond), _ptr(uncond), _ptr(draft_lo),
                          _ptr(draft_tok_lo), _ptr(nn), _ptr(out["out_tok"]), _ptr(out["reject"]),
                          _ptr(out["expand"]), _ptr(out["p_tok"]), _ptr(out["q_tok"]),
                          _ptr(out["accept_prob"]), _ptr(out["flags"]), _ptr(out["cand_tok"]),
                          _ptr(out["counts"]))
    return out
