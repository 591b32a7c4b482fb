"""Benchmark of the fused MuLo-SD draft-and-verify round.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C4] [--impl ours|reference]

A step is one fused round (``mulo_round``) over one batch of synthetic logits that
is already resident in HBM.  Prints ONE JSON line: verified grid positions per
second (whole job), the HBM roofline of the row kernel, the same metric end to end
from host buffers, and the CPU oracle timed on a bounded sample of the workload.
Under torchrun (N > 1) every rank runs the same batch shape on its own GPU
(independent images, no collective on the data path; image_offset = rank * B).
"""
from __future__ import annotations

import argparse
import concurrent.futures as cf
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2601_05149_b200 import synth  # noqa: E402

METRIC = "verified_grid_positions_per_sec"
UNIT = "positions/s"

# DRAM traffic of the row kernel per grid position, by (workload, kernel): dram__bytes_read.sum +
# dram__bytes_write.sum of one ncu capture of the workload at B = 2, divided by its 8192 positions
# (traffic grows in proportion to the positions, every row being read once).  An entry is removed when
# its kernel changes, and the line then reports null until the counters have been taken again.
TRAFFIC_BYTES_PER_POSITION = {
    ("C4", "lane"): 74268.0,   # 608.4 MB per launch of 8192 positions (algorithmic: 73,752 B per position)
    ("P4", "full"): 66598.0,   # 545.6 MB per launch of 8192 positions (algorithmic: 67,560 B; the lists come from L2)
}
L2_BYTES = 126 << 20


def shard_for_rank(cfg, rank):
    """Batch sharding over ranks: every rank runs cfg.B images of its own (weak scaling); the global image
    indices of rank r are [r * B, (r + 1) * B), which is also what keys its random streams."""
    return dataclasses.replace(cfg, seed=cfg.seed + 1000 * rank), rank * cfg.B


def reduce_max_ms(dist, elapsed_ms, device):
    """The slowest rank's device time (all ranks get it)."""
    t = torch.tensor([elapsed_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, positions_per_rank, steps, elapsed_ms):
    """Positions per second of the whole job: what all ranks processed over the slowest rank's time."""
    return world * positions_per_rank * steps / (elapsed_ms * 1e-3)


def workload_desc(cfg):
    return (f"{cfg.name}: B={cfg.B} target {cfg.H}x{cfg.W} / draft {cfg.h}x{cfg.w}, V={cfg.V}, {cfg.dtype} "
            f"logits, CFG {cfg.cfg_scale}, top-k {cfg.top_k}, pool_k {cfg.pool_k}, radius {cfg.radius}, "
            f"sigma {cfg.sigma}")


# ----------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.15] or [l for (_, l) in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------- CPU oracle

def _crop_for_oracle(cfg, rows=16):
    """A bounded sample of the workload for the CPU oracle: the first `rows` grid rows
    of an image (same V, dtype, knobs), one such crop per host thread."""
    rows = min(rows, cfg.H)
    rows -= rows % cfg.r
    return dataclasses.replace(cfg, name=cfg.name + "-crop", B=1, H=rows)


def time_oracle(cfg, steps, warmup, cores=None):
    """Times the oracle as it stands on this host: `cores` threads, each running the
    whole round on its own crop.  Returns (positions/s, per-step seconds, cores, sample)."""
    import oracle as orc
    cores = cores or min(os.cpu_count() or 1, 16)
    crop = _crop_for_oracle(cfg)
    inputs = []
    for b in range(cores):
        img = synth.make_image(dataclasses.replace(cfg, H=cfg.H), b, "cpu")
        cut = lambda t, n: None if t is None else synth.to_numpy_logits(t[:n].contiguous())
        draft = cut(img["draft_lo"], crop.h)
        tok = orc.sample_draft_tokens(orc.make_params(
            crop.H, crop.W, crop.V, crop.r, orc.BF16 if crop.dtype == "bf16" else orc.F32,
            temperature=crop.temperature, top_k=crop.top_k, seed=crop.seed, image=b), draft)
        inputs.append((cut(img["cond"], crop.H), cut(img["uncond"], crop.H), draft, tok))
    nn = None
    if cfg.pool_k > 1:
        nn = synth.neighbours_to_numpy(synth.codebook_neighbours(cfg.V, cfg.pool_k, cfg.seed))
    orc.lib()

    def one(args):
        b, rnd = args
        c, u, d, t = inputs[b]
        prm = orc.make_params(
            crop.H, crop.W, crop.V, crop.r, orc.BF16 if crop.dtype == "bf16" else orc.F32,
            temperature=crop.temperature, top_k=crop.top_k, cfg_scale=crop.cfg_scale,
            accept_mode=crop.accept_mode, tau=crop.tau, pool_k=crop.pool_k, pool_delta=crop.pool_delta,
            radius=crop.radius, clip_before_first=crop.clip_before_first, resample_mode=crop.resample_mode,
            seed=crop.seed, round=rnd, image=b)
        return orc.round_image(prm, c, u, d, t, nn)

    times = []
    with cf.ThreadPoolExecutor(max_workers=cores) as ex:
        for s in range(warmup + steps):
            t0 = time.perf_counter()
            list(ex.map(one, [(b, s) for b in range(cores)]))
            dt = time.perf_counter() - t0
            if s >= warmup:
                times.append(dt)
    per_step = sum(times) / len(times)
    positions = cores * crop.H * crop.W
    sample = (f"{cores} threads x one {crop.H}x{crop.W} crop (first {crop.H} grid rows) of a {cfg.name} image, "
              f"{positions} positions per step")
    return positions / per_step, per_step, cores, sample


# ------------------------------------------------------------------- arms

def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, args.steps)
    warmup = max(0, min(args.warmup, 2))
    value, per_step, cores, sample = time_oracle(cfg, steps, warmup)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_desc(cfg), "note": "CPU oracle on a bounded sample of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours(args, cfg):
    from paper_2601_05149_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the round has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    binding.lib()
    ctx = binding.Context(local)
    dev = torch.device("cuda", local)

    # this rank's images: global indices [rank*B, (rank+1)*B)
    rcfg, image_offset = shard_for_rank(cfg, rank)
    batch = synth.build_batch(rcfg, dev)
    p = binding.params_from_config(cfg, image_offset=image_offset)
    ctx.ensure_workspace(p)
    ctx.mulo_sample_draft(p, batch["draft_lo"], batch["tok_lo"])     # the drafter's tokens (Step 1)
    out = binding.alloc_round_outputs(p, dev, probs=False)
    stream = torch.cuda.current_stream()

    positions = cfg.B * cfg.H * cfg.W
    alg_bytes = cfg.algorithmic_bytes_per_position() * positions
    # inputs that fit the L2 twice over would be served from it on every step after the first: such
    # workloads get 256 MB written between steps, and every step is timed by an event pair of its
    # own so that the writes stay outside the timed regions
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if alg_bytes < 2 * L2_BYTES else None

    def step(rnd):
        p.round = rnd
        ctx.mulo_round(p, batch["cond"], batch["uncond"], batch["draft_lo"], batch["tok_lo"], batch["nn"],
                       out["out_tok"], out["reject_bits"], out["expand_bits"], None, None, None,
                       out["n_reject"], out["n_expand"], out["first_reject"], stream)

    W, K = max(3, args.warmup), max(1, args.steps)
    # E over x~ ~ q of the acceptance probability = sum_x min(p, q) (Eq. 1), averaged over the grid:
    # the mean of the round's own accept_prob output, taken once before the timed region
    probs = torch.empty((cfg.B, cfg.H, cfg.W), dtype=torch.float32, device=dev)
    p.round = 0
    ctx.mulo_round(p, batch["cond"], batch["uncond"], batch["draft_lo"], batch["tok_lo"], batch["nn"],
                   out["out_tok"], out["reject_bits"], out["expand_bits"], None, None, probs,
                   out["n_reject"], out["n_expand"], out["first_reject"], stream)
    expected_acceptance = float(probs.double().mean().item())
    del probs
    for s in range(W):
        step(s)
    torch.cuda.synchronize()
    ctx.set_timing(K)
    launches0 = ctx.kernel_launches()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for s in range(K):
            step(W + s)
        e1.record(stream)
        pairs = [(e0, e1)]
    else:
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for s in range(K):
            flush.zero_()
            pairs[s][0].record(stream)
            step(W + s)
            pairs[s][1].record(stream)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    elapsed_ms = sum(a.elapsed_time(b) for a, b in pairs)
    row_ms, row_n = ctx.read_timing()
    ctx.set_timing(0)
    launches = ctx.kernel_launches() - launches0
    if dist:
        elapsed_ms = reduce_max_ms(dist, elapsed_ms, dev)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None

    value = whole_job_value(world, positions, K, elapsed_ms)
    n_rej = int(out["n_reject"].sum().item())
    n_exp = int(out["n_expand"].sum().item())
    acc = 1.0 - n_rej / positions
    status = ctx.poll_device_status()
    fallback = ctx.poll_fallback_counts()

    # roofline of the row kernel: algorithmic bytes of one launch / its mean duration
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = 6650.0, "fallback (6.65 TB/s)"
    row_avg_ms = row_ms / max(1, row_n)
    achieved = alg_bytes / (row_avg_ms * 1e-3) / 1e9
    which = ctx.round_kernel(p, cfg.has_uncond)
    kernel = {"full": "k_round_full",
              "lane": "k_round_lane (+ k_verify_failed for rows that left the fast path)",
              "stream": "k_round_stream (+ k_verify_failed for rows that left the fast path)",
              "general": "k_verify_rows"}[which]
    roofline = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                "frac_of_nominal_8TBps": achieved / 8000.0, "traffic": None,
                "bytes_per_launch": alg_bytes, "avg_launch_ms": row_avg_ms, "launches_timed": row_n}
    per_pos = TRAFFIC_BYTES_PER_POSITION.get((args.workload, which))
    if per_pos is not None:
        roofline["traffic"] = per_pos * positions

    e2e = None
    cpu = None
    if rank == 0:
        e2e = run_e2e(ctx, cfg, p, batch, world, args)
    if dist:
        dist.barrier()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, per_step, cores, sample = time_oracle(cfg, steps=1, warmup=0)
        v1, per_step1, _, sample1 = time_oracle(cfg, steps=1, warmup=0, cores=1)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
               "seconds": per_step, "host_cpus": os.cpu_count(),
               "single_thread": {"value": v1, "unit": UNIT, "sample": sample1, "seconds": per_step1}}
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_desc(cfg), "per_gpu_batch": cfg.B, "logit_dtype": cfg.dtype,
                       "l2": ("inputs per step (%.2f GB) exceed the 126 MB L2; no flush needed" % (alg_bytes / 1e9)
                              if flush is None else
                              "inputs per step (%.1f MB) would stay in the 126 MB L2: 256 MB written between steps, "
                              "outside the per-step timed regions" % (alg_bytes / 1e6)),
                       "acceptance_rate": acc, "expected_acceptance_mean_sum_min_p_q": expected_acceptance,
                       "speedup_theoretical_S_T": (cfg.H * cfg.W) / ((1.0 - acc) * cfg.H * cfg.W + cfg.h * cfg.w),
                       "expanded_fraction": n_exp / positions,
                       "device_status": status,
                       "rows_redone_by_general_kernel": fallback[0], "fallback_reasons": fallback[1:]},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
        }))
    ctx.close()
    if dist:
        dist.destroy_process_group()


def run_e2e(ctx, cfg, p, batch, world, args):
    """The same round through mulo_round_host: pinned host inputs copied to the device,
    results copied back, all inside the timed region (rank 0's GPU; at N > 1 the other
    ranks idle, so this is a single-GPU figure scaled by nothing)."""
    from paper_2601_05149_b200 import binding
    dev = batch["cond"].device
    try:
        host = {k: (None if v is None else v.cpu().pin_memory()) for k, v in batch.items()}
    except RuntimeError as e:
        return {"value": None, "unit": UNIT, "error": f"pinning host memory failed: {e}"}
    arena = torch.empty(binding.Context.round_host_arena_bytes(p, cfg.has_uncond), dtype=torch.uint8, device=dev)
    o = binding.alloc_round_outputs(p, "cpu", probs=False)
    o = {k: v.pin_memory() for k, v in o.items()}
    c2 = binding.Context(dev.index)
    stream = torch.cuda.current_stream()
    steps = max(1, min(args.steps, 3))

    def step(rnd):
        p.round = rnd
        c2.mulo_round_host(p, arena, host["cond"], host["uncond"], host["draft_lo"], host["tok_lo"], host["nn"],
                           o["out_tok"], o["reject_bits"], o["expand_bits"], None, None, None,
                           o["n_reject"], o["n_expand"], o["first_reject"], stream)

    step(0)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for s in range(steps):
        step(1 + s)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    h2d = sum(v.numel() * v.element_size() for v in host.values() if v is not None)
    d2h = sum(v.numel() * v.element_size() for v in o.values())
    c2.close()
    return {"value": cfg.B * cfg.H * cfg.W / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "n_gpus": 1}


def run_sweep(args):
    """The throughput sweep (grids x vocabularies x batches x noise levels): one JSON line per point with
    positions/s, the HBM roofline fraction of the row kernels and the measured acceptance.  Single GPU."""
    from paper_2601_05149_b200 import binding
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the round has no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = binding.Context(0)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
    pts = synth.sweep_points()
    if args.sweep_limit:
        pts = pts[:args.sweep_limit]
    groups = {}
    for c in pts:
        groups.setdefault((c.H, c.V, c.sigma), []).append(c)
    K, Wm = max(1, min(args.steps, 5)), 3
    for (g, V, sigma), cs in groups.items():
        big = max(cs, key=lambda c: c.B)
        batch = synth.build_batch(big, dev)      # the smaller batches are its leading images
        pb = binding.params_from_config(big)
        ctx.ensure_workspace(pb)
        ctx.mulo_sample_draft(pb, batch["draft_lo"], batch["tok_lo"])
        for c in sorted(cs, key=lambda c: c.B):
            cut = {k: (v if v is None or k == "nn" else v[:c.B]) for k, v in batch.items()}
            p = binding.params_from_config(dataclasses.replace(big, B=c.B))
            ctx.ensure_workspace(p)
            out = binding.alloc_round_outputs(p, dev, probs=False)

            def step(rnd):
                p.round = rnd
                ctx.mulo_round(p, cut["cond"], cut["uncond"], cut["draft_lo"], cut["tok_lo"], cut["nn"],
                               out["out_tok"], out["reject_bits"], out["expand_bits"], None, None, None,
                               out["n_reject"], out["n_expand"], out["first_reject"])
            for s_ in range(Wm):
                step(s_)
            torch.cuda.synchronize()
            ctx.set_timing(K)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for s_ in range(K):
                step(Wm + s_)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / K
            row_ms, row_n = ctx.read_timing()
            ctx.set_timing(0)
            positions = c.B * c.H * c.W
            alg = c.algorithmic_bytes_per_position() * positions
            gbs = alg / (row_ms / max(1, row_n) * 1e-3) / 1e9
            print(json.dumps({
                "sweep_point": c.name, "grid": c.H, "V": c.V, "B": c.B, "sigma": c.sigma, "metric": METRIC,
                "value": positions / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
                "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak},
                "l2_resident": alg < 126e6,
                "acceptance_rate": 1.0 - int(out["n_reject"].sum().item()) / positions,
                "expanded_fraction": int(out["n_expand"].sum().item()) / positions,
                "rows_redone_by_general_kernel": ctx.poll_fallback_counts()[0]}), flush=True)
        del batch
        torch.cuda.empty_cache()
    ctx.close()


def run_islands(args, cfg):
    """Rejection islands (Eq. 8) of the masks one round of the workload leaves: one JSON line per batch size
    (the workload's own batch, then the same masks repeated to 1024 images), with the CPU oracle timed on the
    same masks.  Single GPU."""
    from paper_2601_05149_b200 import binding
    import numpy as np
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the islands kernel has no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = binding.Context(0)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
    batch = synth.build_batch(cfg, dev)
    p = binding.params_from_config(cfg)
    ctx.ensure_workspace(p)
    ctx.mulo_sample_draft(p, batch["draft_lo"], batch["tok_lo"])
    out = binding.alloc_round_outputs(p, dev, probs=False)
    ctx.mulo_round(p, batch["cond"], batch["uncond"], batch["draft_lo"], batch["tok_lo"], batch["nn"],
                   out["out_tok"], out["reject_bits"], out["expand_bits"], None, None, None,
                   out["n_reject"], out["n_expand"], out["first_reject"])
    torch.cuda.synchronize()
    del batch
    W, K = max(3, args.warmup), max(1, args.steps)
    cap = 256
    for B in (cfg.B, max(cfg.B, 1024)):
        reps = (B + cfg.B - 1) // cfg.B
        bits = out["expand_bits"].repeat(reps, 1, 1)[:B].contiguous()
        pb = binding.params_from_config(dataclasses.replace(cfg, B=B))
        labels = torch.empty((B, cfg.H, cfg.W), dtype=torch.int32, device=dev)
        n = torch.empty((B,), dtype=torch.int32, device=dev)
        rows = torch.empty((B, cap, 2), dtype=torch.int32, device=dev)
        size = torch.empty((B, cap), dtype=torch.int32, device=dev)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2
        launches0 = ctx.kernel_launches()
        e = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for s_ in range(W + K):
            flush.zero_()
            if s_ >= W:
                e[s_ - W][0].record()
            ctx.mulo_islands(pb, bits, labels, n, rows, size)
            if s_ >= W:
                e[s_ - W][1].record()
        torch.cuda.synchronize()
        ms = statistics.mean(a.elapsed_time(b) for a, b in e)
        positions = B * cfg.H * cfg.W
        alg = bits.numel() * 4 + labels.numel() * 4 + n.numel() * 4 + rows.numel() * 4 + size.numel() * 4
        cpu = None
        if B == cfg.B and not args.no_cpu_baseline:
            import oracle
            masks = binding.unpack_bits(bits, cfg.W).numpy().astype(np.uint8)
            t0 = time.time()
            total = sum(oracle.islands(masks[b])[1] for b in range(B))
            dt = time.time() - t0
            assert total == int(n.sum().item())
            cpu = {"value": positions / dt, "unit": "positions/s", "cores": 1, "kind": "oracle",
                   "sample": f"all {B} masks of the batch", "seconds": dt}
        print(json.dumps({
            "stage": "mulo_islands", "metric": "island_labelled_positions_per_sec",
            "value": positions / (ms * 1e-3), "unit": "positions/s", "ms_per_step": ms, "steps": K, "warmup": W,
            "dtype": "int32", "data": "synthetic",
            "config": {"workload": workload_desc(cfg), "images": B, "islands_per_image": int(n.sum().item()) / B,
                       "l2": "256 MB written between timed launches"},
            "roofline": {"bound": "hbm", "kernel": "k_islands", "achieved": alg / (ms * 1e-3) / 1e9, "peak": peak,
                         "unit": "GB/s", "frac": alg / (ms * 1e-3) / 1e9 / peak, "bytes_per_launch": alg,
                         "traffic": None},
            "cpu_baseline": cpu, "gpu_launches": ctx.kernel_launches() - launches0}), flush=True)
        if B != cfg.B:
            continue
        # the schedule of the redraw: islands concurrently, a row window of 16 inside an island (ZipAR-16)
        window = 16
        step = torch.empty((B, cfg.H, cfg.W), dtype=torch.int32, device=dev)
        n_steps = torch.empty((B,), dtype=torch.int32, device=dev)
        e = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for s_ in range(W + K):
            flush.zero_()
            if s_ >= W:
                e[s_ - W][0].record()
            ctx.mulo_island_schedule(pb, labels, window, step, n_steps)
            if s_ >= W:
                e[s_ - W][1].record()
        torch.cuda.synchronize()
        ms = statistics.mean(a.elapsed_time(b) for a, b in e)
        n_rx = int(out["n_expand"].sum().item())
        acc = 1.0 - int(out["n_reject"].sum().item()) / positions
        t_p, t_q = cfg.H * cfg.W, cfg.h * cfg.w
        cpu = None
        if not args.no_cpu_baseline:
            lab = labels.cpu().numpy()
            t0 = time.time()
            total = sum(oracle.island_schedule(lab[b], window)[1] for b in range(B))
            dt = time.time() - t0
            assert total == int(n_steps.sum().item())
            cpu = {"value": positions / dt, "unit": "positions/s", "cores": 1, "kind": "oracle",
                   "sample": f"all {B} images", "seconds": dt}
        alg = 2 * labels.numel() * 4 + n_steps.numel() * 4
        print(json.dumps({
            "stage": "mulo_island_schedule", "metric": "scheduled_positions_per_sec",
            "value": positions / (ms * 1e-3), "unit": "positions/s", "ms_per_step": ms, "steps": K, "warmup": W,
            "dtype": "int32", "data": "synthetic",
            "config": {"workload": workload_desc(cfg), "images": B, "window": window,
                       "positions_to_redraw_per_image": n_rx / B,
                       "sequential_target_steps_per_image": int(n_steps.sum().item()) / B,
                       "acceptance_rate": acc,
                       "theoretical_speedup_S_T": t_p / ((1.0 - acc) * t_p + t_q)},
            "roofline": {"bound": "hbm", "kernel": "k_island_schedule", "achieved": alg / (ms * 1e-3) / 1e9,
                         "peak": peak, "unit": "GB/s", "frac": alg / (ms * 1e-3) / 1e9 / peak,
                         "bytes_per_launch": alg, "traffic": None},
            "cpu_baseline": cpu}), flush=True)
    ctx.close()


def run_draft_io(args, cfg):
    """Step 1 (the drafter's own sampling on given logits) and the Step 7 stand-in (majority down-sampler) on
    the workload's shapes: one JSON line each, with the CPU oracle timed on a bounded sample.  Single GPU."""
    from paper_2601_05149_b200 import binding
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: these stages have no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = binding.Context(0)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
    batch = synth.build_batch(cfg, dev)
    p = binding.params_from_config(cfg)
    ctx.ensure_workspace(p)
    W, K = max(3, args.warmup), max(1, args.steps)
    esz = 2 if cfg.dtype == "bf16" else 4
    cells = cfg.B * cfg.h * cfg.w
    tok_lo = torch.empty((cfg.B, cfg.h, cfg.w), dtype=torch.int32, device=dev)
    tok_hi = torch.randint(0, cfg.V, (cfg.B, cfg.H, cfg.W), dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2

    def timed(fn):
        e = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for s_ in range(W + K):
            flush.zero_()
            p.round = s_
            if s_ >= W:
                e[s_ - W][0].record()
            fn()
            if s_ >= W:
                e[s_ - W][1].record()
        torch.cuda.synchronize()
        return statistics.mean(a.elapsed_time(b) for a, b in e)

    def line(stage, kernel, metric, units, ms, alg, cpu):
        print(json.dumps({
            "stage": stage, "metric": metric, "value": units / (ms * 1e-3), "unit": metric.split("_per_")[0] + "/s",
            "ms_per_step": ms, "steps": K, "warmup": W, "dtype": "f32" if stage == "mulo_sample_draft" else "int32",
            "data": "synthetic",
            "config": {"workload": workload_desc(cfg), "l2": "256 MB written between timed launches"},
            "roofline": {"bound": "hbm", "kernel": kernel, "achieved": alg / (ms * 1e-3) / 1e9, "peak": peak,
                         "unit": "GB/s", "frac": alg / (ms * 1e-3) / 1e9 / peak, "bytes_per_launch": alg,
                         "traffic": None},
            "cpu_baseline": cpu}), flush=True)

    def orc_params(b):
        import oracle
        return oracle.make_params(cfg.H, cfg.W, cfg.V, cfg.r, oracle.BF16 if cfg.dtype == "bf16" else oracle.F32,
                                  temperature=cfg.temperature, top_k=cfg.top_k, seed=cfg.seed, round=0, image=b)
    ms = timed(lambda: ctx.mulo_sample_draft(p, batch["draft_lo"], tok_lo))
    cpu = None
    if not args.no_cpu_baseline:
        import oracle   # the CPU-baseline leg is the only user of the oracle here
        n_img = min(cfg.B, 2)
        t0 = time.time()
        for b in range(n_img):
            oracle.sample_draft_tokens(orc_params(b), synth.to_numpy_logits(batch["draft_lo"][b]))
        dt = time.time() - t0
        cpu = {"value": n_img * cfg.h * cfg.w / dt, "unit": "cells/s", "cores": 1, "kind": "oracle",
               "sample": f"{n_img} of {cfg.B} images", "seconds": dt}
    line("mulo_sample_draft", "k_round_stream<sampling mode> (+ k_sample_failed)", "cells_per_sec", cells, ms, cells * (cfg.V * esz + 4), cpu)

    ms = timed(lambda: ctx.mulo_downsample(p, tok_hi, tok_lo))
    cpu = None
    if not args.no_cpu_baseline:
        import oracle
        x = tok_hi.cpu().numpy()
        t0 = time.time()
        for b in range(cfg.B):
            oracle.downsample_majority(x[b], cfg.r)
        dt = time.time() - t0
        cpu = {"value": cells / dt, "unit": "cells/s", "cores": 1, "kind": "oracle",
               "sample": f"all {cfg.B} images", "seconds": dt}
    line("mulo_downsample", "k_downsample", "cells_per_sec", cells, ms, cells * 4 * (cfg.r * cfg.r + 1), cpu)
    ctx.close()


def run_driver(args, cfg):
    """The host loop over rounds (draft draw, fused round, islands, redraw schedule, down-sampled prefix) on
    fresh synthetic logits per round: one JSON line per round with what the paper's latency analysis uses,
    then one line with the device time of the library's own launches per round.  Single GPU."""
    from paper_2601_05149_b200 import binding, driver
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the driver has no CPU path")
    torch.cuda.set_device(0)
    ctx = binding.Context(0)
    d = driver.RoundDriver(cfg, ctx, window=16)
    K = max(1, args.steps)
    for r in d.run(K):
        print(json.dumps({"stage": "round_driver", **dataclasses.asdict(r)}), flush=True)
    # the library's launches of one round, timed on given logits (the logit generator is not the subject)
    batch = synth.build_batch(cfg, "cuda")
    p, out = d.p, d.out
    ctx.mulo_sample_draft(p, batch["draft_lo"], batch["tok_lo"])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = ctx.kernel_launches()

    def one(rnd):
        p.round = rnd
        ctx.mulo_sample_draft(p, batch["draft_lo"], d.tok_lo)
        ctx.mulo_round(p, batch["cond"], batch["uncond"], batch["draft_lo"], d.tok_lo, batch["nn"],
                       out["out_tok"], out["reject_bits"], out["expand_bits"], None, None, None,
                       out["n_reject"], out["n_expand"], out["first_reject"])
        ctx.mulo_islands(p, out["expand_bits"], d.labels, d.n_islands)
        ctx.mulo_island_schedule(p, d.labels, d.window, d.step, d.n_steps)
        ctx.mulo_downsample(p, out["out_tok"], d.prefix_lo)
    for r in range(3):
        one(r)
    torch.cuda.synchronize()
    n0 = ctx.kernel_launches()
    e0.record()
    for r in range(K):
        one(3 + r)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / K
    print(json.dumps({"stage": "round_driver", "metric": "rounds_per_sec", "value": 1e3 / ms, "unit": "rounds/s",
                      "ms_per_round": ms, "steps": K, "gpu_launches_per_round": (ctx.kernel_launches() - n0) / K,
                      "config": {"workload": workload_desc(cfg), "window": 16}, "data": "synthetic"}), flush=True)
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4", choices=sorted(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch size")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="run the throughput sweep instead of the bench line")
    ap.add_argument("--sweep-limit", type=int, default=0, help="only the first N sweep points")
    ap.add_argument("--islands", action="store_true",
                    help="time the rejection-island labelling of the workload's masks instead of the bench line")
    ap.add_argument("--draft-io", action="store_true",
                    help="time the drafter's sampling and the down-sampler stand-in instead of the bench line")
    ap.add_argument("--driver", action="store_true",
                    help="run the host loop over rounds (all stages, fresh synthetic logits per round)")
    args = ap.parse_args()
    cfg = synth.CONFIGS[args.workload]
    if args.batch:
        cfg = dataclasses.replace(cfg, B=args.batch, name=f"{cfg.name}(B={args.batch})")
    if args.sweep:
        run_sweep(args)
    elif args.islands:
        run_islands(args, cfg)
    elif args.draft_io:
        run_draft_io(args, cfg)
    elif args.driver:
        run_driver(args, cfg)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
