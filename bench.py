#!/usr/bin/env python
"""Benchmark of the policy-gated block-sparse joint attention path.

    python bench.py --gpus N --steps K --warmup W [--workload flux_1024] [--impl reference]

A "step" is one rapid3_gated_step over one synthetic batch (pool -> scores -> mask select ->
attention, the whole hot path).  The headline value is the effective TFLOP/s counting only the
kept tiles (4*rows*cols*D flops per kept 64x64 tile, tail tiles by their valid tokens),
aggregated over all ranks; ms_per_step is the time of one call.  Ranks are independent
replicas with their own batch (no collective on the data path): weak scaling.

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_22323_b200 import inputs  # noqa: E402

METRIC = "block-sparse joint-attn ms/call & effective TFLOPS (kept tiles) vs bf16 peak"
UNIT = "TFLOP/s (kept tiles)"
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch, from the ncu summary in
# profiles/ (null until a capture of that workload exists)
ATTN_DRAM_BYTES_PER_LAUNCH = {"flux_1024": 423511808, "flux_2048": 579094784, "sd3_1024": 94116608}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# ----------------------------------------------------------------------------- flop accounting
def kept_flops_from_masks(masks, n_tokens, D):
    """masks: list of [H, nb, nb] uint8 (or None for a dense image) -> kept-tile flops."""
    nb = (n_tokens + 63) // 64
    valid = np.full(nb, 64.0)
    valid[-1] = n_tokens - 64 * (nb - 1)
    w = np.outer(valid, valid)                      # rows x cols of every tile
    total = 0.0
    tiles = 0
    for m, H in masks:
        if m is None:
            total += 4.0 * D * w.sum() * H
            tiles += nb * nb * H
        else:
            total += 4.0 * D * float((m.astype(np.float64) * w[None]).sum())
            tiles += int(m.sum())
    return total, tiles


# ----------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
            "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append((time.time(), [t.strip() for t in line.split(",")]))
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=5)

    def summary(self, t0, t1):
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 and len(r) >= 7] or [r for (_, r) in self.rows if len(r) >= 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        def num(x):
            try:
                return float(x)
            except ValueError:
                return None
        sm = [num(r[0]) for r in rows if num(r[0]) is not None]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
        pw = [num(r[2]) for r in rows if num(r[2]) is not None]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": num(rows[0][1]), "reasons": reasons,
                "power_w_max": max(pw) if pw else None, "samples": len(rows)}


# ----------------------------------------------------------------------------- CPU oracle legs
class OracleSample:
    """The oracle (as it stands) on a bounded sample of the workload: mask selection of one sparse
    image, then attention of WHOLE heads of that image (one oracle call per head over all its query
    blocks, inputs converted to bit patterns once) until the time budget is used."""

    def __init__(self, wl, image=None):
        import oracle
        self.oracle = oracle
        self.wl = wl
        if image is None:
            image = next((b for b, r in enumerate(wl.keep_ratios) if r < 1.0), 0)
        self.image = image
        self.ratio = wl.keep_ratios[image]
        q, k, v = (inputs.make_tensor(wl, t, 0, image, "cpu") for t in range(3))
        self.q, self.k, self.v = (np.ascontiguousarray(x.view(torch.int16).numpy().view(np.uint16)) for x in (q, k, v))
        nb = wl.n_blocks
        self.valid = np.full(nb, 64.0)
        self.valid[-1] = wl.n_tokens - 64 * (nb - 1)

    def run(self, budget_s, head=None):
        """Returns (TFLOP/s on kept tiles, seconds, cores, description).  With `head` set the sample is
        that one head; otherwise heads 0, 1, ... until `budget_s` seconds of attention have run."""
        wl, oracle = self.wl, self.oracle
        heads = list(range(wl.heads)) if head is None else [head]
        flops, secs, done = 0.0, 0.0, 0
        for h in heads:
            q, k, v = self.q[h:h + 1], self.k[h:h + 1], self.v[h:h + 1]
            t0 = time.perf_counter()
            if self.ratio < 1.0:
                _, mask, _ = oracle.image_mask(q, k, wl.n_text, self.ratio)
            else:
                mask = np.ones((1, wl.n_blocks, wl.n_blocks), np.uint8)
            oracle.masked_attention(q, k, v, mask, wl.softmax_scale)
            secs += time.perf_counter() - t0
            flops += 4.0 * wl.head_dim * float((mask[0] * np.outer(self.valid, self.valid)).sum())
            done += 1
            if secs > budget_s:
                break
        desc = (f"{wl.name} image {self.image} (keep ratio {self.ratio}): {done} whole head(s) of {wl.heads}, "
                f"mask selection + attention over all {wl.n_blocks} query blocks of each")
        return flops / secs / 1e12, secs, oracle.num_threads(), desc


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def oracle_tiny_single_thread():
    """Seconds the oracle takes for the whole `tiny` workload on one thread (a child process, because the
    OpenMP thread count is fixed when the oracle's library is loaded)."""
    code = ("import time, oracle; from paper_2509_22323_b200 import inputs; wl = inputs.WORKLOADS['tiny'];"
            "Q, K, V = inputs.make_qkv(wl, 0, device='cpu'); a, r = inputs.make_actions(wl, 0);"
            "oracle.num_threads(); t = time.perf_counter();"
            "oracle.gated_step(Q, K, V, a, r, wl.n_text, wl.softmax_scale); print(time.perf_counter() - t)")
    try:
        env = dict(os.environ, OMP_NUM_THREADS="1")
        out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
        return float(out.stdout.strip().split()[-1])
    except Exception:
        return None


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = OracleSample(wl)
    vals, secs_all = [], []
    cores, desc = 0, ""
    # every step is a bounded sample: one whole head (cycled) of one image
    for it in range(args.warmup + args.steps):
        v, secs, cores, desc = sample.run(0.0, head=it % wl.heads)
        if it >= args.warmup:
            vals.append(v)
            secs_all.append(secs)
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs_all)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "batch": wl.batch, "heads": wl.heads, "head_dim": wl.head_dim,
                       "n_text": wl.n_text, "n_image": wl.n_image, "keep_ratios": list(wl.keep_ratios)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- multi-rank plumbing
def rank_step(rank: int, s: int) -> int:
    """Step index a rank draws its inputs with: every rank gets its own batch (weak scaling)."""
    return rank * 1000 + s


def aggregate(dist, device, ms_total: float, flops_total: float, launches: int):
    """Whole-job figures from per-rank ones: the slowest rank's time, the sum of the work.
    `dist` is torch.distributed (any backend) or None for a single process."""
    if dist is None:
        return ms_total, flops_total, launches
    t = torch.tensor([ms_total], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    f = torch.tensor([flops_total, float(launches)], device=device, dtype=torch.float64)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(t.item()), float(f[0].item()), int(f[1].item())


# ----------------------------------------------------------------------------- CUDA arm
class Prepared:
    """One workload ready to step: context, rotated input sets, per-step actions, and the kept-tile
    flops of every step computed from the masks the library itself selected."""

    def __init__(self, wl, rank, dev):
        from paper_2509_22323_b200 import binding
        self.binding, self.wl, self.dev = binding, wl, dev
        self.ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
        self.set_bytes = 3 * wl.batch * wl.heads * wl.n_tokens * wl.head_dim * 2
        # input sets are rotated so that a step never finds its inputs in L2 (126 MB): enough sets that the
        # others together exceed 200 MB; the `tiny` workload would need hundreds, so there a buffer larger
        # than L2 is rewritten before every step instead (outside the step's event pair)
        nsets = max(2, -(-200_000_000 // self.set_bytes) + 1)
        self.flush = None
        if nsets > 8:
            nsets = 2
            self.flush = torch.empty(192 << 20, dtype=torch.uint8, device=dev)
        steps_of = list(range(nsets))
        if wl.steps > 1:
            steps_of = list(range(wl.steps))           # the gated trajectory: fresh Q/K/V per step
            nsets = min(wl.steps, 4)
        self.nsets = nsets
        # each rank draws its own data (weak scaling): shift the step index by the rank
        self.sets = [inputs.make_qkv(wl, rank_step(rank, st), device=dev) for st in range(nsets)]
        self.out = torch.empty_like(self.sets[0][0])
        self.plan = [(self.sets[i % nsets],) + tuple(inputs.make_actions(wl, steps_of[i % len(steps_of)]))
                     for i in range(len(steps_of))]
        self.flops_step, self.tiles_step = [], []
        for i in range(len(self.plan)):
            self.step(i)
            torch.cuda.synchronize()
            _, acts, ratios = self.plan[i]
            sparse = [b for b, (a, r) in enumerate(zip(acts, ratios)) if a == binding.ACT_ATTEND and r < 1.0]
            dense = [b for b, (a, r) in enumerate(zip(acts, ratios)) if a == binding.ACT_ATTEND and r >= 1.0]
            masks = [(None, wl.heads)] * len(dense)
            if sparse:
                ws = self.ctx.workspace(len(sparse), device=dev)
                dm = binding.bitmask_to_dense(ws[1], wl.n_blocks).numpy()
                masks += [(dm[sl], wl.heads) for sl in range(len(sparse))]
            f, t = kept_flops_from_masks(masks, wl.n_tokens, wl.head_dim)
            self.flops_step.append(f)
            self.tiles_step.append(t)
        assert self.ctx.last_status() == 0, "device status word is set"

    def step(self, i):
        (Q, K, V), acts, ratios = self.plan[i % len(self.plan)]
        self.ctx.rapid3_gated_step(Q, K, V, self.out, acts, ratios, self.wl.softmax_scale)

    def flops(self, steps):
        return sum(self.flops_step[i % len(self.plan)] for i in range(steps))

    def l2_note(self):
        if self.flush is not None:
            return (f"inputs smaller than L2: a {self.flush.numel() >> 20} MiB buffer is rewritten before every step, "
                    "each step between its own event pair")
        return f"inputs larger than L2 ({self.set_bytes / 1e6:.0f} MB per set), {self.nsets} input sets rotated"


def timed_region(pw, steps, warmup, dist=None):
    """W warm-up steps, then K steps between one event pair (barrier + synchronize on both sides),
    with an event pair around every attention launch inside.  Returns (ms_total, launches,
    (attention ms, attention launches), wall-clock window)."""
    ctx = pw.ctx
    for i in range(warmup):
        pw.step(i)
    torch.cuda.synchronize()
    ctx.profile(2)                     # an event pair around the attention kernel only: the roofline's duration
    ctx.profile_read()
    n0 = ctx.launch_count()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    w0 = time.time()
    if pw.flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            pw.step(i)
        e1.record()
        torch.cuda.synchronize()
        ms_total = e0.elapsed_time(e1)
    else:
        ms_total = sum(per_step_times(pw, steps))   # L2 flushed before every step, outside its event pair
    w1 = time.time()
    if dist is not None:
        dist.barrier()
    launches = ctx.launch_count() - n0
    attn = ctx.profile_read()["attention"]
    ctx.profile(False)
    return ms_total, launches, attn, (w0, w1)


def per_step_times(pw, n):
    """n steps, each between its own event pair (for a workload smaller than L2 the flush buffer is
    rewritten before the pair): the list of step times in ms."""
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    torch.cuda.synchronize()
    for i, (a, b) in enumerate(pairs):
        if pw.flush is not None:
            pw.flush.fill_(i & 0xFF)
        a.record()
        pw.step(i)
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in pairs]


def side_kernels(pw, n):
    """Durations of all four kernels from a short pass with an event pair around every launch."""
    pw.ctx.profile(1)
    pw.ctx.profile_read()
    for i in range(n):
        pw.step(i)
    torch.cuda.synchronize()
    pr = pw.ctx.profile_read()
    pw.ctx.profile(False)
    return pr


def attention_roofline(pw, steps, attn, ms_total, peaks, traffic):
    attn_ms, attn_n = attn
    attn_avg_ms = attn_ms / max(1, attn_n)
    achieved = pw.flops(steps) / max(1, attn_n) / (attn_avg_ms * 1e-3) / 1e12 if attn_n else None
    # a timed region under a second is a burst (clocks at their maximum, far below the power cap);
    # a seconds-long one settles at the power cap, where the sustained GEMM figure is the fair peak
    burst = ms_total < 1000.0
    peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    which = "bf16_tflops" if burst else "bf16_tflops_sustained"
    return {"bound": "tensor", "kernel": "attn_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
            "frac": (achieved / peak) if achieved else None, "traffic": traffic,
            "peak_source": f"{which} of {peaks['source']} (timed region {ms_total / 1e3:.3f} s: "
                           f"{'burst' if burst else 'sustained'})",
            "frac_of_burst_peak": (achieved / peaks["bf16_tflops"]) if achieved else None,
            "frac_of_sustained_peak": (achieved / peaks["bf16_tflops_sustained"]) if achieved else None,
            "frac_of_nominal_2250": (achieved / 2250.0) if achieved else None,
            "avg_launch_ms": attn_avg_ms, "launches": attn_n}


def keep_ratio_sweep(pw, n=20):
    """The whole batch at one keep ratio: ratio 1.0 is the dense reference, the others show how the
    time follows the kept-tile fraction."""
    binding, wl, ctx = pw.binding, pw.wl, pw.ctx
    (Q, K, V) = pw.sets[0]
    sweep = []
    for r in (1.0, 0.5, 0.25):
        acts, ratios = [binding.ACT_ATTEND] * wl.batch, [r] * wl.batch
        for _ in range(3):
            ctx.rapid3_gated_step(Q, K, V, pw.out, acts, ratios, wl.softmax_scale)
        torch.cuda.synchronize()
        frac = 1.0
        if r < 1.0:
            frac = float(binding.bitmask_to_dense(ctx.workspace(wl.batch, device=pw.dev)[1], wl.n_blocks).numpy().mean())
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            ctx.rapid3_gated_step(Q, K, V, pw.out, acts, ratios, wl.softmax_scale)
        b.record()
        torch.cuda.synchronize()
        step_ms = a.elapsed_time(b) / n
        ctx.profile(True)
        ctx.profile_read()
        for _ in range(n):
            ctx.rapid3_gated_step(Q, K, V, pw.out, acts, ratios, wl.softmax_scale)
        torch.cuda.synchronize()
        pr = ctx.profile_read()
        ctx.profile(False)
        sweep.append({"keep_ratio": r, "kept_tile_fraction": frac, "step_ms": step_ms,
                      "attention_ms": pr["attention"][0] / pr["attention"][1],
                      "kernels_ms_sum": sum(v[0] for v in pr.values()) / n})
    for e in sweep:
        e["attention_speedup_vs_ratio_1"] = sweep[0]["attention_ms"] / e["attention_ms"]
        e["step_speedup_vs_ratio_1"] = sweep[0]["step_ms"] / e["step_ms"]
        e["proportional_speedup"] = 1.0 / e["kept_tile_fraction"]
    return sweep


def workload_entry(name, peaks, steps=30, warmup=5):
    """One line of the per-workload list: the same measurement as the headline, on another workload."""
    wl = inputs.WORKLOADS[name]
    dev = torch.device("cuda", torch.cuda.current_device())
    pw = Prepared(wl, 0, dev)
    if wl.steps > 1:
        steps = 2 * wl.steps
    ms_total, launches, attn, _ = timed_region(pw, steps, warmup)
    roof = attention_roofline(pw, steps, attn, ms_total, peaks, None)
    ts = per_step_times(pw, max(50, wl.steps * 2))
    pr = side_kernels(pw, max(len(pw.plan), 20))
    e = {"workload": name, "steps": steps, "ms_per_step": ms_total / steps,
         "ms_per_step_median": statistics.median(ts) if ts else None, "ms_per_step_min": min(ts) if ts else None,
         "attention_ms": roof["avg_launch_ms"], "value": pw.flops(steps) / (ms_total * 1e-3) / 1e12, "unit": UNIT,
         "attention_tflops": roof["achieved"], "frac_of_burst_peak": roof["frac_of_burst_peak"],
         "frac_of_nominal_2250": roof["frac_of_nominal_2250"], "gpu_launches": int(launches),
         "kept_flops_per_step": pw.flops_step[0], "l2": pw.l2_note(),
         "kernels_avg_ms": {k: (v[0] / v[1]) if v[1] else None for k, v in pr.items()}}
    if wl.steps > 1:
        per_traj = steps // wl.steps
        e["ms_per_trajectory"] = ms_total / per_traj
        e["launched_image_steps_per_trajectory"] = sum(
            sum(1 for a in pw.plan[i][1] if a == pw.binding.ACT_ATTEND) for i in range(wl.steps))
        e["kept_flops_per_trajectory"] = pw.flops(wl.steps)
    elif name != "tiny":
        e["keep_ratio_sweep"] = keep_ratio_sweep(pw)
    assert pw.ctx.last_status() == 0, f"{name}: device status word is set"
    del pw
    torch.cuda.empty_cache()
    return e


def run_ours(args, wl):
    from paper_2509_22323_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    pw = Prepared(wl, rank, dev)
    ctx, sets, plan, out = pw.ctx, pw.sets, pw.plan, pw.out
    flops_step, tiles_step = pw.flops_step, pw.tiles_step

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ms_total, launches, attn, (w0, w1) = timed_region(pw, args.steps, args.warmup, dist)
    # the other kernels' durations come from a short pass of their own (an event pair around every launch
    # costs a few microseconds of stream time each, which the timed region should not carry four times per step)
    prof = side_kernels(pw, max(len(plan), min(args.steps, 50)))
    prof["attention"] = attn
    step_ts = per_step_times(pw, max(50, 2 * len(plan)))
    assert ctx.last_status() == 0, "device status word is set after the timed region"
    if rank == 0:
        time.sleep(0.2)
        sampler.stop()
    rank_ms = ms_total
    ms_total, flops_total, launches = aggregate(dist, dev, ms_total, pw.flops(args.steps), launches)
    value = flops_total / (ms_total * 1e-3) / 1e12

    # ---- end to end through the host-buffer entry point (rank-local, then max over ranks)
    e2e = None
    if not args.no_e2e:
        hQ, hK, hV = [t.cpu().pin_memory() for t in sets[0]]
        hO = torch.empty_like(hQ).pin_memory()
        _, acts, ratios = plan[0]
        up, down = ctx.rapid3_gated_step_host(hQ, hK, hV, hO, acts, ratios, wl.softmax_scale)   # allocates staging
        torch.cuda.synchronize()
        n_e2e = max(3, min(args.steps, 20))
        if dist is not None:
            dist.barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        h0 = time.perf_counter()
        for _ in range(n_e2e):
            up, down = ctx.rapid3_gated_step_host(hQ, hK, hV, hO, acts, ratios, wl.softmax_scale)
        host_us = (time.perf_counter() - h0) / n_e2e * 1e6
        a1.record()
        torch.cuda.synchronize()
        ms_e2e = a0.elapsed_time(a1)
        if dist is not None:
            t = torch.tensor([ms_e2e], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_e2e = float(t.item())
        e2e = {"value": world * flops_step[0] * n_e2e / (ms_e2e * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": int(up), "d2h_bytes_per_step": int(down), "ms_per_step": ms_e2e / n_e2e,
               "steps": n_e2e, "host_us_per_call": host_us, "checksum": float(hO[0, 0, 0, :8].float().sum())}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    roofline = attention_roofline(pw, args.steps, attn, rank_ms, peaks, ATTN_DRAM_BYTES_PER_LAUNCH.get(wl.name))
    pool_ms, pool_n = prof["block_pool"]
    pool_bytes = None
    if pool_n:
        n_sparse_launch = sum(1 for r in plan[0][2] if r < 1.0) if wl.steps == 1 else None
        if n_sparse_launch:
            pool_bytes = 2.0 * n_sparse_launch * wl.heads * wl.n_tokens * wl.head_dim * 2
    kernels = {k: {"ms_total": v[0], "launches": v[1], "avg_ms": (v[0] / v[1]) if v[1] else None} for k, v in prof.items()}
    if pool_bytes:
        kernels["block_pool"]["achieved_gbs"] = pool_bytes / (pool_ms / pool_n * 1e-3) / 1e9
        kernels["block_pool"]["frac_of_hbm_peak"] = kernels["block_pool"]["achieved_gbs"] / peaks["hbm_gbs"]

    sweep = None
    if not args.no_sweep and wl.steps == 1 and world == 1:
        sweep = keep_ratio_sweep(pw)

    # the entry points beside the headline step, timed on the same inputs (device events, 20 calls each)
    variants = None
    if not args.no_sweep and wl.steps == 1 and world == 1:
        variants = {}
        (Q, K, V) = sets[0]
        acts, ratios = plan[0][1], plan[0][2]

        def timed(fn, n=20):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(n):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n

        # one keep ratio per (image, head): the image's ratio scaled by 0.5 / 1.0 / 1.5 in turn over the heads
        head_ratios = [[min(1.0, r * (0.5 + 0.5 * (h % 3))) if r < 1.0 else 1.0 for h in range(wl.heads)] for r in ratios]
        variants["gated_step_heads_ms"] = timed(lambda: ctx.rapid3_gated_step_heads(Q, K, V, out, acts, head_ratios,
                                                                                  wl.softmax_scale))
        variants["gated_step_ms"] = timed(lambda: ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale))
        # host time of one call through the Python binding (gate, compaction, four launches; nothing waits on the GPU)
        torch.cuda.synchronize()
        h0 = time.perf_counter()
        for _ in range(100):
            ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
        variants["host_us_per_call"] = (time.perf_counter() - h0) / 100 * 1e6
        torch.cuda.synchronize()
        a_dev = torch.tensor(acts, dtype=torch.int32, device=dev)
        r_dev = torch.tensor(ratios, dtype=torch.float32, device=dev)
        variants["gated_step_device_ms"] = timed(lambda: ctx.rapid3_gated_step_device(Q, K, V, out, a_dev, r_dev,
                                                                                    wl.softmax_scale))
        n_sp = sum(1 for a, r in zip(acts, ratios) if a == binding.ACT_ATTEND and r < 1.0)
        if n_sp:
            sc = ctx.workspace(n_sp, device=dev)[0].clone()
            variants["select_mask_mass_ms"] = timed(lambda: ctx.rapid3_select_mask_mass(sc, [0.5] * n_sp,
                                                                                      4.0 * wl.softmax_scale))
            variants["select_mask_ms"] = timed(lambda: ctx.rapid3_select_mask(sc, [0.5] * n_sp))
            variants["select_images"] = n_sp
        # the gated step with the Q/K producer folded in (RMS norm, gain, rotary embedding, pooling): its
        # first kernel replaces the pooling kernel; bytes = raw Q, K read + Q, K written for the attending images
        gq = torch.ones(wl.head_dim, device=dev)
        gk = torch.ones(wl.head_dim, device=dev)
        # identity rotations (the inputs already carry their rotary embedding): the table is read like any
        # other, and the block structure the masks depend on stays that of the workload
        rot = torch.zeros((wl.n_tokens, wl.head_dim // 2, 2), device=dev)
        rot[..., 0] = 1.0
        q2, k2 = torch.empty_like(Q), torch.empty_like(K)
        fused = lambda: ctx.rapid3_gated_step_fused(Q, K, V, gq, gk, rot, 1e-6, q2, k2, out, acts, ratios,
                                                    wl.softmax_scale)
        variants["gated_step_fused_ms"] = timed(fused)
        ctx.profile(True)
        ctx.profile_read()
        for _ in range(20):
            fused()
        torch.cuda.synchronize()
        pr = ctx.profile_read()
        ctx.profile(False)
        n_att = sum(1 for a in acts if a == binding.ACT_ATTEND)
        prod_ms = pr["block_pool"][0] / pr["block_pool"][1]
        variants["fused_step_kernels_ms"] = {kk: vv[0] / max(vv[1], 1) for kk, vv in pr.items()}
        variants["producer_ms"] = prod_ms
        variants["producer_gbs"] = n_att * 4 * wl.heads * wl.n_tokens * wl.head_dim * 2 / (prod_ms * 1e-3) / 1e9
        x = Q.reshape(wl.batch, -1)
        o2, delta = torch.empty_like(x), torch.zeros_like(x)
        cache_acts = [(binding.ACT_ATTEND, binding.ACT_REUSE)[b % 2] for b in range(wl.batch)]
        ms = timed(lambda: binding.rapid3_cache_step(x, o2, delta, cache_acts))
        variants["cache_step_ms"] = ms
        variants["cache_step_gbs"] = 3 * x.numel() * 2 / (ms * 1e-3) / 1e9
        del q2, k2, o2, delta, rot

    cfg_l2 = pw.l2_note()
    del pw, ctx, sets, plan, out
    torch.cuda.empty_cache()

    # every workload of the configuration list on the same GPU in the same run (short regions: burst peak)
    per_workload = None
    if not args.no_per_workload and world == 1:
        per_workload = []
        for name in inputs.WORKLOADS:
            try:
                per_workload.append(workload_entry(name, peaks))
            except Exception as exc:  # a failing side measurement must not lose the headline line
                per_workload.append({"workload": name, "error": f"{type(exc).__name__}: {exc}"})

    cpu = None
    if not args.no_cpu_baseline and world == 1:          # the oracle is timed at N = 1 only
        v, secs, cores, desc = OracleSample(wl).run(args.cpu_budget)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "seconds": secs,
               "cpu_model": cpu_model(), "tiny_1thread_seconds": oracle_tiny_single_thread()}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps,
            "ms_per_step_median": statistics.median(step_ts) if step_ts else None,
            "ms_per_step_min": min(step_ts) if step_ts else None,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "batch": wl.batch, "heads": wl.heads, "head_dim": wl.head_dim,
                       "n_text": wl.n_text, "n_image": wl.n_image, "keep_ratios": list(wl.keep_ratios),
                       "trajectory_steps": wl.steps, "kept_tiles_per_step": tiles_step[0],
                       "kept_flops_per_step": flops_step[0], "l2": cfg_l2},
            "clocks": sampler.summary(w0, w1), "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu, "kernels": kernels, "keep_ratio_sweep": sweep, "variants": variants,
            "per_workload": per_workload}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def spawn_ranks(args) -> int:
    """`--gpus N` with N > 1 from a plain `python bench.py`: start N ranks of this script, one per GPU,
    through torch.distributed.run on this node and pass their output through."""
    import socket
    n_dev = torch.cuda.device_count()
    if n_dev < args.gpus:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} asked for, {n_dev} CUDA device(s) visible\n")
        return 2
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="flux_1024", choices=list(inputs.WORKLOADS))
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    wl = inputs.WORKLOADS[args.workload]
    world = int(os.environ.get("WORLD_SIZE", "0"))
    if world == 0 and args.gpus > 1 and args.impl == "ours":
        sys.exit(spawn_ranks(args))             # not under a launcher: start the N ranks here
    if world > 0 and world != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}")
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
