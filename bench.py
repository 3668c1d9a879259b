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
ATTN_DRAM_BYTES_PER_LAUNCH = {"flux_1024": 421726208, "flux_2048": 579465216, "sd3_1024": 93985536}
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
    image on all heads, plus attention on as many (head, query-block) units as fit the budget."""

    def __init__(self, wl, image=None):
        import oracle
        self.oracle = oracle
        self.wl = wl
        if image is None:
            image = next((b for b, r in enumerate(wl.keep_ratios) if r < 1.0), 0)
        self.image = image
        self.ratio = wl.keep_ratios[image]
        self.q, self.k, self.v = (inputs.make_tensor(wl, t, 0, image, "cpu") for t in range(3))
        nb = wl.n_blocks
        self.valid = np.full(nb, 64.0)
        self.valid[-1] = wl.n_tokens - 64 * (nb - 1)
        # every (head, query-block) unit of the image in a fixed scattered order (stride coprime to
        # the unit count), so that any prefix mixes text rows, image rows, the tail and all heads
        n_units = wl.heads * nb
        stride = next(s for s in range(max(2, int(0.618 * n_units)), 2 * n_units + 2) if np.gcd(s, n_units) == 1)
        self.units = [divmod((u * stride) % n_units, nb) for u in range(n_units)]

    def run(self, budget_s, head=None):
        """Returns (TFLOP/s on kept tiles, seconds, cores, description).  With `head` set, the
        sample is that one head only (mask selection and attention units of that head)."""
        wl, oracle = self.wl, self.oracle
        heads = list(range(wl.heads)) if head is None else [head]
        q, k, v = (x[heads[0]:heads[-1] + 1] for x in (self.q, self.k, self.v))
        t0 = time.perf_counter()
        S32, mask, gap = oracle.image_mask(q, k, wl.n_text, self.ratio)
        t_mask = time.perf_counter() - t0
        flops, done, t_att = 0.0, 0, 0.0
        for h, i in self.units:
            if h not in heads:
                continue
            hl = h - heads[0]
            t1 = time.perf_counter()
            oracle.masked_attention(q, k, v, mask, wl.softmax_scale, qb_lo=i, qb_hi=i + 1, heads=[hl])
            t_att += time.perf_counter() - t1
            flops += 4.0 * wl.head_dim * self.valid[i] * float((mask[hl, i] * self.valid).sum())
            done += 1
            if t_att > budget_s:
                break
        # the mask pass covers every tile of the sampled heads; charge it in proportion to the sampled units
        secs = t_att + t_mask * done / (len(heads) * wl.n_blocks)
        desc = (f"{wl.name} image {self.image} (keep ratio {self.ratio}): mask selection on {len(heads)} head(s), "
                f"attention on {done} sampled (head, query-block) units; mask time charged pro rata")
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
    # every step is a bounded sample (one head, cycled); the whole run stays within ~2.5 minutes
    budget = max(0.01, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    for it in range(args.warmup + args.steps):
        v, secs, cores, desc = sample.run(budget, head=it % wl.heads)
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

    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    nsets = 2
    steps_of = list(range(nsets))
    if wl.steps > 1:
        steps_of = list(range(wl.steps))           # the gated trajectory: fresh Q/K/V per step
        nsets = min(wl.steps, 4)
    # each rank draws its own data (weak scaling): shift the step index by the rank
    sets = [inputs.make_qkv(wl, rank_step(rank, s), device=dev) for s in range(nsets)]
    out = torch.empty_like(sets[0][0])
    plan = [(sets[i % nsets],) + tuple(inputs.make_actions(wl, steps_of[i % len(steps_of)])) for i in range(len(steps_of))]

    def one_step(i):
        (Q, K, V), acts, ratios = plan[i % len(plan)]
        ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)

    # flops per step from the masks the library itself selected (marshalling for the report only)
    flops_step, tiles_step, launches_img = [], [], []
    for i in range(len(plan)):
        one_step(i)
        torch.cuda.synchronize()
        (Q, K, V), acts, ratios = plan[i]
        sparse = [b for b, (a, r) in enumerate(zip(acts, ratios)) if a == binding.ACT_ATTEND and r < 1.0]
        dense = [b for b, (a, r) in enumerate(zip(acts, ratios)) if a == binding.ACT_ATTEND and r >= 1.0]
        masks = [(None, wl.heads)] * len(dense)
        if sparse:
            ws = ctx.workspace(len(sparse), device=dev)
            dm = binding.bitmask_to_dense(ws[1], wl.n_blocks).numpy()
            masks += [(dm[s], wl.heads) for s in range(len(sparse))]
        f, t = kept_flops_from_masks(masks, wl.n_tokens, wl.head_dim)
        flops_step.append(f)
        tiles_step.append(t)
        launches_img.append(len(sparse) + len(dense))
    assert ctx.last_status() == 0, "device status word is set"

    for i in range(args.warmup):
        one_step(i)
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ctx.profile(2)                     # an event pair around the attention kernel only: the roofline's duration
    ctx.profile_read()
    n0 = ctx.launch_count()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    e0.record()
    for i in range(args.steps):
        one_step(i)
    e1.record()
    torch.cuda.synchronize()
    w1 = time.time()
    if dist is not None:
        dist.barrier()
    ms_total = e0.elapsed_time(e1)
    launches = ctx.launch_count() - n0
    prof = ctx.profile_read()
    # the other kernels' durations come from a short pass of their own (an event pair around every launch
    # costs a few microseconds of stream time each, which the timed region should not carry four times per step)
    ctx.profile(1)
    n_side = max(len(plan), min(args.steps, 50))
    for i in range(n_side):
        one_step(i)
    torch.cuda.synchronize()
    prof_side = ctx.profile_read()
    ctx.profile(False)
    assert ctx.last_status() == 0, "device status word is set after the timed region"
    for kind in ("block_pool", "block_scores", "select_mask"):
        prof[kind] = prof_side[kind]
    if rank == 0:
        time.sleep(0.2)
        sampler.stop()
    flops_total = sum(flops_step[i % len(plan)] for i in range(args.steps))
    ms_total, flops_total, launches = aggregate(dist, dev, ms_total, flops_total, launches)
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
        for _ in range(n_e2e):
            up, down = ctx.rapid3_gated_step_host(hQ, hK, hV, hO, acts, ratios, wl.softmax_scale)
        a1.record()
        torch.cuda.synchronize()
        ms_e2e = a0.elapsed_time(a1)
        if dist is not None:
            t = torch.tensor([ms_e2e], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_e2e = float(t.item())
        e2e = {"value": world * flops_step[0] * n_e2e / (ms_e2e * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": int(up), "d2h_bytes_per_step": int(down), "ms_per_step": ms_e2e / n_e2e,
               "steps": n_e2e, "checksum": float(hO[0, 0, 0, :8].float().sum())}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    attn_ms, attn_n = prof["attention"]
    rank_flops = sum(flops_step[i % len(plan)] for i in range(args.steps))
    attn_avg_ms = attn_ms / max(1, attn_n)
    achieved = rank_flops / max(1, attn_n) / (attn_avg_ms * 1e-3) / 1e12 if attn_n else None
    peak = peaks["bf16_tflops_sustained"]
    traffic = ATTN_DRAM_BYTES_PER_LAUNCH.get(wl.name)
    roofline = {"bound": "tensor", "kernel": "attn_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                "peak_source": f"bf16_tflops_sustained of {peaks['source']}",
                "frac_of_burst_peak": (achieved / peaks["bf16_tflops"]) if achieved else None,
                "frac_of_nominal_2250": (achieved / 2250.0) if achieved else None,
                "avg_launch_ms": attn_avg_ms, "launches": attn_n}
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

    # time of the same attention kernel at one keep ratio for the whole batch: ratio 1.0 is the dense
    # reference, the others show how the time follows the kept-tile fraction
    sweep = None
    if not args.no_sweep and wl.steps == 1 and world == 1:
        sweep = []
        (Q, K, V) = sets[0]
        for r in (1.0, 0.5, 0.25):
            acts, ratios = [binding.ACT_ATTEND] * wl.batch, [r] * wl.batch
            for _ in range(3):
                ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
            torch.cuda.synchronize()
            if r < 1.0:
                dm = binding.bitmask_to_dense(ctx.workspace(wl.batch, device=dev)[1], wl.n_blocks).numpy()
                frac = float(dm.mean())
            else:
                frac = 1.0
            ctx.profile(True)
            ctx.profile_read()
            for _ in range(20):
                ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
            torch.cuda.synchronize()
            pr = ctx.profile_read()
            ctx.profile(False)
            step_ms = sum(v[0] for v in pr.values()) / 20.0
            sweep.append({"keep_ratio": r, "kept_tile_fraction": frac, "attention_ms": pr["attention"][0] / pr["attention"][1],
                          "all_kernels_ms": step_ms})
        for e in sweep:
            e["attention_speedup_vs_ratio_1"] = sweep[0]["attention_ms"] / e["attention_ms"]
            e["step_speedup_vs_ratio_1"] = sweep[0]["all_kernels_ms"] / e["all_kernels_ms"]

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

    cpu = None
    if not args.no_cpu_baseline and world == 1:          # the oracle is timed at N = 1 only
        v, secs, cores, desc = OracleSample(wl).run(args.cpu_budget)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "seconds": secs,
               "cpu_model": cpu_model(), "tiny_1thread_seconds": oracle_tiny_single_thread()}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "batch": wl.batch, "heads": wl.heads, "head_dim": wl.head_dim,
                       "n_text": wl.n_text, "n_image": wl.n_image, "keep_ratios": list(wl.keep_ratios),
                       "trajectory_steps": wl.steps, "kept_tiles_per_step": tiles_step[0],
                       "kept_flops_per_step": flops_step[0],
                       "l2": f"inputs larger than L2 ({3 * sets[0][0].numel() * 2 / 1e6:.0f} MB per set), "
                             f"{nsets} input sets rotated"},
            "clocks": sampler.summary(w0, w1), "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu, "kernels": kernels, "keep_ratio_sweep": sweep, "variants": variants}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


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
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    wl = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
