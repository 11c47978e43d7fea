#!/usr/bin/env python
"""Benchmark of the region-aware denoising step (RegionE hot path) on B200.

A "step" is one pass of the whole hot path over one batch of synthetic input of
the FLUX-Kontext-shaped workload (4096 image + 4096 reference + 512 text tokens,
24 heads x 128, two-ellipse 20 % edit mask): partition, row lists, gathers, RIKV
store, region attention with its rows scattered back, velocity decay + Euler, merge (7 library calls,
8 kernel launches on two streams).

Prints ONE JSON line (rank 0).  `value` = region-attention FLOPs of the step
divided by the whole step's device time (inputs resident in HBM).  `roofline`
covers the dominant kernel (the attention) timed by CUDA events inside the
same timed steps.  `--impl reference` times the fp64 CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "region-attention TFLOP/s over the whole region-aware denoise step"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                        bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                        source="measured")
        except Exception:
            pass
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# DRAM bytes per attention launch on config 2 (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture of this workload), valid for the kernel source with this digest only.
ATTENTION_TRAFFIC = dict(source_sha256_16="923074f802733a8a", config=2, dram_bytes_per_launch=229.5e6)


def recorded_traffic(cfg):
    """DRAM bytes per attention launch from the committed ncu summary, or None when the kernel source
    has changed since the counters were taken (or another workload is timed)."""
    import hashlib
    path = os.path.join(ROOT, "paper_2510_25590_b200", "csrc", "attention_tc.cu")
    try:
        digest = hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    if digest != ATTENTION_TRAFFIC["source_sha256_16"] or cfg != ATTENTION_TRAFFIC["config"]:
        return None
    return ATTENTION_TRAFFIC["dram_bytes_per_launch"]


def shard_requests(total: int, world_size: int, rank: int):
    """Contiguous shard of `total` independent requests for `rank` (no data-path collective)."""
    base, extra = divmod(total, world_size)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1]))
            except ValueError:
                continue
            for nme, val in zip(names, parts[3:7]):
                if val == "Active":
                    reasons.add(nme)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=sorted(reasons), samples=len(sm))


def attention_flops(n_q, n_kv, H, D):
    return float(4.0 * H * D * np.sum(n_q.astype(np.float64) * n_kv.astype(np.float64)))


def make_workload(cfg: int, stream: int):
    from paper_2510_25590_b200 import synth
    wl = synth.WORKLOADS[cfg]
    lat = synth.make_latents(wl, stream=stream)
    qkv = synth.make_qkv_full(wl, stream=stream)
    return wl, lat, qkv


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def time_oracle(wl, lat, qkv, heads, steps, warmup):
    from oracle import step_oracle
    t, scale, dt, dt_u = lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0
    times = []
    res = None
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        res = step_oracle.region_step(wl, lat, qkv, t, scale, dt, dt_u, heads=heads)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    n_kv = res["n_q"] + res["n_cache"]
    flops = attention_flops(res["n_q"], n_kv, heads, wl.head_dim)
    return flops, float(np.mean(times))


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        n = 1
    try:
        n = min(n, len(os.sched_getaffinity(0)))
    except Exception:
        pass
    return int(n)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = args.config
    wl, lat, qkv = make_workload(cfg, 0)
    heads = wl.heads
    steps = 3 if args.steps is None else max(1, min(args.steps, 20))
    warmup = 1 if args.warmup is None else max(0, min(args.warmup, 3))
    flops, sec = time_oracle(wl, lat, qkv, heads, steps, warmup)
    val = flops / sec / 1e12
    cores = host_threads()
    sample = (f"whole step on config {cfg} ({wl.name}) with the attention restricted to {heads} of "
              f"{wl.heads} heads; all other stages at full size")
    line = dict(metric=METRIC, value=val, unit=UNIT, impl="reference", n_gpus=args.gpus, steps=steps,
                warmup=warmup, ms_per_step=sec * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=f"config {cfg}: {wl.name}", sample=sample),
                cpu_baseline=dict(value=val, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def hbm_sweep(torch, binding, step, d, flush_l2, peak_gbs, iters=10):
    """Achieved GB/s (algorithmic bytes / CUDA-event time, untimed L2 flush before each launch) of the
    memory-bound kernels on instances large enough for the figure to mean HBM bandwidth: the cache
    store and a 6 KB-row gather at the bench workload's size, and partition / velocity decay / merge
    at 2^21 tokens of 16 channels (32 requests of 65536 tokens)."""
    bf, i32 = torch.bfloat16, torch.int32
    out = []

    def timed(name, nbytes, fn):
        for _ in range(2):
            fn()
        ts = []
        for _ in range(iters):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e-3)
        sec = float(np.median(ts))
        out.append(dict(kernel=name, mbytes=round(nbytes / 1e6, 1), us=round(sec * 1e6, 1),
                        gbs=round(nbytes / sec / 1e9, 0), frac_of_measured=round(nbytes / sec / 1e9 / peak_gbs, 3)))

    s = step.shp
    row = s.H * s.D * 2
    n_cache = int(step.n_cache.sum().item())
    timed("rikv_store (bench workload)", n_cache * (4 * row + 4),
          lambda: binding.rikv_store(d["k"], d["vv"], step.cache_rows, step.n_cache, step.k_cache, step.v_cache))
    # the same store at config 5's size (4 requests, 17562 of 18944 rows kept each): 1.7 GB, long enough
    # that the ramp and the tail of the launch no longer count
    gs5 = torch.Generator(device="cuda"); gs5.manual_seed(12)
    k5 = torch.empty((4, 18944, s.H, s.D), dtype=bf, device="cuda").normal_(generator=gs5)
    v5 = torch.empty((4, 18944, s.H, s.D), dtype=bf, device="cuda").normal_(generator=gs5)
    keep5 = torch.stack([torch.randperm(18944, device="cuda", generator=gs5)[:17562].sort()[0] for _ in range(4)]).to(i32).contiguous()
    n5 = torch.full((4,), 17562, dtype=i32, device="cuda")
    kc5 = torch.empty((4, 17562, s.H, s.D), dtype=bf, device="cuda"); vc5 = torch.empty_like(kc5)
    timed("rikv_store (config 5's size)", 4 * 17562 * (4 * row + 4),
          lambda: binding.rikv_store(k5, v5, keep5, n5, kc5, vc5))
    del k5, v5, kc5, vc5
    rows, src_rows = 16384, 32768                           # 100 MB read + 100 MB written, every row once
    gs = torch.Generator(device="cuda"); gs.manual_seed(11)
    src = torch.empty((1, src_rows, s.H, s.D), dtype=bf, device="cuda").normal_(generator=gs)
    idx = torch.randperm(src_rows, device="cuda", generator=gs)[:rows].sort()[0].to(i32).reshape(1, rows).contiguous()
    n_rows = torch.full((1,), rows, dtype=i32, device="cuda")
    dst = torch.empty((1, rows, s.H, s.D), dtype=bf, device="cuda")
    timed("gather of 16384 distinct rows of 6 KB", rows * (2 * row + 4),
          lambda: binding.gather(src, idx, n_rows, dst))
    del src, dst
    B, N, C = 32, 65536, 16
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    ref = torch.randn((B, N, C), device="cuda", generator=g).to(bf)
    # edit regions are spatially coherent, as in the paper's workloads: one ellipse per request on the
    # 256 x 256 token grid covering 20 % of it, centre shifted from request to request; edited tokens get
    # an estimate opposite to the reference (cosine -1), the others the reference itself (cosine +1)
    side = 256
    yy, xx = torch.meshgrid(torch.arange(side, device="cuda"), torch.arange(side, device="cuda"), indexing="ij")
    ax, ay = 0.36 * side, 0.2 * side / (3.14159265 * 0.36)
    blobs = []
    for b in range(B):
        cx, cy = side * (0.4 + 0.2 * ((b * 7) % 10) / 10), side * (0.4 + 0.2 * ((b * 3) % 10) / 10)
        blobs.append((((xx - cx) / ax) ** 2 + ((yy - cy) / ay) ** 2 < 1.0).reshape(N))
    blob = torch.stack(blobs)
    x_t = torch.where(blob[:, :, None], -ref, ref)
    v = torch.zeros_like(ref)
    mask = torch.empty((B, N), dtype=torch.uint8, device="cuda")
    e, k, sl = (torch.empty((B, N), dtype=i32, device="cuda") for _ in range(3))
    ne = torch.empty(B, dtype=i32, device="cuda")
    timed("partition, 2^21 tokens", B * N * (3 * C * 2 + 9),
          lambda: binding.partition(x_t, v, ref, 0.7, binding.METRIC_COSINE, 0.1, mask, e, k, sl, ne))
    n_e = int(ne.sum().item())
    assert n_e == int(blob.sum().item()), (n_e, int(blob.sum().item()))
    x_e = torch.zeros((B, N, C), dtype=bf, device="cuda"); v_e = torch.zeros_like(x_e); v_c = torch.zeros_like(x_e)
    n_all = torch.full((B,), N, dtype=i32, device="cuda")          # every row live: traffic well above L2
    timed("velocity_decay with cache refresh", B * N * 4 * C * 2,
          lambda: binding.velocity_decay(v_e, 1.0, 1.0 / 28, x_e, n_all, v_cache_out=v_c))
    timed("velocity_decay reusing the cache", B * N * 3 * C * 2,
          lambda: binding.velocity_decay(v_e, 0.9, 1.0 / 28, x_e, n_all))
    x_out = torch.empty_like(x_t)
    timed(f"merge, 2^21 tokens, elliptic regions ({100.0 * n_e / (B * N):.0f} % edited)",
          (B * N - n_e) * (3 * C * 2 + 4) + n_e * (2 * C * 2 + 4),
          lambda: binding.merge(x_t, v, x_e, sl, 5.0 / 28, x_out))
    # worst case for the merge: every token edited or not independently of its neighbours (random
    # latents against the threshold), so the reads of the unedited rows skip single 32-byte rows
    x_r, v_r = (torch.randn((B, N, C), device="cuda", generator=g).to(bf) for _ in range(2))
    binding.partition(x_r, v_r, ref, 0.7, binding.METRIC_COSINE, 0.1, mask, e, k, sl, ne)
    n_r = int(ne.sum().item())
    timed(f"merge, 2^21 tokens, per-token random mask ({100.0 * n_r / (B * N):.0f} % edited)",
          (B * N - n_r) * (3 * C * 2 + 4) + n_r * (2 * C * 2 + 4),
          lambda: binding.merge(x_r, v_r, x_e, sl, 5.0 / 28, x_out))
    return out


def ratio_sweep(torch, binding, synth, flush_l2, to_dev, steps=20):
    """Denoise-step time against the edit-mask ratio on the Qwen-Image-Edit-shaped workload (config 3):
    one region step (7 library calls, 8 launches) and its attention call per ratio, CUDA events, L2
    flushed per step."""
    from paper_2510_25590_b200.step import RegionStep, StepShapes, plan_capacity
    wl = synth.WORKLOADS[3]
    qkv = synth.make_qkv_full(wl)
    dq, dk, dv = (to_dev(qkv[k]) for k in ("q", "k", "v"))
    out = []
    for ratio in wl.ratios:
        lat = synth.make_latents(wl, ratio)
        x_t, v, ref = (to_dev(lat[k]) for k in ("x_t", "v", "ref"))
        cap = plan_capacity(x_t, v, ref, lat["t"], binding.METRIC_COSINE, wl.threshold)
        step = RegionStep(StepShapes(wl.batch, wl.n_img, wl.n_text, wl.n_ref, wl.channels, wl.heads,
                                     wl.head_dim, cap, binding.METRIC_COSINE, wl.threshold))
        run = lambda: step.run(x_t, v, ref, dq, dk, dv, lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0)
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
        for i in range(steps):
            flush_l2()
            step.attention_events = (ev[i][1], ev[i][2])
            ev[i][0].record(); run(); ev[i][3].record()
        torch.cuda.synchronize()
        step.attention_events = None
        assert int(step.dev_status[0]) == 0
        n_q = int(step.n_q[0]); n_kv = n_q + int(step.n_cache[0])
        st_us = float(np.mean([e[0].elapsed_time(e[3]) for e in ev]) * 1e3)
        at_us = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]) * 1e3)
        fl = 4.0 * wl.heads * wl.head_dim * n_q * n_kv
        out.append(dict(ratio=ratio, n_q=n_q, n_kv=n_kv, step_us=round(st_us, 1), attention_us=round(at_us, 1),
                        attention_tflops=round(fl / at_us / 1e6, 1)))
        del step
    return out


def per_config_rows(torch, binding, synth, flush_l2, to_dev, peaks, steps=12):
    """The other configurations beside the headline one, each timed like it (CUDA events, L2 flushed
    before every step): the tiny layer (config 1), the Step1X-Edit-shaped attention layer with the
    paper's membership and the L2 partition (config 4's shape) and the batch of four large requests
    (config 5); then config 4's 28-step loop, library calls only."""
    from paper_2510_25590_b200.step import RegionStep, StepShapes, plan_capacity
    rows = []
    for cfg, membership in ((1, "edited_queries"), (4, "paper"), (5, "edited_queries")):
        wl = synth.WORKLOADS[cfg]
        lat = synth.make_latents(wl)
        qkv = synth.make_qkv_full(wl)
        x_t, v, ref = (to_dev(lat[k]) for k in ("x_t", "v", "ref"))
        dq, dk, dv = (to_dev(qkv[k]) for k in ("q", "k", "v"))
        del qkv
        metric = binding.METRIC_COSINE if wl.metric == "cosine" else binding.METRIC_L2
        cap = plan_capacity(x_t, v, ref, lat["t"], metric, wl.threshold)
        step = RegionStep(StepShapes(wl.batch, wl.n_img, wl.n_text, wl.n_ref, wl.channels, wl.heads,
                                     wl.head_dim, cap, metric, wl.threshold,
                                     binding.ROWS_PAPER if membership == "paper" else binding.ROWS_EDITED_QUERIES))
        run = lambda: step.run(x_t, v, ref, dq, dk, dv, lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0)
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
        for i in range(steps):
            flush_l2()
            step.attention_events = (ev[i][1], ev[i][2])
            ev[i][0].record(); run(); ev[i][3].record()
        torch.cuda.synchronize()
        step.attention_events = None
        assert int(step.dev_status[0]) == 0
        n_q = step.n_q.cpu().numpy(); n_kv = n_q + step.n_cache.cpu().numpy()
        fl = attention_flops(n_q, n_kv, wl.heads, wl.head_dim)
        st_us = float(np.mean([e[0].elapsed_time(e[3]) for e in ev]) * 1e3)
        at_us = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]) * 1e3)
        tf = fl / at_us / 1e6
        # the same step without the cache store: Algorithm 1 writes the cache at full steps only, a run of
        # region steps in between reuses it
        reuse = []
        for i in range(steps):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            step.run(x_t, v, ref, dq, dk, dv, lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0, store_cache=False)
            b.record()
            reuse.append((a, b))
        torch.cuda.synchronize()
        reuse_us = float(np.mean([a.elapsed_time(b) for a, b in reuse]) * 1e3)
        graph_us = None
        if cfg == 1:
            # the tiny layer's step is launch-bound (8 kernels of a few microseconds each): the same step
            # captured once into a CUDA graph and replayed shows the device time without the host's
            # launch path in between
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    step.run(x_t, v, ref, dq, dk, dv, lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0, stream=side)
            torch.cuda.synchronize()
            ts = []
            for _ in range(steps):
                flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); graph.replay(); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b) * 1e3)
            graph_us = round(float(np.median(ts)), 1)
            assert int(step.dev_status[0]) == 0
        rows.append(dict(config=cfg, workload=wl.name, membership=membership, batch=wl.batch,
                         n_q=int(n_q[0]), n_kv=int(n_kv[0]), heads=wl.heads, head_dim=wl.head_dim,
                         step_us=round(st_us, 1), step_us_cache_reused=round(reuse_us, 1),
                         step_us_cuda_graph=graph_us,
                         attention_us=round(at_us, 1), attention_tflops=round(tf, 1),
                         attention_frac_of_measured_burst=round(tf / peaks["bf16_tflops"], 3),
                         attention_frac_of_nominal_2250=round(tf / NOMINAL_BF16_TFLOPS, 3),
                         step_tflops_equivalent=round(fl / st_us / 1e6, 1)))
        del step, dq, dk, dv
        torch.cuda.empty_cache()
    rows.append(full_step_row(torch, binding, synth, flush_l2, to_dev, peaks))
    rows.append(kv_e4m3_row(torch, binding, synth, flush_l2, to_dev, peaks))
    rows.append(fresh_qkv_row(torch, binding, synth, flush_l2, to_dev, peaks))
    rows.append(loop_row(torch, binding, synth, to_dev))
    rows.append(stack_loop_row(torch, binding, synth, to_dev))
    return rows


def full_step_row(torch, binding, synth, flush_l2, to_dev, peaks, iters=10):
    """The forced full step on the Qwen-Image-Edit-shaped layer (8448 joint rows, 24 heads x 128, the
    cache keeps text + unedited + reference rows of the 25 % mask): plain joint attention followed by
    the RIKV store as two calls, against the one call that writes the cache from the staged tiles."""
    wl = synth.WORKLOADS[3]
    lat = synth.make_latents(wl, 0.25)
    qkv = synth.make_qkv_full(wl)
    q, k, v = (to_dev(qkv[x]) for x in ("q", "k", "v"))
    del qkv
    n, H, D, N = wl.n_full, wl.heads, wl.head_dim, wl.n_img
    i32, bf = torch.int32, torch.bfloat16
    # the rows to retain come from the library's own partition and row lists
    mask = torch.empty((1, N), dtype=torch.uint8, device="cuda")
    e_idx, k_idx, slot = (torch.empty((1, N), dtype=i32, device="cuda") for _ in range(3))
    n_edit, n_query, n_keep = (torch.zeros(1, dtype=i32, device="cuda") for _ in range(3))
    query_rows = torch.zeros((1, n), dtype=i32, device="cuda")
    keep = torch.zeros((1, n), dtype=i32, device="cuda")
    binding.partition_rows(to_dev(lat["x_t"]), to_dev(lat["v"]), to_dev(lat["ref"]), lat["t"],
                           binding.METRIC_COSINE, wl.threshold, mask, e_idx, k_idx, slot, n_edit,
                           wl.n_text, wl.n_ref, binding.ROWS_EDITED_QUERIES, query_rows, n_query, keep, n_keep)
    kept = int(n_keep[0])
    n_rows = torch.tensor([n], dtype=i32, device="cuda"); zero = torch.zeros(1, dtype=i32, device="cuda")
    kc = torch.empty((1, n, H, D), dtype=bf, device="cuda"); vc = torch.empty_like(kc)
    out = torch.empty_like(q)
    ws = torch.empty(max(binding.full_attention_store_workspace(1, n, H, D), 256), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=i32, device="cuda")

    def two_calls():
        binding.region_attention(q, k, v, None, None, n_rows, n_rows, zero, out, workspace=ws, dev_status=st)
        binding.rikv_store(k, v, keep, n_keep, kc, vc, dev_status=st)

    def one_call():
        binding.full_attention_store(q, k, v, n_rows, keep, n_keep, kc, vc, out, workspace=ws, dev_status=st)

    res = {}
    for name, fn in (("attention_then_rikv_store_us", two_calls), ("full_attention_store_us", one_call)):
        for _ in range(2):
            fn()
        ts = []
        for _ in range(iters):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3)
        res[name] = round(float(np.median(ts)), 1)
    assert int(st[0]) == 0
    fl = 4.0 * H * D * n * n
    res.update(workload="config 3 shape, forced full step with cache refresh", rows=n, kept_rows=kept,
               full_attention_store_tflops=round(fl / res["full_attention_store_us"] / 1e6, 1),
               frac_of_measured_burst=round(fl / res["full_attention_store_us"] / 1e6 / peaks["bf16_tflops"], 3))
    return res


def kv_e4m3_row(torch, binding, synth, flush_l2, to_dev, peaks, iters=10):
    """The 8-bit (E4M3) variant of the cache on the headline layer's shape and on the batch of four large
    requests: the store that quantises the retained rows, the pass that widens them back to bf16 before a
    region step's attention, both as HBM passes against the measured copy bandwidth, and the bytes one
    cached layer holds in either form."""
    i32, bf = torch.int32, torch.bfloat16
    out = dict(workload="one layer's retained rows: bf16 store, E4M3 store, E4M3 widening", sizes=[])
    for cfg in (2, 5):
        wl = synth.WORKLOADS[cfg]
        qkv = synth.make_qkv_full(wl)
        k, v = to_dev(qkv["k"]), to_dev(qkv["v"])
        del qkv
        B, n, H, D = wl.batch, wl.n_full, wl.heads, wl.head_dim
        kept = n - int(round(wl.ratios[0] * wl.n_img))
        keep = (torch.arange(kept, dtype=i32, device="cuda") + (n - kept)).repeat(B, 1).contiguous()
        n_keep = torch.full((B,), kept, dtype=i32, device="cuda")
        kq = torch.empty((B, kept, H, D), dtype=torch.uint8, device="cuda"); vq = torch.empty_like(kq)
        ks = torch.empty((B, kept, H), dtype=torch.float32, device="cuda"); vs = torch.empty_like(ks)
        kc = torch.empty((B, kept, H, D), dtype=bf, device="cuda"); vc = torch.empty_like(kc)
        st = torch.zeros(1, dtype=i32, device="cuda")
        rows = B * kept
        calls = (("rikv_store_bf16", 2 * 2 * 2 * rows * H * D,
                  lambda: binding.rikv_store(k, v, keep, n_keep, kc, vc, dev_status=st)),
                 ("rikv_store_e4m3", 2 * rows * H * (3 * D + 4),
                  lambda: binding.rikv_store_e4m3(k, v, keep, n_keep, kq, vq, ks, vs, dev_status=st)),
                 ("rikv_load_e4m3", 2 * rows * H * (3 * D + 4),
                  lambda: binding.rikv_load_e4m3(kq, vq, ks, vs, n_keep, kc, vc, dev_status=st)))
        res = dict(config=cfg, requests=B, kept_rows=kept, cache_bytes_bf16=2 * 2 * rows * H * D,
                   cache_bytes_e4m3=2 * rows * H * (D + 4))
        for name, nbytes, fn in calls:
            for _ in range(3):
                fn()
            ts = []
            for _ in range(iters):
                flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b) * 1e3)
            us = float(np.median(ts))
            res[name] = dict(us=round(us, 1), algorithmic_bytes=nbytes, gbs=round(nbytes / us / 1e3, 1),
                             frac_of_measured_hbm=round(nbytes / us / 1e3 / peaks["hbm_gbs"], 3))
        assert int(st[0]) == 0
        out["sizes"].append(res)
        del k, v, kq, vq, kc, vc
        torch.cuda.empty_cache()
    return out


def fresh_qkv_row(torch, binding, synth, flush_l2, to_dev, peaks, iters=10):
    """The producer of fresh Q / K / V rows (gather + per-head RMS normalisation + rotary embedding in one
    pass) beside the plain gather of the same rows: at the headline layer's region step (819 rows) and as
    an HBM pass over every row of config 5's batch (what a full step's producer moves)."""
    i32, bf = torch.int32, torch.bfloat16
    out = dict(workload="fresh Q/K/V rows: plain gather of three tensors, and gather + RMS norm + rotary embedding", sizes=[])
    for cfg, all_rows in ((2, False), (5, True)):
        wl = synth.WORKLOADS[cfg]
        qkv = synth.make_qkv_full(wl)
        q, k, v = (to_dev(qkv[x]) for x in ("q", "k", "v"))
        del qkv
        B, n, H, D = wl.batch, wl.n_full, wl.heads, wl.head_dim
        rows = n if all_rows else int(round(wl.ratios[0] * wl.n_img))
        idx = (torch.arange(rows, dtype=i32, device="cuda") + (0 if all_rows else wl.n_text)).repeat(B, 1).contiguous()
        cnt = torch.full((B,), rows, dtype=i32, device="cuda")
        pos = torch.arange(n, dtype=torch.float64, device="cuda")[:, None]
        inv = 10000.0 ** (-torch.arange(D // 2, dtype=torch.float64, device="cuda") * 2.0 / D)
        cos, sin = torch.cos(pos * inv).float().contiguous(), torch.sin(pos * inv).float().contiguous()
        w = torch.ones(D, dtype=bf, device="cuda")
        dq, dk, dv = (torch.empty((B, rows, H, D), dtype=bf, device="cuda") for _ in range(3))
        st = torch.zeros(1, dtype=i32, device="cuda")
        nbytes = B * rows * (3 * 2 * H * D * 2 + 4 + 2 * (D // 2) * 4)
        calls = (("gather_multi", lambda: binding.gather_multi([q, k, v], idx, cnt, [dq, dk, dv], dev_status=st)),
                 ("fresh_qkv", lambda: binding.fresh_qkv(q, k, v, idx, cnt, w, w, 1e-6, cos, sin, binding.ROPE_INTERLEAVED,
                                                         dq, dk, dv, dev_status=st)))
        res = dict(config=cfg, requests=B, rows=rows, heads=H, head_dim=D, algorithmic_bytes=nbytes)
        for name, fn in calls:
            for _ in range(3):
                fn()
            ts = []
            for _ in range(iters):
                flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b) * 1e3)
            us = float(np.median(ts))
            res[name] = dict(us=round(us, 1), gbs=round(nbytes / us / 1e3, 1),
                             frac_of_measured_hbm=round(nbytes / us / 1e3 / peaks["hbm_gbs"], 3))
        assert int(st[0]) == 0
        out["sizes"].append(res)
        del q, k, v, dq, dk, dv
        torch.cuda.empty_cache()
    return out


def loop_row(torch, binding, synth, to_dev):
    """Config 4's sampler loop (4096 tokens x 16 channels, L2 partition after step 6, cache refresh every
    5 steps, alternate region steps reused: 28 steps): device time of the library calls alone.  The
    velocity model is scaffold around the path, so its outputs are recorded in a first pass and replayed
    from memory in the timed passes (no model kernel runs inside them); the host decisions depend on the
    schedule only, so the whole loop is also captured once into a CUDA graph and replayed."""
    from paper_2510_25590_b200 import loop as gloop
    wl = synth.WORKLOADS[4]
    lat = synth.make_latents(wl, stream=4)
    rng = np.random.default_rng(4)
    m = lat["mask"].astype(bool)
    ref_h = lat["ref"]
    target = to_dev(synth.bf16_round(np.where(m[..., None], rng.standard_normal(ref_h.shape), ref_h).astype(np.float32))).float()
    noise = to_dev(synth.bf16_round(rng.standard_normal(ref_h.shape).astype(np.float32)))
    ref = to_dev(ref_h)
    kinds, after = gloop.alternating_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    cfg = gloop.LoopConfig(kinds, after, ts, [1.0] * (T + 1), 0.05, binding.METRIC_L2, wl.threshold)
    B, N, C = noise.shape
    lp = gloop.RegionELoop(B, N, C, cfg)

    class Recording:
        def __init__(self):
            self.full_out, self.region_out = [], []

        def full(self, x, t, store):
            self.full_out.append(((x.float() - target) / t).to(x.dtype))
            return self.full_out[-1]

        def region(self, x_e, t, edit_idx, n_edit):
            idx = edit_idx.long().clamp(0, N - 1)
            tgt = torch.gather(target, 1, idx.unsqueeze(-1).expand(B, x_e.shape[1], C))
            self.region_out.append(((x_e.float() - tgt) / t).to(x_e.dtype))
            return self.region_out[-1]

    class Replay:
        def __init__(self, rec):
            self.rec, self.i, self.j = rec, 0, 0

        def full(self, x, t, store):
            self.i += 1
            return self.rec.full_out[self.i - 1]

        def region(self, x_e, t, edit_idx, n_edit):
            self.j += 1
            return self.rec.region_out[self.j - 1]

    rec = Recording()
    x = noise.clone()
    _, trace = lp.run(x, ref, rec)
    torch.cuda.synchronize()
    assert int(lp.dev_status[0]) == 0

    def replay_once():
        x.copy_(noise)
        return lp.run(x, ref, Replay(rec))

    eager = []
    for i in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        x.copy_(noise)
        a.record(); lp.run(x, ref, Replay(rec)); b.record()
        torch.cuda.synchronize()
        eager.append(a.elapsed_time(b) * 1e3)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            lp.run(x, ref, Replay(rec), stream=side)
    torch.cuda.synchronize()
    graphed = []
    for i in range(10):
        x.copy_(noise)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); graph.replay(); b.record()
        torch.cuda.synchronize()
        graphed.append(a.elapsed_time(b) * 1e3)
    n_reuse = sum(1 for s_ in trace.steps if s_[2] == "reuse")
    return dict(config=4, workload=wl.name + ": 28-step loop, library calls only", schedule=kinds,
                image_tokens=N, channels=C, full_steps=kinds.count("F"), region_steps=kinds.count("R"),
                reused_region_steps=n_reuse, library_launches=trace.launches,
                loop_us_eager_python=round(float(np.median(eager)), 1),
                loop_us_cuda_graph=round(float(np.median(graphed)), 1),
                us_per_launch_cuda_graph=round(float(np.median(graphed)) / max(trace.launches, 1), 2))


def stack_loop_row(torch, binding, synth, to_dev, blocks=8):
    """The sampler-loop configuration at its stated size: the 28-step loop around a stand-in stack of 8 random blocks
    (hidden 3072, 24 heads x 128, MLP ratio 4; 256 text + 4096 image + 4096 reference tokens), once with
    every step a full step and once under the region-aware schedule (partition after step 6 with the L2
    threshold, cache refreshed every 5 steps, alternate region steps reused).  The blocks' GEMMs,
    normalisations and activations are scaffold (torch); the Q / K / V producer, every attention, every
    cache store and all latent updates are library calls.  Device time by CUDA events around the loop."""
    from paper_2510_25590_b200 import loop as gloop
    from paper_2510_25590_b200.mmdit_scaffold import MMDiTScaffold
    wl = synth.WORKLOADS[4]
    hidden, H, D, C = wl.heads * wl.head_dim, wl.heads, wl.head_dim, wl.channels
    lat = synth.make_latents(wl, stream=4)
    gen = torch.Generator(device="cuda"); gen.manual_seed(4)
    w = {}
    for name, (shape, std, mean) in synth.mmdit_weight_shapes(hidden, D, C, wl.n_text, blocks).items():
        w[name] = (mean + std * torch.randn(shape, device="cuda", generator=gen)).to(torch.bfloat16)
    cos, sin = (torch.from_numpy(a).cuda() for a in synth.rope_tables(wl.n_full, D))
    ref = to_dev(lat["ref"])
    planted = torch.from_numpy(lat["mask"].astype(bool)).cuda()
    model = MMDiTScaffold(w, wl.n_text, wl.n_img, wl.n_ref, H, D, blocks, cos, sin, ref, planted, binding.ROWS_PAPER)
    noise = (torch.randn(ref.shape, device="cuda", generator=gen)).to(torch.bfloat16)
    kinds, after = gloop.alternating_schedule()
    T = len(kinds)
    ts = [1.0 - k / T for k in range(T + 1)]
    res = dict(workload="config 4: 28-step loop around 8 stand-in blocks (scaffold GEMMs by torch, path by the library)",
               blocks=blocks, hidden=hidden, rows=wl.n_full, schedule=kinds)
    for label, k_, after_ in (("all_full", "F" * T, T + 1), ("region_aware", kinds, after)):
        cfg = gloop.LoopConfig(k_, after_, ts, [1.0] * (T + 1), 0.05, binding.METRIC_L2, wl.threshold)
        lp = gloop.RegionELoop(1, wl.n_img, C, cfg)
        model.bind(lp)
        times = []
        for it in range(2):                                  # the first pass warms up (GEMM plans, kernel set-up)
            x = noise.clone()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); _, trace = lp.run(x, ref, model); b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        assert int(lp.dev_status[0]) == 0 and int(model.dev_status[0]) == 0
        res[label] = dict(loop_ms=round(times[-1], 1), model_full_calls=trace.model_full_calls,
                          model_region_calls=trace.model_region_calls)
        if label == "region_aware":
            res[label]["edited_tokens"] = int(lp.n_edit[0])
            res[label]["mask_recovered"] = bool(torch.equal(lp.mask.bool(), planted))
    res["speedup_region_aware_over_all_full"] = round(res["all_full"]["loop_ms"] / res["region_aware"]["loop_ms"], 2)
    del model, w
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2510_25590_b200 import binding, build as _build, synth
    from paper_2510_25590_b200.step import RegionStep, StepShapes, plan_capacity

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    binding.load()

    steps = 3000 if args.steps is None else args.steps
    warmup = 10 if args.warmup is None else max(3, args.warmup)
    cfg = args.config
    # weak scaling: every rank owns its own request(s) (a different seed stream), no exchange
    wl, lat, qkv = make_workload(cfg, shard_requests(world, world, rank)[0])
    bf = torch.bfloat16

    def dev(a):
        bits = synth.f32_to_bf16_bits(a).reshape(a.shape)
        return torch.from_numpy(bits.view(np.int16)).cuda().view(bf)

    def pinned(a):
        bits = synth.f32_to_bf16_bits(a).reshape(a.shape)
        return torch.from_numpy(bits.view(np.int16)).view(bf).pin_memory()

    host = {k: pinned(v) for k, v in (("x_t", lat["x_t"]), ("v", lat["v"]), ("ref", lat["ref"]),
                                      ("q", qkv["q"]), ("k", qkv["k"]), ("vv", qkv["v"]))}
    d = {k: v.cuda() for k, v in host.items()}
    t, scale, dt, dt_u = lat["t"], 0.97, 1.0 / 28.0, 5.0 / 28.0
    metric = binding.METRIC_COSINE if wl.metric == "cosine" else binding.METRIC_L2
    cap = plan_capacity(d["x_t"], d["v"], d["ref"], t, metric, wl.threshold)
    shp = StepShapes(wl.batch, wl.n_img, wl.n_text, wl.n_ref, wl.channels, wl.heads, wl.head_dim, cap,
                     metric, wl.threshold)
    step = RegionStep(shp)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # > 126 MB L2
    drain = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def flush_l2():
        """Writes 256 MiB (evicts everything), then reads another 256 MiB so that the dirty lines of
        that write are back in HBM before the timed work starts: L2 is cold and clean."""
        flush.zero_()
        drain.view(torch.int32).max()

    def one():
        step.run(d["x_t"], d["v"], d["ref"], d["q"], d["k"], d["vv"], t, scale, dt, dt_u)

    for _ in range(warmup):
        one()
    torch.cuda.synchronize()
    assert int(step.dev_status[0]) == 0, binding.status_string(int(step.dev_status[0]))
    n_q = step.n_q.cpu().numpy()
    n_kv = n_q + step.n_cache.cpu().numpy()
    flops = attention_flops(n_q, n_kv, wl.heads, wl.head_dim)

    # ---- timed region: K steps, L2 flushed before each, per-step and per-attention events ----
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    aev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    sampler = ClockSampler(local)
    launches0 = step.launches
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    wall0 = time.perf_counter()
    for i in range(steps):
        flush_l2()
        step.attention_events = aev[i]
        ev[i][0].record()
        one()
        ev[i][1].record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()
    step.attention_events = None
    launches = step.launches - launches0
    step_ms = np.array([a.elapsed_time(b) for a, b in ev])
    attn_ms = np.array([a.elapsed_time(b) for a, b in aev])
    total_ms = float(step_ms.sum())
    if world > 1:
        tt = torch.tensor([total_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
    ms_per_step = total_ms / steps
    value = world * flops / (ms_per_step * 1e-3) / 1e12

    # ---- end to end: pinned host inputs -> device, the step, result -> host, every step ----
    e2e_steps = max(3, min(steps, 50))
    out_host = torch.empty_like(step.x_out, device="cpu").pin_memory()
    o_host = torch.empty_like(step.o_e, device="cpu").pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    d2h = out_host.numel() * 2 + o_host.numel() * 2
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def one_e2e():
        for k in host:
            d[k].copy_(host[k], non_blocking=True)
        one()
        # the step leaves the attention rows at their joint-sequence positions; the host wants them dense
        binding.gather(step.o_full, step.query_rows, step.n_q, step.o_e, dev_status=step.dev_status)
        out_host.copy_(step.x_out, non_blocking=True)
        o_host.copy_(step.o_e, non_blocking=True)

    for _ in range(2):
        one_e2e()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0.record()
    for _ in range(e2e_steps):
        one_e2e()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        tt = torch.tensor([e2e_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        e2e_ms = float(tt.item())
    e2e_val = world * flops / (e2e_ms / e2e_steps * 1e-3) / 1e12

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # the headline step without its cache store (a region step between two full steps of Algorithm 1)
    reuse = []
    for _ in range(min(steps, 50)):
        flush_l2()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        step.run(d["x_t"], d["v"], d["ref"], d["q"], d["k"], d["vv"], t, scale, dt, dt_u, store_cache=False)
        b.record()
        reuse.append((a, b))
    torch.cuda.synchronize()
    reuse_us = float(np.mean([a.elapsed_time(b) for a, b in reuse]) * 1e3)

    peaks = measured_peaks()
    hbm_kernels = None
    if world == 1 and not args.no_hbm_sweep:
        hbm_kernels = hbm_sweep(torch, binding, step, d, flush_l2, peaks["hbm_gbs"])
    step_vs_ratio = None
    if world == 1 and not args.no_ratio_sweep:
        step_vs_ratio = ratio_sweep(torch, binding, synth, flush_l2, dev)
    per_config = None
    if world == 1 and not args.no_per_config:
        per_config = per_config_rows(torch, binding, synth, flush_l2, dev, peaks)
    attn_us = float(np.mean(attn_ms) * 1e3)
    achieved = flops / (attn_us * 1e-6) / 1e12
    roofline = dict(bound="tensor", achieved=achieved, peak=peaks["bf16_tflops"], unit="TFLOP/s",
                    frac=achieved / peaks["bf16_tflops"], traffic=recorded_traffic(cfg),
                    kernel=f"region_attention_tc_kernel<{wl.head_dim}> (+ merge of shared items)",
                    us_per_launch=attn_us,
                    peak_source=f"bf16_tflops (burst) of {peaks['source']}",
                    frac_of_nominal_2250=achieved / NOMINAL_BF16_TFLOPS)

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        heads = wl.heads
        fl, sec = time_oracle(wl, lat, qkv, heads, 2, 1)
        cpu_baseline = dict(value=fl / sec / 1e12, unit=UNIT, cores=host_threads(), kind="oracle",
                            sample=f"whole step on config {cfg} with the attention restricted to {heads} of "
                                   f"{wl.heads} heads ({sec:.2f} s per step); other stages at full size")

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=steps, warmup=warmup,
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16", data="synthetic",
                config=dict(workload=f"config {cfg}: {wl.name}", batch=wl.batch, image_tokens=wl.n_img,
                            reference_tokens=wl.n_ref, text_tokens=wl.n_text, heads=wl.heads,
                            head_dim=wl.head_dim, n_q=int(n_q[0]), n_kv=int(n_kv[0]),
                            cache_policy="L2 flushed before every timed step (256 MiB written, then 256 MiB read to drain the dirty lines)",
                            parallelism=f"replicas x{world} (independent requests, no collective)"),
                clocks=clocks,
                e2e=dict(value=e2e_val, unit=UNIT, h2d_bytes_per_step=int(h2d), d2h_bytes_per_step=int(d2h),
                         steps=e2e_steps, ms_per_step=e2e_ms / e2e_steps),
                gpu_launches=int(launches), roofline=roofline, cpu_baseline=cpu_baseline,
                hbm_kernels=hbm_kernels, denoise_step_us_vs_mask_ratio=step_vs_ratio, per_config=per_config,
                step_us=dict(mean=float(step_ms.mean() * 1e3), min=float(step_ms.min() * 1e3),
                             median=float(np.median(step_ms) * 1e3)),
                attention_us=dict(mean=attn_us, min=float(attn_ms.min() * 1e3)),
                step_us_cache_reused=reuse_us,
                wall_s_timed_region=wall)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 5])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-hbm-sweep", action="store_true")
    ap.add_argument("--no-ratio-sweep", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
