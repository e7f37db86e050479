"""Benchmark of the integer-only ViT forward pass on B200 (DeiT-S shapes, batch 64, synthetic weights).

  python bench.py [--gpus N] [--steps K] [--warmup W]         # the CUDA library
  python bench.py --impl reference [...]                      # the CPU oracle, as it stands

A step is one full forward of the workload (patch embedding, 12 encoder blocks, classifier) over
one batch of 64 synthetic images.  Prints one JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "int-only ViT images/s (DeiT-S b64)"
WORKLOAD = "deit_small_b64"
# dram__bytes_read.sum + dram__bytes_write.sum per GEMM launch of this workload, averaged over the four Dense
# layers of an encoder block in one ncu capture of this command (24.9, 5.4, 9.9, 5.5 MB): well below the 10 to 34 MB
# of operands and results per launch, because the activations stay in L2.
GEMM_DRAM_BYTES_PER_LAUNCH = 11.4e6
CONFIG_INDEX = 1
MIN_TIMED_SECONDS = 2.0     # the K-step loop is repeated until the timed region is at least this long
# the paper's latencies (RTX 2080Ti, TVM, batch 8, Table of Sec. 4.2): context beside the batch-8 figures
PAPER_MS_B8 = {"deit_tiny": 1.61, "deit_small": 2.97, "vit_base": 7.93, "swin_tiny": 4.29}


def vit_int8_ops(p) -> float:
    """Algorithmic int8 operations (2 per multiply-accumulate) of one forward of a ViT-family model."""
    B, T, D, H, h = p.B, p.T, p.D, p.H, p.heads
    M, d = B * T, p.D // p.heads
    blk = 2 * M * D * 3 * D + 2 * (B * h * 2 * T * T * d) + 2 * M * D * D + 2 * 2 * M * D * H
    return p.depth * blk + 2 * B * (T - 1) * (3 * p.patch * p.patch) * D + 2 * B * D * p.classes


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi; stop() keeps the samples taken inside the timed region."""

    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index, self.proc = gpu_index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self, t_begin: float, t_end: float) -> dict:
        """t_begin, t_end: time.time() at the two ends of the timed region."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                if ts < t_begin - 0.02 or ts > t_end + 0.02:
                    continue
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        top = sorted(sm)[len(sm) // 2:]   # the busier half of the samples: the clock under load
        return {"sm_mhz": statistics.median(top), "sm_max_mhz": max(mx), "samples": len(sm),
                "power_w_max": max(power), "reasons": sorted(reasons)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def two_in_flight(binding, model, image, dev, dm, pairs):
    """Throughput with two independent batch-64 forwards in flight (two contexts, two streams, their own inputs,
    outputs and workspaces; the weights are shared): the fill and drain of one forward's kernels overlap the other's.
    Reported beside the headline, which stays one forward at a time."""
    import torch
    lanes = []
    for _ in range(2):
        ctx = binding.Context(dev.index)
        st = torch.cuda.Stream(device=dev)
        ctx.set_stream(st)
        with torch.cuda.stream(st):
            ws = dm.host_workspace()
            d_img = torch.from_numpy(image).to(dev)
            d_out = torch.empty((model.B, model.classes), dtype=torch.int32, device=dev)
            for _ in range(3):
                ctx.vit_forward(dm, d_img, logits=d_out, workspace=ws)
            st.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=st):
                ctx.vit_forward(dm, d_img, logits=d_out, workspace=ws)
        lanes.append((ctx, st, graph, ws, d_img, d_out))
    (c0, s0, g0, *_), (c1, s1, g1, *_) = lanes
    for _ in range(3):
        with torch.cuda.stream(s0):
            g0.replay()
        with torch.cuda.stream(s1):
            g1.replay()
    torch.cuda.synchronize()
    begin, end, joined = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), torch.cuda.Event())
    begin.record(s0)
    s1.wait_event(begin)
    for _ in range(pairs):
        with torch.cuda.stream(s0):
            g0.replay()
        with torch.cuda.stream(s1):
            g1.replay()
    joined.record(s1)
    s0.wait_event(joined)
    end.record(s0)
    torch.cuda.synchronize()
    ms = begin.elapsed_time(end)
    status = c0.poll_status() or c1.poll_status()
    if status != 0:
        raise RuntimeError(f"device-side error {status}")
    same = bool(torch.equal(lanes[0][5], lanes[1][5]))
    return {"images_per_s": round(2 * model.B * pairs / (ms * 1e-3), 1), "ms_per_pair": round(ms / pairs, 4),
            "outputs_equal": same,
            "note": "two batch-64 forwards at a time on two streams (one CUDA graph each); working set of the pair above L2"}


def gemm_probe(ctx, binding, peaks, dev):
    """The Dense kernel alone on two tensor-bound shapes (ViT-B FC1 at batch 128, and 8192^3): back-to-back launches
    between one pair of CUDA events, against the burst int8 peak (2 x the measured burst bf16 rate)."""
    import numpy as np
    import torch
    from ivit_inputs import Scale
    from ivit_inputs.gen import dyadic
    out = []
    rng = np.random.default_rng(0)
    for M, N, K in ((25216, 3072, 768), (8192, 8192, 8192)):
        A = torch.from_numpy(rng.integers(-127, 128, (M, K), dtype=np.int8)).to(dev)
        W = torch.from_numpy(rng.integers(-127, 128, (N, K), dtype=np.int8)).to(dev)
        sc = binding.DevScale(Scale(*dyadic(1.0 / (40.0 * 74.0 * np.sqrt(K)))), dev)
        o = torch.empty((M, N), dtype=torch.int8, device=dev)
        reps = 10
        for _ in range(3):
            ctx.linear(A, W, None, sc, out=o)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            ctx.linear(A, W, None, sc, out=o)
        b.record()
        torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(b) / reps
        tops = 2.0 * M * N * K / (us * 1e-6) / 1e12
        out.append({"shape": f"{M}x{N}x{K}", "us": round(us, 2), "TOPS": round(tops, 1),
                    "frac_of_burst_int8_peak": round(tops / (2.0 * peaks["bf16_tflops"]), 4)})
        del A, W, o
    return out


def time_oracle(model, image, budget_s: float = 15.0):
    """Times the CPU oracle on a bounded sample of the workload's images; returns (images/s, n, seconds, threads)."""
    from oracle import api as O
    t0 = time.perf_counter()
    O.vit_forward(model, image[:1])
    t1 = time.perf_counter() - t0
    n = int(max(1, min(image.shape[0], budget_s / max(t1, 1e-3))))
    t0 = time.perf_counter()
    O.vit_forward(model, image[:n])
    dt = time.perf_counter() - t0
    return n / dt, n, dt, O.num_threads()


def run_reference(args):
    """The CPU oracle timed as the reference arm (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from ivit_inputs import make_config
    from oracle import api as O
    model, image = make_config(CONFIG_INDEX)
    t0 = time.perf_counter()
    O.vit_forward(model, image[:1])
    t1 = time.perf_counter() - t0
    # each step is a sample of n images, sized so that steps + warmup stay within about two minutes
    n = int(max(1, min(image.shape[0], 120.0 / max(t1, 1e-3) / max(1, args.steps + args.warmup))))
    for _ in range(args.warmup):
        O.vit_forward(model, image[:n])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.vit_forward(model, image[:n])
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = f"{n} of {image.shape[0]} images per step (images are independent)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "images/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "images_per_step": n, "note": "CPU oracle, plain int64 loops, OpenMP over rows"},
        "cpu_baseline": {"value": value, "unit": "images/s", "cores": O.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def reduce_max(values, dist, device):
    """Max over ranks of each value (the slowest rank defines the step time); identity without a process group."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(batch_per_rank: int, world: int, steps: int, ms_total: float) -> float:
    """Images per second of the whole job: every rank processed `batch_per_rank` images per step (weak scaling)."""
    return batch_per_rank * world * steps / (ms_total * 1e-3)


def time_loop(torch, step_fn, steps, flush, barrier, min_seconds):
    """The K-step loop (each step inside its own CUDA-event pair, L2 flushed between steps outside the pairs),
    repeated until the timed region lasts at least `min_seconds`.  Returns (ms of the median repeat, repeats)."""
    totals, spent = [], 0.0
    while True:
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        t0 = time.perf_counter()
        for a, b in ev:
            flush.zero_()
            a.record()
            step_fn()
            b.record()
        barrier()
        spent += time.perf_counter() - t0
        totals.append(sum(a.elapsed_time(b) for a, b in ev))
        if spent >= min_seconds or len(totals) >= 4096:
            break
    return statistics.median(totals), len(totals)


def other_configs(ctx, binding, torch, np, flush, dev):
    """The other four workloads (parity-test cases, timed for the record): one forward at a time, stream launches,
    inputs resident, L2 flushed between steps; one image of each is recomputed by the oracle."""
    from ivit_inputs import make_config
    from ivit_inputs.gen import CONFIGS
    from oracle import api as O
    out = {}

    def time_steps(fn, steps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush.zero_()
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in ev)

    # config 0: one DeiT-Tiny encoder block, one image: latency, not a roofline case
    blk, X = make_config(0)
    dblk = binding.DeviceBlock(blk, dev)
    dX = torch.from_numpy(X).to(dev)
    dY = torch.empty_like(dX)
    wsb = dblk.workspace()
    l0 = ctx.launch_count()
    ctx.block_forward(dblk, dX, dY, workspace=wsb)
    nl = ctx.launch_count() - l0
    ms = time_steps(lambda: ctx.block_forward(dblk, dX, dY, workspace=wsb), 200)
    ok = bool(np.array_equal(dY.cpu().numpy(), O.block_forward(blk, X)))
    out[CONFIGS[0]["name"]] = {"us_per_block": round(1e3 * ms, 2), "launches": int(nl), "oracle_check": ok,
                               "note": "latency-bound: 0.2 GOP cannot fill 148 SMs"}
    del dblk, dX, dY, wsb
    for idx in (2, 4):
        model, image = make_config(idx)
        dm = binding.DeviceVit(model, dev)
        ws = dm.workspace()
        d_img = torch.from_numpy(image).to(dev)
        d_out = torch.empty((model.B, model.classes), dtype=torch.int32, device=dev)
        ms = time_steps(lambda: ctx.vit_forward(dm, d_img, logits=d_out, workspace=ws), 20)
        last = model.B - 1
        ok = bool(np.array_equal(d_out[last:].cpu().numpy(), O.vit_forward(model, image[last:])))
        out[CONFIGS[idx]["name"]] = {"ms_per_forward": round(ms, 4), "images_per_s": round(model.B / (ms * 1e-3), 1),
                                     "int8_TOPS": round(vit_int8_ops(model) / (ms * 1e-3) / 1e12, 1),
                                     "oracle_check": ok, "image_checked": last}
        del dm, ws, d_img, d_out, model, image
    model, image = make_config(3)
    dm = binding.DeviceSwin(model, dev)
    d_img = torch.from_numpy(image).to(dev)
    d_out = torch.empty((model.B, model.classes), dtype=torch.int32, device=dev)
    wsw = dm.host_workspace()
    ms = time_steps(lambda: binding.swin_forward(ctx, dm, d_img, logits=d_out, workspace=wsw), 20)
    h_img = torch.from_numpy(image).pin_memory()
    h_out = torch.empty((model.B, model.classes), dtype=torch.int32).pin_memory()
    ctx.set_host_graph(True)   # the host entry replays its own captured graph from the third call on
    for _ in range(4):
        binding.swin_forward_host(ctx, dm, h_img, h_out, wsw)
    ms_e2e = time_steps(lambda: binding.swin_forward_host(ctx, dm, h_img, h_out, wsw), 20)
    ctx.set_host_graph(False)
    torch.cuda.synchronize()
    one, _ = make_config(3, batch=1)
    want = O.swin_forward(one, image[63:])
    ok = bool(np.array_equal(d_out[63:].cpu().numpy(), want)) and bool(np.array_equal(h_out[63:].numpy(), want))
    out[CONFIGS[3]["name"]] = {"ms_per_forward": round(ms, 4), "images_per_s": round(model.B / (ms * 1e-3), 1),
                               "int8_TOPS": round(574.8e9 / (ms * 1e-3) / 1e12, 1), "oracle_check": ok, "image_checked": 63,
                               "e2e": {"images_per_s": round(model.B / (ms_e2e * 1e-3), 1), "ms_per_forward": round(ms_e2e, 4),
                                       "h2d_bytes": int(h_img.numel()), "d2h_bytes": int(h_out.numel() * 4),
                                       "entry": "ivit_swin_forward_host with ivit_ctx_set_host_graph(1)"}}
    del dm, d_img, wsw
    return out


def batch8_latencies(ctx, binding, torch, flush, dev):
    """Forward latency at batch 8, the batch size of the paper's latency table (other hardware, other weights:
    context only)."""
    from ivit_inputs.gen import make_image, make_swin, make_vit
    shapes = {"deit_tiny": dict(D=192, heads=3, H=768), "deit_small": dict(D=384, heads=6, H=1536),
              "vit_base": dict(D=768, heads=12, H=3072)}
    out = {}

    def lat(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(30)]
        for a, b in ev:
            flush.zero_()
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in ev)

    for k, (name, sh) in enumerate(shapes.items()):
        model = make_vit(100 + k, 8, 224, sh["D"], sh["heads"], sh["H"], 12)
        dm = binding.DeviceVit(model, dev)
        ws = dm.workspace()
        d_img = torch.from_numpy(make_image(100 + k, 8, 224)).to(dev)
        d_out = torch.empty((8, 1000), dtype=torch.int32, device=dev)
        ms = lat(lambda: ctx.vit_forward(dm, d_img, logits=d_out, workspace=ws))
        out[name] = {"ms": round(ms, 4), "paper_ms_rtx2080ti_tvm": PAPER_MS_B8[name]}
        del dm, ws
    sw = make_swin(103, 8)
    dsw = binding.DeviceSwin(sw, dev)
    d_img = torch.from_numpy(make_image(103, 8, 224)).to(dev)
    d_o8 = torch.empty((8, 1000), dtype=torch.int32, device=dev)
    ms = lat(lambda: binding.swin_forward(ctx, dsw, d_img, logits=d_o8))
    out["swin_tiny"] = {"ms": round(ms, 4), "paper_ms_rtx2080ti_tvm": PAPER_MS_B8["swin_tiny"]}
    return out


def standalone_ops(ctx, binding, torch, np, peaks, dev):
    """Every operator of the block timed alone on the DeiT-S batch-64 shapes.  The row kernels (I-LayerNorm,
    Shiftmax, ShiftGELU) run on buffers rotated through more than twice the L2 capacity the device reports, so that
    their GB/s are HBM rates, and once more on a single L2-resident buffer pair (labelled).  Beside every GPU rate:
    the CPU oracle's rate for the same operator on a bounded sample of the rows."""
    from ivit_inputs import ExpParams, make_config
    from oracle import api as O
    model, _ = make_config(CONFIG_INDEX, batch=1)
    blk = model.blocks[0]
    B, T, D, H, h = 64, model.T, model.D, model.H, model.heads
    M = B * T
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    rng = np.random.default_rng(7)
    hbm, spec = peaks["hbm_gbs"], 8000.0

    def rate(fn_of_i, nbuf, launches):
        """ms per launch, device time: the launches are captured into one CUDA graph (no host launch cost between
        them) and the replay is timed with one event pair."""
        for i in range(min(nbuf, 3)):
            fn_of_i(i)
        torch.cuda.synchronize()
        stream = torch.cuda.current_stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(launches):
                fn_of_i(i % nbuf)
        graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best = None
        for _ in range(3):
            a.record()
            graph.replay()
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / launches
            best = ms if best is None or ms < best else best
        return best

    def cpu_rate(fn, units):
        fn()
        t0 = time.perf_counter()
        n = 0
        while time.perf_counter() - t0 < 1.0:
            fn()
            n += 1
        return units * n / (time.perf_counter() - t0)

    out = {"l2_bytes": int(l2), "shapes": "DeiT-S, batch 64", "hbm_peak_gbs_measured": hbm, "hbm_peak_gbs_spec": spec}

    def row_kernel(name, rows, cols, ld, launch, oracle_fn, sample_rows):
        per = rows * ld
        nbuf = int(2 * l2 // (2 * per)) + 2                    # in + out of every launch are fresh lines
        src = torch.from_numpy(rng.integers(-128, 128, (nbuf, rows, ld), dtype=np.int8)).to(dev)
        dst = torch.empty_like(src)
        cold = rate(lambda i: launch(src[i, :, :cols], dst[i, :, :cols]), nbuf, 3 * nbuf)
        warm = rate(lambda i: launch(src[0, :, :cols], dst[0, :, :cols]), 1, 200)
        bytes_ = 2.0 * rows * cols
        x = src[0, :sample_rows, :cols].cpu().numpy()
        out[name] = {"rows": rows, "cols": cols, "buffers_rotated": nbuf, "rotated_MB": round(2 * per * nbuf / 1e6),
                     "us_hbm_cold": round(1e3 * cold, 2), "GBs_hbm_cold": round(bytes_ / (cold * 1e-3) / 1e9, 1),
                     "frac_of_measured_hbm": round(bytes_ / (cold * 1e-3) / 1e9 / hbm, 4),
                     "frac_of_spec_hbm": round(bytes_ / (cold * 1e-3) / 1e9 / spec, 4),
                     "us_l2_warm": round(1e3 * warm, 2), "GBs_l2_warm": round(bytes_ / (warm * 1e-3) / 1e9, 1),
                     "oracle_elements_per_s": round(cpu_rate(lambda: oracle_fn(x), x.size)),
                     "gpu_elements_per_s_hbm_cold": round(rows * cols / (cold * 1e-3))}
        del src, dst

    g1 = binding.DevScale(blk.ln1_gamma, dev)
    b1 = torch.from_numpy(blk.ln1_beta).to(dev)
    row_kernel("layernorm", M, D, D, lambda x, y: ctx.layernorm(x, g1, b1, blk.M_ln, out=y),
               lambda x: O.layernorm(x, blk.ln1_gamma, blk.ln1_beta, blk.M_ln), 4096)
    ldS = (T + 15) // 16 * 16
    row_kernel("shiftmax", B * h * T, T, ldS, lambda x, y: ctx.shiftmax(x, blk.smax, out=y),
               lambda x: O.shiftmax(x, blk.smax), 8192)
    post = binding.DevScale(blk.gelu_post, dev)
    row_kernel("shiftgelu", M, H, H, lambda x, y: ctx.shiftgelu(x, blk.gelu, post, out=y),
               lambda x: O.shiftgelu(x, blk.gelu, blk.gelu_post), 2048)

    # Dense (QKV shape) and the two MatMuls of the attention, L2-resident operands
    A = torch.from_numpy(rng.integers(-100, 100, (M, D), dtype=np.int8)).to(dev)
    W = torch.from_numpy(blk.Wqkv).to(dev)
    bq = torch.from_numpy(blk.bqkv).to(dev)
    sc = binding.DevScale(blk.qkv_scale, dev)
    o = torch.empty((M, 3 * D), dtype=torch.int8, device=dev)
    ms = rate(lambda i: ctx.linear(A, W, bq, sc, out=o), 1, 50)
    xs = A[:1024].cpu().numpy()
    out["linear_qkv"] = {"M": M, "N": 3 * D, "K": D, "us": round(1e3 * ms, 2),
                         "TOPS": round(2.0 * M * 3 * D * D / (ms * 1e-3) / 1e12, 1),
                         "oracle_GOPS": round(cpu_rate(lambda: O.linear(xs, blk.Wqkv, blk.bqkv, blk.qkv_scale),
                                                       2.0 * 1024 * 3 * D * D) / 1e9, 2)}
    d = D // h
    nb = B * h
    Q = torch.from_numpy(rng.integers(-100, 100, (nb, T, d), dtype=np.int8)).to(dev)
    K = torch.from_numpy(rng.integers(-100, 100, (nb, T, d), dtype=np.int8)).to(dev)
    qk = binding.DevScale(blk.qk_scale, dev)
    S = torch.zeros((nb, T, ldS), dtype=torch.int8, device=dev)[:, :, :T]
    ms = rate(lambda i: ctx.matmul(Q, K, True, qk, out=S), 1, 50)
    qs, ks = Q[:16].cpu().numpy(), K[:16].cpu().numpy()
    out["matmul_qk"] = {"batches": nb, "M": T, "N": T, "K": d, "us": round(1e3 * ms, 2),
                        "TOPS": round(2.0 * nb * T * T * d / (ms * 1e-3) / 1e12, 1),
                        "oracle_GOPS": round(cpu_rate(lambda: O.matmul(qs, ks, True, blk.qk_scale), 2.0 * 16 * T * T * d) / 1e9, 2)}
    return out


def run_gpu(args):
    import numpy as np
    import torch
    from ivit_inputs import make_config
    from paper_2207_01405_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    build.build()
    ctx = binding.Context(local_rank)
    dev = ctx.device
    # everything runs on one side stream (a forward is captured into a CUDA graph below: not possible on the
    # legacy default stream)
    side = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(side)
    ctx.set_stream(side)

    # every rank serves its own batch of the same synthetic workload (weak scaling, no exchange step)
    from ivit_inputs.gen import CONFIGS
    model, image = make_config(args.config)
    workload = CONFIGS[args.config]["name"]
    metric = METRIC if args.config == CONFIG_INDEX else f"int-only ViT images/s ({workload})"
    if args.config != CONFIG_INDEX:
        args.headline_only = True
    dm = binding.DeviceVit(model, dev)
    B = model.B
    ws = dm.host_workspace()
    d_image = torch.from_numpy(image).to(dev)
    d_logits = torch.empty((B, model.classes), dtype=torch.int32, device=dev)
    h_image = torch.from_numpy(image).pin_memory()
    h_logits = torch.empty((B, model.classes), dtype=torch.int32).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > L2 (126 MB)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def step_resident():
        ctx.vit_forward(dm, d_image, logits=d_logits, workspace=ws)

    def step_e2e():
        binding.vit_forward_host(ctx, dm, h_image, h_logits, ws)

    sampler = ClockSampler(local_rank)
    sampler.start()   # before the warm-up: the first sample takes a while to come
    for _ in range(max(args.warmup, 3)):
        step_resident()
    torch.cuda.synchronize()

    # One forward = a few dozen kernels with programmatic dependencies: captured once, replayed per step.  The graph
    # holds exactly the launches of step_resident(); if the capture is refused the steps are launched one by one.
    launches0 = ctx.launch_count()
    step_resident()
    launches_per_step = ctx.launch_count() - launches0
    torch.cuda.synchronize()
    step_timed, launch_mode = step_resident, "stream launches"
    try:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step_resident()
        graph.replay()
        torch.cuda.synchronize()
        step_timed, launch_mode = graph.replay, "one CUDA graph per forward"
    except Exception as exc:   # noqa: BLE001
        print(f"graph capture unavailable ({exc}); timing stream launches", file=sys.stderr)
    t_begin = time.time()
    min_s = 0.0 if args.headline_only else MIN_TIMED_SECONDS
    ms_total, repeats = time_loop(torch, step_timed, args.steps, flush, barrier, min_s)
    t_end = time.time()
    launches = launches_per_step * args.steps
    clocks = sampler.stop(t_begin, t_end)
    ms_eager, _ = time_loop(torch, step_resident, min(args.steps, 50), flush, barrier, 0.0)

    # the host-buffer entry point replays its own captured graph from the third call on (one per staging buffer)
    ctx.set_host_graph(True)
    for _ in range(8):
        step_e2e()
    torch.cuda.synchronize()
    ms_e2e, _ = time_loop(torch, step_e2e, args.steps, flush, barrier, min_s / 2)
    ctx.set_host_graph(False)
    status = ctx.poll_status()
    if status != 0:
        raise RuntimeError(f"device-side error {status}")

    # per-kernel times of the same step, event-bracketed launch by launch (a separate pass: the
    # event pairs serialise launches, so this pass is not the throughput number)
    prof_steps = min(args.steps, 5)
    ctx.profile_start()
    for _ in range(prof_steps):
        # ~2 ms of device work queued first, so that the host has submitted the whole step before the device
        # reaches it: an event pair then spans its kernel, not the host's launch latency
        for _ in range(30):
            flush.zero_()
        step_resident()
    records = ctx.profile_stop()

    ms_total, ms_e2e = reduce_max([ms_total, ms_e2e], dist, dev)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peak_src = measured_peaks()
    by_kind = {}
    for kind, ms, work in records:
        k = by_kind.setdefault(kind, {"launches": 0, "ms": 0.0, "work": 0.0})
        k["launches"] += 1
        k["ms"] += ms
        k["work"] += work
    total_kernel_ms = sum(k["ms"] for k in by_kind.values())
    if args.detail:
        shapes = {}
        for kind, ms, work in records:
            k = shapes.setdefault((kind, work), [0, 0.0])
            k[0] += 1
            k[1] += ms
        for (kind, work), (n, ms) in sorted(shapes.items(), key=lambda kv: -kv[1][1]):
            unit = "TOP/s" if kind.startswith(("gemm", "attention")) else "GB/s"
            rate = work / (ms / n * 1e-3) / (1e12 if unit == "TOP/s" else 1e9)
            print(f"  {kind:16s} work={work:14.0f} launches/step={n // prof_steps:3d} us/launch={1e3 * ms / n:8.2f} "
                  f"{rate:9.1f} {unit}", file=sys.stderr)
    kernels = {}
    for kind, k in sorted(by_kind.items(), key=lambda kv: -kv[1]["ms"]):
        per_step_ms = k["ms"] / prof_steps
        rate = k["work"] / prof_steps / (per_step_ms * 1e-3) if per_step_ms > 0 else 0.0
        is_gemm = kind.startswith("gemm") or kind.startswith("attention")
        kernels[kind] = {"launches_per_step": k["launches"] // prof_steps, "ms_per_step": round(per_step_ms, 4),
                         "share": round(k["ms"] / total_kernel_ms, 4),
                         ("TOPS" if is_gemm else "GB/s (L2-resident, in step)"): round(rate / (1e12 if is_gemm else 1e9), 2)}

    # the int8 tensor ceiling measured on this device: tcgen05.mma.kind::i8 issue-only loop
    probe_ms, probe_ops = ctx.probe_int8_mma(8192)
    int8_probe = probe_ops / (probe_ms * 1e-3) / 1e12
    dom = next(iter(kernels))
    dk = by_kind[dom]
    int8_peak = 2.0 * peaks["bf16_tflops_sustained"]      # int8 dense = 2 x bf16 (nominal ratio), sustained: timed inside a long step
    if dom.startswith("gemm") or dom.startswith("attention"):
        # Average duration of this kernel's launches INSIDE the timed region: the timed step (CUDA events around the
        # whole forward) x this kernel's share of the per-launch event times (the share agrees with ncu's launch
        # list).  `achieved_alone` divides by the per-launch event times themselves: an event pair around every launch
        # adds a few microseconds and stops the overlap of a kernel's set-up with its predecessor's tail.
        alone = dk["work"] / (dk["ms"] * 1e-3) / 1e12
        achieved = dk["work"] / prof_steps / (ms_total / args.steps * 1e-3 * dk["ms"] / total_kernel_ms) / 1e12
        roofline = {"kernel": dom, "bound": "tensor", "achieved": round(achieved, 2), "peak": int8_peak, "unit": "TOP/s",
                    "frac": round(achieved / int8_peak, 4),
                    "traffic": GEMM_DRAM_BYTES_PER_LAUNCH if args.config == CONFIG_INDEX else None,
                    "achieved_alone": round(alone, 2), "frac_alone": round(alone / int8_peak, 4),
                    "us_per_launch_in_step": round(ms_total / args.steps * 1e3 * dk["ms"] / total_kernel_ms / (dk["launches"] / prof_steps), 2),
                    "us_per_launch_alone": round(dk["ms"] * 1e3 / dk["launches"], 2),
                    "frac_of_mma_issue_probe": round(achieved / int8_probe, 4),
                    "frac_of_spec_4500": round(achieved / 4500.0, 4),
                    "peak_source": f"2 x {peak_src} sustained bf16 cuBLAS ({peaks['bf16_tflops_sustained']} TFLOP/s)"}
    else:
        achieved = dk["work"] / (dk["ms"] * 1e-3) / 1e9
        roofline = {"kernel": dom, "bound": "hbm", "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": round(achieved / peaks["hbm_gbs"], 4), "traffic": None, "peak_source": f"{peak_src} copy bandwidth"}

    extras = {}
    if not args.headline_only:
        probe = gemm_probe(ctx, binding, peaks, dev)
        for pr in probe:
            pr["frac_of_mma_issue_probe"] = round(pr["TOPS"] / int8_probe, 4)
        # the same forward with the static-maximum ShiftGELU variant (a different function from the paper's Algorithm 2,
        # applied inside the FC1 epilogue): reported beside the headline, never as the headline
        import copy
        vmodel = copy.copy(model)
        vmodel.blocks = [copy.copy(b) for b in model.blocks]
        for b in vmodel.blocks:
            b.gelu_static_max = True
        vdm = binding.DeviceVit(vmodel, dev)
        for _ in range(3):
            ctx.vit_forward(vdm, d_image, logits=d_logits, workspace=ws)
        vsteps = min(args.steps, 50)
        ms_variant, _ = time_loop(torch, lambda: ctx.vit_forward(vdm, d_image, logits=d_logits, workspace=ws), vsteps, flush, barrier, 0.0)
        variant = {"images_per_s": round(B * vsteps / (ms_variant * 1e-3), 1),
                   "note": "ShiftGELU with I_max fixed at I_p(127), fused into the FC1 epilogue; not Algorithm 2"}
        del vdm
        # the same forward with LayerNorm / ShiftGELU run inside the Dense kernels that produce their rows (off by default)
        ctx.set_row_fusion(True)
        l0 = ctx.launch_count()
        for _ in range(3):
            step_resident()
        fused_launches = (ctx.launch_count() - l0) // 3
        ms_fused, _ = time_loop(torch, step_resident, vsteps, flush, barrier, 0.0)
        ctx.set_row_fusion(False)
        fused = {"images_per_s": round(B * vsteps / (ms_fused * 1e-3), 1), "kernels_per_forward": int(fused_launches),
                 "note": "ivit_ctx_set_row_fusion(1): same bytes, row operators inside the Dense kernels; stream launches"}
        in_flight = two_in_flight(binding, model, image, dev, dm, min(args.steps, 100))
        cpu_rate, cpu_n, cpu_s, cpu_threads = time_oracle(model, image)
        # the timed steps really computed the forward: spot-check one image against the oracle
        from oracle import api as O
        ok = bool(np.array_equal(h_logits[:1].numpy(), O.vit_forward(model, image[:1])))
        ops_standalone = standalone_ops(ctx, binding, torch, np, peaks, dev)
        configs = other_configs(ctx, binding, torch, np, flush, dev)
        b8 = batch8_latencies(ctx, binding, torch, flush, dev)
        extras = {
            "gemm_probe": probe, "static_gelu_variant": variant, "row_fusion_variant": fused, "two_forwards_in_flight": in_flight,
            "cpu_baseline": {"value": cpu_rate, "unit": "images/s", "cores": cpu_threads, "kind": "oracle",
                             "sample": f"{cpu_n} of {B} images ({cpu_s:.1f} s; images are independent)"},
            "nonlinear_standalone": {k: v for k, v in ops_standalone.items() if k not in ("linear_qkv", "matmul_qk")},
            "per_op_gpu_vs_oracle": {k: v for k, v in ops_standalone.items() if k in ("linear_qkv", "matmul_qk")},
            "configs": configs, "batch8_latency_ms": b8, "parity_spot_check": ok,
        }
    status = ctx.poll_status()
    if status != 0:
        raise RuntimeError(f"device-side error {status}")

    ops = vit_int8_ops(model)
    line = {
        "metric": metric, "value": whole_job_rate(B, world, args.steps, ms_total), "unit": "images/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8 x int8 -> int32",
        "data": "synthetic", "config": {"workload": workload, "batch_per_gpu": B, "tokens": model.T, "embed": model.D,
                                        "heads": model.heads, "mlp": model.H, "blocks": model.depth,
                                        "l2": "256 MB buffer written between steps, outside the per-step event pairs",
                                        "timed_region": f"the {args.steps}-step loop repeated {repeats} times "
                                                        f"(>= {MIN_TIMED_SECONDS} s); value = the median repeat",
                                        "parallelism": f"dp{world} (independent batches, no collective)"},
        "e2e": {"value": whole_job_rate(B, world, args.steps, ms_e2e), "unit": "images/s", "h2d_bytes_per_step": int(h_image.numel()),
                "d2h_bytes_per_step": int(h_logits.numel() * 4), "ms_per_step": ms_e2e / args.steps,
                "launch": "ivit_vit_forward_host with ivit_ctx_set_host_graph(1): copies + one graph launch per call"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
        "launch": {"mode": launch_mode, "kernels_per_forward": int(launches_per_step),
                   "stream_launch_images_per_s": round(B * world * min(args.steps, 50) / (ms_eager * 1e-3), 1)},
        "int8_peak_probe": {"TOPS": round(int8_probe, 1), "ms": round(probe_ms, 4),
                            "what": "tcgen05.mma.kind::i8 M128 N256 K32, issue-only, operands fixed in shared memory, one CTA per SM",
                            "spec_TOPS": 4500.0, "twice_bf16_sustained": int8_peak, "twice_bf16_burst": 2.0 * peaks["bf16_tflops"]},
        "int8_tops_whole_step": round(ops / (ms_total / args.steps * 1e-3) / 1e12, 2),
        "kernels": kernels,
    }
    line.update(extras)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ivit", choices=["ivit", "reference"])
    ap.add_argument("--detail", action="store_true", help="print per-shape kernel times to stderr")
    ap.add_argument("--config", type=int, default=CONFIG_INDEX, choices=[1, 2, 4],
                    help="ViT-family configuration to time (default 1, the headline; 2 and 4 print the same line for that workload, without the extra sections)")
    ap.add_argument("--headline-only", action="store_true",
                    help="time the headline workload only (K steps once, no extra sections): the command the ncu captures run")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
