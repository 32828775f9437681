#!/usr/bin/env python
"""Benchmark of the FlashCache compression pass (score + allocate + select + compact).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl reference]

A step is one pass of the whole hot path over all layers of the workload, inputs
resident in HBM.  Prints ONE JSON line (rank 0): KV tokens compressed per second,
the roofline of the dominant kernel measured with CUDA events inside the timed
region, the same metric end to end from pinned host buffers, the fp64 CPU oracle
timed on a bounded sample of the same workload, and the SM clocks sampled during
the timed region.  With N > 1 (launched by torch.distributed.run) every rank
runs an independent replica of the workload on its own GPU; nothing is exchanged.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "kv_tokens_compressed_per_s"
UNIT = "tokens/s"
FP32_LANES_PER_SM = 128          # FP32 FMA lanes per SM on B200
DEFAULT_CONFIG = "cfg3"          # the 32k-token workload the target fraction is quoted on

# DRAM bytes read + written per launch of the dominant kernel as an ncu capture counted them (a constant from
# that capture, not a measurement of this run; None where no capture of the kernel and workload exists):
# pass 2 of cfg3, 0.73 MB read + 0.84 MB written on average over 8 launches with the intermediate in the
# persisting part of L2 (ncu --cache-control none, one pass per launch).
NCU_TRAFFIC_BYTES = {
    ("cfg3", "pass2"): 1.57e6,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, sm_max_mhz=1965.0, source="fallback")


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 25):
        self.out = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=timestamp," + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", str(period_ms)],
                stdout=self.out, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t0_wall: float, t1_wall: float):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"], samples=0)
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.out.flush()
        self.out.seek(0)
        import datetime
        rows = []
        for line in self.out.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), parts[4:9]))
            except ValueError:
                continue
        os.unlink(self.out.name)
        inside = [r for r in rows if t0_wall - 0.02 <= r[0] <= t1_wall + 0.02] or rows
        if not inside:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"], samples=0)
        sm = sorted(r[1] for r in inside)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in inside:
            for name, val in zip(names, r[3][1:]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=sm[len(sm) // 2], sm_max_mhz=inside[0][2], reasons=sorted(reasons),
                    samples=len(inside))


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    ids = [x.strip() for x in vis.split(",") if x.strip()]
    if local_rank < len(ids) and ids[local_rank].isdigit():
        return int(ids[local_rank])
    return local_rank


# --------------------------------------------------------------------------- accounting
def step_accounting(binding, handle, cfg):
    """Algorithmic flops and HBM bytes of one step, per kernel class (what the shipped
    algorithm has to compute and move, not what the hardware happened to do)."""
    d, H, L = cfg.head_dim, cfg.num_heads, cfg.num_layers
    s = 4 if cfg.dtype == "f32" else 2
    acc = {k: dict(flops=0.0, bytes=0.0) for k in ("pass1", "pass2", "pass3", "select", "gather")}
    rows = 0
    for N in cfg.seqlens:
        if N == 0:
            continue
        plan = binding.fc_describe_plan(handle, N, cfg.gamma)
        M, n1, n2 = plan["nfft"], plan["n1"], plan["n2"]
        cols = H * d * L                       # complex columns (K + jV) of this sequence
        reps = 2 if plan["bluestein"] else 1   # chirp path: two convolutions, each a forward+inverse transform
        acc["pass1"]["flops"] += reps * cols * M * 5.0 * math.log2(n1)
        acc["pass2"]["flops"] += reps * cols * M * (10.0 * math.log2(n2) + 8.0)
        acc["pass3"]["flops"] += reps * cols * M * 5.0 * math.log2(n1) + cols * N * 4.0
        acc["pass1"]["bytes"] += N * H * L * 2.0 * d * s               # K and V rows, read once
        acc["pass3"]["bytes"] += N * H * L * 4.0                       # score write
        acc["select"]["bytes"] += N * H * L * 4.0                      # score read
        acc["gather"]["bytes"] += cfg.rho * N * H * L * (4.0 * d * s + 4.0)
        rows += N * H * L
    return acc, rows


# --------------------------------------------------------------------------- CPU baseline (oracle)
def oracle_sample(cfg, Ks_host, Vs_host, budget_s: float, threads: int = 1):
    """Times the fp64 oracle ("fft" tier, as it stands) on whole layers of the workload until about
    budget_s seconds are used; returns tokens/s scaled to the full layer count.  With threads > 1 the
    (layer, head) units go to a pool of host threads, one oracle call each (the oracle's numpy / scipy
    routines release the interpreter lock); the oracle itself is untouched."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    from oracle import flashcache_oracle as O
    L, H = cfg.num_layers, cfg.num_heads
    cu = cfg.cu_seqlens
    pool = ThreadPoolExecutor(max_workers=threads) if threads > 1 else None

    def run(fn, items):
        return list(pool.map(fn, items)) if pool else [fn(x) for x in items]

    def score_unit(lh):                      # one head of one layer, every sequence: scores and energy sums
        l, h = lh
        sc = np.zeros(cfg.total_tokens)
        en = np.zeros((len(cfg.seqlens), 4))
        for b, n in enumerate(cfg.seqlens):
            if n == 0:
                continue
            s, e = O.score_head(Ks_host[l][cu[b]:cu[b + 1], h].astype(np.float64),
                                Vs_host[l][cu[b]:cu[b + 1], h].astype(np.float64), cfg.gamma, "fft")
            sc[cu[b]:cu[b + 1]] = s
            en[b] = e
        return sc, en

    t0 = time.perf_counter()
    used, scores, energy = 0, [], []
    step = max(1, threads // H)              # layers scored per round, so that every thread has a unit
    while used < len(Ks_host):
        ls = list(range(used, min(len(Ks_host), used + step)))
        res = run(score_unit, [(l, h) for l in ls for h in range(H)])
        for i, l in enumerate(ls):
            scores.append(np.stack([res[i * H + h][0] for h in range(H)]))
            energy.append(sum(res[i * H + h][1] for h in range(H)))
        used += len(ls)
        el = time.perf_counter() - t0
        if el + el / used * len(ls) > budget_s:
            break
    budgets, offsets = O.allocate_budgets(np.stack(energy), list(cfg.seqlens), cfg.rho, cfg.min_keep)

    def select_unit(lh):
        l, h = lh
        for b, n in enumerate(cfg.seqlens):
            idx = O.select_topk(scores[l][h, cu[b]:cu[b + 1]], int(budgets[l, b]))
            O.compact_rows(Ks_host[l][cu[b]:cu[b + 1], h], idx)
            O.compact_rows(Vs_host[l][cu[b]:cu[b + 1], h], idx)

    run(select_unit, [(l, h) for l in range(used) for h in range(H)])
    el = time.perf_counter() - t0
    if pool:
        pool.shutdown()
    tokens_per_s = cfg.total_tokens / (el * L / used)
    return tokens_per_s, used, el


def run_reference(args):
    """--impl reference: the oracle on the host cores.  Each step is a bounded sample of the workload
    (one KV head of one layer, all sequences: transform, scores, budget rule, top-k, row copy), scaled
    by layers x heads, so that a few hundred steps still end within minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2511_16786_b200 import synth_kv as S
    cfg = S.paper_configs()[args.config]
    K, V = S.make_layer(cfg, 0, "cpu")
    one = S.scaled(cfg, cfg.name, num_layers=1, num_heads=1)
    Ks, Vs = [K[:, :1].float().numpy()], [V[:, :1].float().numpy()]
    times = []
    for i in range(max(args.warmup, 0) + args.steps):
        _, _, el = oracle_sample(one, Ks, Vs, budget_s=1e9)
        if i >= args.warmup:
            times.append(el)
    ms = 1000.0 * sum(times) / len(times)
    value = cfg.total_tokens / ((ms / 1000.0) * cfg.num_layers * cfg.num_heads)
    sample = "1 KV head of 1 layer (of %d x %d), all sequences, per step; scaled by layers x heads" % (
        cfg.num_layers, cfg.num_heads)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name + ": " + cfg.note, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# --------------------------------------------------------------------------- decoding step on the compacted cache
def run_decode(args):
    """Latency of the attention of one decoding step (fc_decode_attention, every layer) against the
    context length, on the full cache and on caches compressed to 20 % and 10 %: the quantity behind the
    paper's decoding-latency figure, for the attention part only.  L2 is flushed before every step, so
    the K and V rows come from HBM; the roofline is their bytes over the measured HBM bandwidth."""
    import torch
    from paper_2511_16786_b200 import binding
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    L, H, G, d, B = 28, 4, 7, 128, 1
    dtype = torch.bfloat16
    handle = binding.fc_create(0, 1024)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    g = torch.Generator(device=dev).manual_seed(0)
    points = []
    lengths = (args.decode_n,) if args.decode_n else (2048, 4096, 8192, 16384, 32768, 65536)
    ratios = (args.decode_rho,) if args.decode_rho else (1.0, 0.2, 0.1)
    for N in lengths:
        base_ms = None
        for rho in ratios:
            rows = max(1, int(rho * N + 0.5))
            ck = torch.randn((L, rows, H, d), generator=g, device=dev, dtype=torch.float32).to(dtype)
            cv = torch.randn((L, rows, H, d), generator=g, device=dev, dtype=torch.float32).to(dtype)
            q = torch.randn((B, H * G, d), generator=g, device=dev, dtype=torch.float32).to(dtype)
            off = torch.tensor([0, rows], dtype=torch.int64, device=dev)
            out = torch.empty((L, B, H * G, d), dtype=dtype, device=dev)
            argl = [binding.make_decode_args(q, ck[l], cv[l], off, rows) for l in range(L)]
            ws = torch.empty(binding.fc_decode_workspace_bytes(handle, argl[0]), dtype=torch.uint8, device=dev)

            def step():
                for l in range(L):
                    binding.fc_decode_attention(handle, argl[l], out[l], ws)

            for _ in range(3):
                step()
            torch.cuda.synchronize()
            binding._check(binding.fc_last_device_status(handle), "device status")
            n_rep = 20
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_rep)]
            for e0, e1 in ev:
                flush.zero_()
                e0.record()
                step()
                e1.record()
            torch.cuda.synchronize()
            ms = sorted(e0.elapsed_time(e1) for e0, e1 in ev)[n_rep // 2]
            # the same step replayed from a CUDA graph, as a serving loop would issue it
            graph = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream(dev))
            with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
                step()
            for e0, e1 in ev:
                flush.zero_()
                e0.record()
                graph.replay()
                e1.record()
            torch.cuda.synchronize()
            ms_graph = sorted(e0.elapsed_time(e1) for e0, e1 in ev)[n_rep // 2]
            del graph
            nbytes = 2.0 * L * rows * H * d * 2
            gbs = nbytes / (ms_graph * 1e-3) / 1e9
            if base_ms is None:
                base_ms = ms_graph
            points.append({"N": N, "rho": rho, "rows_per_layer": rows, "ms_per_step_eager": ms, "ms_per_step": ms_graph,
                           "gbytes": nbytes / 1e9,
                           "achieved_gbs": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"],
                           "speedup_vs_first_ratio": base_ms / ms_graph})
            del ck, cv
    binding.fc_destroy(handle)
    print(json.dumps({
        "metric": "decode_attention_ms_per_token", "unit": "ms", "higher_is_better": False, "n_gpus": 1,
        "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
        "config": {"workload": "attention of one decoding step over the compacted caches of 28 layers, "
                               "4 KV heads x 7 query heads, head_dim 128, batch 1",
                   "l2_policy": "256 MB written before every step (flush)", "median_of": 20},
        "roofline": {"bound": "hbm", "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "peak_source": "MEASURED_PEAKS.json hbm_gbs (%s)" % peaks["source"]},
        "points": points}))


# --------------------------------------------------------------------------- FP32 pipes against the tensor pipe
def run_proto(args):
    """One radix-16 transform stage on an L2-resident tile (16 x 65536 complex columns, 8.4 MB each way), on the
    FP32 pipes, on the tensor pipe (3 x TF32) and as a plain copy; then the arithmetic alone (64 repetitions on the
    loaded registers).  Median of 20 launches each, CUDA events."""
    import torch
    from paper_2511_16786_b200 import binding
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    h = binding.fc_create(0, 1024)
    ncols = 65536
    x = torch.randn((16, ncols, 2), device=dev)
    y = torch.empty_like(x)
    res = {}
    for rep in (1, 64):
        for variant, name in ((0, "fp32_pipes"), (1, "tensor_pipe_3xtf32"), (2, "copy_only")):
            if variant == 2 and rep > 1:
                continue
            for _ in range(3):
                binding.fc_proto_dft16_stage(h, x, y, variant, rep)
            torch.cuda.synchronize()
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
            for e0, e1 in ev:
                e0.record()
                binding.fc_proto_dft16_stage(h, x, y, variant, rep)
                e1.record()
            torch.cuda.synchronize()
            res["%s_repeat%d_us" % (name, rep)] = 1000.0 * sorted(a.elapsed_time(b) for a, b in ev)[10]
    binding._check(binding.fc_last_device_status(h), "device status")
    binding.fc_destroy(h)
    a, t = res["fp32_pipes_repeat64_us"], res["tensor_pipe_3xtf32_repeat64_us"]
    res["arithmetic_us_per_stage_fp32_pipes"] = (a - res["fp32_pipes_repeat1_us"]) / 63.0
    res["arithmetic_us_per_stage_tensor_pipe"] = (t - res["tensor_pipe_3xtf32_repeat1_us"]) / 63.0
    print(json.dumps({"metric": "dft16_stage_us", "unit": "us", "higher_is_better": False, "n_gpus": 1,
                      "dtype": "f32 / tf32x3", "data": "synthetic",
                      "config": {"workload": "one radix-16 stage over 65536 complex columns (16 points each), "
                                             "tile resident in L2", "median_of": 20}, "times": res}))


# --------------------------------------------------------------------------- spectrum diagnostics
def run_spectrum(args):
    """Time of fc_power_spectrum (Eq. 11 per layer) over all layers of a config; a diagnostic, reported beside
    the transform work it repeats (pass 1 and half of pass 2 of the scoring)."""
    import torch
    from paper_2511_16786_b200 import binding, synth_kv as S
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = S.paper_configs()[args.config]
    L = cfg.num_layers
    Kd, Vd = zip(*[S.make_layer(cfg, l, dev) for l in range(L)])
    handle = binding.fc_create(0, max(cfg.seqlens))
    spec = torch.empty((L, cfg.total_tokens, 2), dtype=torch.float64, device=dev)
    ws = torch.empty(binding.fc_power_spectrum_workspace_bytes(handle, Kd[0], Vd[0], cfg.cu_seqlens),
                     dtype=torch.uint8, device=dev)

    def step():
        for l in range(L):
            binding.fc_power_spectrum(handle, Kd[l], Vd[l], cfg.cu_seqlens, spec[l], ws)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    binding._check(binding.fc_last_device_status(handle), "device status")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = max(3, min(args.steps, 20))
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    binding.fc_destroy(handle)
    print(json.dumps({"metric": "power_spectrum_ms_per_pass", "value": ms, "unit": "ms", "higher_is_better": False,
                      "n_gpus": 1, "steps": steps, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": cfg.name + ": " + cfg.note, "layers": L,
                                 "l2_policy": "inputs exceed L2; no flush"},
                      "tokens_per_s": cfg.total_tokens / (ms / 1000.0)}))


def quick_config(torch, binding, S, name, dev, peaks, alu_peak, warmup=3, steps=10):
    """ms per step, tokens/s and the step's roofline fraction of one configuration (short run, inputs resident)."""
    cfg = S.paper_configs()[name]
    L = cfg.num_layers
    Kd, Vd = zip(*[S.make_layer(cfg, l, dev) for l in range(L)])
    comp = binding.Compressor(L, cfg.num_heads, cfg.head_dim, cfg.cu_seqlens, cfg.torch_dtype, cfg.rho, cfg.gamma,
                              cfg.min_keep, device=dev.index)
    for _ in range(warmup):
        comp.compress(Kd, Vd)
    torch.cuda.synchronize(dev)
    comp.check_device_status()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        comp.compress(Kd, Vd)
    e1.record()
    torch.cuda.synchronize(dev)
    ms = e0.elapsed_time(e1) / steps
    comp.check_device_status()
    acc, rows = step_accounting(binding, comp.handle, cfg)
    s = 4 if cfg.dtype == "f32" else 2
    step_bytes = rows * (2.0 * cfg.head_dim * s + 8.0 + cfg.rho * (4.0 * cfg.head_dim * s + 4.0))
    step_flops = sum(v["flops"] for v in acc.values())
    t_bound = max(step_bytes / (peaks["hbm_gbs"] * 1e9), step_flops / (alu_peak * 1e12))
    input_gb = sum(k.numel() * k.element_size() * 2 for k in Kd) / 1e9
    comp.close()
    del Kd, Vd
    torch.cuda.empty_cache()
    return {"workload": cfg.name + ": " + cfg.note, "ms_per_step": ms, "value": cfg.total_tokens / (ms / 1000.0),
            "unit": UNIT, "steps": steps, "warmup": warmup, "t_bound_ms": 1000.0 * t_bound,
            "roofline_step_frac": t_bound / (ms / 1000.0), "input_gbytes": input_gb,
            "l2_policy": "inputs exceed L2; no flush" if input_gb > 0.2 else "inputs fit L2 (warm); launch-bound, fraction not meaningful"}


# --------------------------------------------------------------------------- main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default=DEFAULT_CONFIG)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--group-mib", type=int, default=0, help="transform group size override (MiB)")
    ap.add_argument("--streams", type=int, default=0, help="internal streams of the scoring calls (default: the library's 2)")
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: keep only the first LAYERS layers")
    ap.add_argument("--seqlens", default="", help="profiling aid: replace the config's sequence lengths (comma-separated)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing")
    ap.add_argument("--no-all-configs", action="store_true", help="skip the short runs of the other four configurations")
    ap.add_argument("--per-layer", action="store_true",
                    help="one index set per layer from the head-averaged score (fc_select_compact_ex)")
    ap.add_argument("--cpu-budget-s", type=float, default=15.0)
    ap.add_argument("--decode", action="store_true",
                    help="time the decoding-step attention on full and compressed caches instead of the compressor")
    ap.add_argument("--spectrum", action="store_true", help="time fc_power_spectrum over all layers of the config")
    ap.add_argument("--proto", action="store_true",
                    help="time one transform stage on the FP32 pipes and on the tensor pipe (measurement aid)")
    ap.add_argument("--decode-n", type=int, default=0, help="--decode: only this context length")
    ap.add_argument("--decode-rho", type=float, default=0.0, help="--decode: only this cache ratio")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.decode:
        run_decode(args)
        return
    if args.spectrum:
        run_spectrum(args)
        return
    if args.proto:
        run_proto(args)
        return

    import torch
    from paper_2511_16786_b200 import binding, replicas, synth_kv as S

    rank, world, local_rank = replicas.world_from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = replicas.init("nccl", torch.device("cuda", local_rank))
    if max(args.warmup, 0) < 3:
        args.warmup = 3

    peaks = load_peaks()
    cfg = S.paper_configs()[args.config]
    if args.layers:
        cfg = S.scaled(cfg, cfg.name, num_layers=args.layers, note=cfg.note + " (first %d layers only)" % args.layers)
    if args.seqlens:
        lens = tuple(int(x) for x in args.seqlens.split(","))
        cfg = S.scaled(cfg, cfg.name, seqlens=lens, note=cfg.note + " (sequence lengths replaced: %s)" % args.seqlens)
    dev = torch.device("cuda", local_rank)
    L = cfg.num_layers
    Kd, Vd = [], []
    for l in range(L):
        k, v = S.make_layer(cfg, l, dev)
        Kd.append(k)
        Vd.append(v)
    comp = binding.Compressor(L, cfg.num_heads, cfg.head_dim, cfg.cu_seqlens, cfg.torch_dtype, cfg.rho,
                              cfg.gamma, cfg.min_keep, device=local_rank,
                              group_bytes=(args.group_mib << 20) if args.group_mib else None,
                              per_layer=args.per_layer)
    if args.streams:
        binding.fc_set_internal_streams(comp.handle, args.streams)
    input_bytes = sum(k.numel() * k.element_size() * 2 for k in Kd)

    def barrier():
        replicas.barrier(dist, dev)

    sampler = ClockSampler(physical_gpu_index(local_rank))
    t_load0 = time.time()
    for _ in range(args.warmup):
        comp.compress(Kd, Vd)
    torch.cuda.synchronize()
    comp.check_device_status()

    # which kernel class dominates: one profiled (untimed) step per class
    shares = {}
    for name, cls in binding.KERNEL_CLASSES.items():
        binding.fc_profile_begin(comp.handle, cls)
        comp.compress(Kd, Vd)
        ms, n = binding.fc_profile_end(comp.handle)
        shares[name] = dict(ms=ms, launches=n)
    dominant = max((k for k in shares if k != "other"), key=lambda k: shares[k]["ms"])
    # the dominant kernel alone on the GPU: one more profiled step with a single internal stream
    binding.fc_set_internal_streams(comp.handle, 1)
    comp.compress(Kd, Vd)
    binding.fc_profile_begin(comp.handle, binding.KERNEL_CLASSES[dominant])
    comp.compress(Kd, Vd)
    a_ms, a_n = binding.fc_profile_end(comp.handle)
    alone_us = 1000.0 * a_ms / max(1, a_n)
    binding.fc_set_internal_streams(comp.handle, args.streams or 2)
    comp.compress(Kd, Vd)
    torch.cuda.synchronize()

    # timed region
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    launches0 = binding.fc_launch_count(comp.handle)
    # inside the timed region every 7th launch of the dominant kernel is bracketed by an event pair
    prof_stride = 7
    binding.fc_profile_stride(comp.handle, prof_stride)
    binding.fc_profile_begin(comp.handle, binding.KERNEL_CLASSES[dominant],
                             max(1, shares[dominant]["launches"]) * args.steps // prof_stride + 8)
    t_wall0 = time.time()
    ev0.record()
    for _ in range(args.steps):
        comp.compress(Kd, Vd)
    ev1.record()
    barrier()
    t_wall1 = time.time()
    elapsed_ms = ev0.elapsed_time(ev1)
    dom_ms, dom_launches = binding.fc_profile_end(comp.handle)
    launches = binding.fc_launch_count(comp.handle) - launches0
    clocks = sampler.stop(t_wall0, t_wall1)
    comp.check_device_status()
    elapsed_ms = replicas.max_over_ranks(elapsed_ms, dist, dev)
    ms_per_step = elapsed_ms / args.steps
    tokens = cfg.total_tokens
    value = replicas.whole_job_rate(tokens, world, ms_per_step)

    # roofline of the dominant kernel and of the whole step
    acc, rows = step_accounting(binding, comp.handle, cfg)
    props = torch.cuda.get_device_properties(dev)
    # ALU peak: nominal (SMs x 128 lanes x 2 x max clock) and what a pure FMA loop sustains in this run; the
    # fractions below divide by the nominal figure (the larger of the two), the measured one is reported beside it
    alu_peak = props.multi_processor_count * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12   # TFLOP/s
    alu_peak_measured = binding.fc_measure_fp32_peak(comp.handle)
    d_acc = acc[dominant]
    launches_per_step = max(1, shares[dominant]["launches"])
    avg_launch_s = dom_ms / 1000.0 / max(1, dom_launches)   # average over the sampled launches of the timed region
    dom_s = avg_launch_s * launches_per_step                # device seconds of that class per step
    t_alu = d_acc["flops"] / (alu_peak * 1e12)
    t_hbm = d_acc["bytes"] / (peaks["hbm_gbs"] * 1e9)
    if t_alu >= t_hbm:
        roof = dict(bound="alu", achieved=d_acc["flops"] / dom_s / 1e12, peak=alu_peak, unit="TFLOP/s")
    else:
        roof = dict(bound="hbm", achieved=d_acc["bytes"] / dom_s / 1e9, peak=peaks["hbm_gbs"], unit="GB/s")
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get((args.config, dominant))
    roof.update(kernel=dominant, launches_per_step=launches_per_step, launches_timed=dom_launches,
                avg_launch_us=1000.0 * dom_ms / max(1, dom_launches), peak_source=(
                    "%d SMs x %d FP32 lanes x 2 x %.0f MHz" % (props.multi_processor_count, FP32_LANES_PER_SM,
                                                              peaks["sm_max_mhz"])
                    if roof["bound"] == "alu" else "MEASURED_PEAKS.json hbm_gbs (%s)" % peaks["source"]),
                peak_measured=alu_peak_measured if roof["bound"] == "alu" else None,
                frac_of_measured=(roof["achieved"] / alu_peak_measured) if roof["bound"] == "alu" else None,
                peak_measured_source="fc_measure_fp32_peak: packed FMA loop on every SM, this run",
                avg_launch_us_alone=alone_us,
                class_ms_per_step={k: v["ms"] for k, v in shares.items()},
                # device time summed over the kernel classes divided by the step: above 1 because the
                # library runs consecutive head groups on two internal streams, whose kernels share the GPU
                # (a launch lasts longer co-scheduled than alone)
                overlap_factor=sum(v["ms"] for v in shares.values()) / ms_per_step)
    s = 4 if cfg.dtype == "f32" else 2
    step_bytes = rows * (2.0 * cfg.head_dim * s + 8.0 + cfg.rho * (4.0 * cfg.head_dim * s + 4.0))
    step_flops = sum(v["flops"] for v in acc.values())
    t_bound = max(step_bytes / (peaks["hbm_gbs"] * 1e9), step_flops / (alu_peak * 1e12))
    roof_step = dict(bound="alu" if step_flops / (alu_peak * 1e12) >= step_bytes / (peaks["hbm_gbs"] * 1e9) else "hbm",
                     t_bound_ms=1000.0 * t_bound, frac=t_bound / (ms_per_step / 1000.0),
                     gflop=step_flops / 1e9, gbytes=step_bytes / 1e9,
                     ms_x_sm_mhz=ms_per_step * (clocks["sm_mhz"] or 0.0))

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg.name + ": " + cfg.note + (", one index set per layer" if args.per_layer else ""),
                   "layers": L, "kv_heads": cfg.num_heads,
                   "head_dim": cfg.head_dim, "seqlens": list(cfg.seqlens), "storage_dtype": cfg.dtype,
                   "rho": cfg.rho, "gamma": cfg.gamma, "replicas": world,
                   "l2_policy": "inputs (%.2f GB) exceed L2; no flush" % (input_bytes / 1e9)},
        "clocks": clocks, "gpu_launches": int(launches),
        "roofline": roof, "roofline_step": roof_step,
    }

    # the same step replayed from a CUDA graph (reported beside the headline, which stays the plain call
    # sequence because only that one carries the per-kernel event timing)
    if not args.no_graph and world == 1:
        graph = comp.capture(Kd, Vd)
        for _ in range(3):
            graph.replay()
        barrier()
        ev0.record()
        for _ in range(args.steps):
            graph.replay()
        ev1.record()
        barrier()
        g_ms = replicas.max_over_ranks(ev0.elapsed_time(ev1), dist, dev) / args.steps
        comp.check_device_status()
        out["cuda_graph"] = {"ms_per_step": g_ms, "value": replicas.whole_job_rate(tokens, world, g_ms), "unit": UNIT}
        del graph

    # end to end through fc_compress_host: K and V start in page-locked host memory, the compacted caches
    # end there; every step's copies in and out are inside the timed region (consecutive steps overlap
    # one step's copies back with the next step's copies in, as a serving loop would)
    if not args.no_e2e:
        hostK = [k.cpu().pin_memory() for k in Kd]
        hostV = [v.cpu().pin_memory() for v in Vd]
        hc = binding.HostCompressor(L, cfg.num_heads, cfg.head_dim, cfg.cu_seqlens, cfg.torch_dtype, cfg.rho,
                                    cfg.gamma, cfg.min_keep, device=dev.index)
        results = [hc.new_result(), hc.new_result()]

        def e2e_steps(n):
            for i in range(n):
                hc.compress(hostK, hostV, results[i % 2])
            torch.cuda.synchronize(dev)

        e2e_steps(2)
        hc.check_device_status()
        n_e2e = max(3, min(10, args.steps))
        barrier()
        t0 = time.perf_counter()
        e2e_steps(n_e2e)
        barrier()
        e2e_ms = 1000.0 * (time.perf_counter() - t0) / n_e2e
        e2e_ms = replicas.max_over_ranks(e2e_ms, dist, dev)
        rows = int(results[0].layer_rows[L])
        d2h_bytes = (2 * rows * cfg.num_heads * cfg.head_dim * s + rows * cfg.num_heads * 4
                     + results[0].budgets.numel() * 4 + results[0].offsets.numel() * 8)
        out["e2e"] = {"value": replicas.whole_job_rate(tokens, world, e2e_ms), "unit": UNIT,
                      "h2d_bytes_per_step": int(input_bytes), "d2h_bytes_per_step": int(d2h_bytes),
                      "ms_per_step": e2e_ms, "steps": n_e2e, "call": "fc_compress_host"}
        hc.close()
        del hostK, hostV, results, hc

    # CPU baseline: the oracle on this machine's host cores, bounded sample (rank 0, single-GPU run only)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_layers_host = min(L, 8)
        Ks_host = [Kd[l].float().cpu().numpy() for l in range(n_layers_host)]
        Vs_host = [Vd[l].float().cpu().numpy() for l in range(n_layers_host)]
        cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
        tps, used, el = oracle_sample(cfg, Ks_host, Vs_host, args.cpu_budget_s, threads=cores)
        out["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "host_cores": os.cpu_count(),
                               "sample": "%d of %d layers (all heads, all sequences), %.1f s on %d host threads "
                                         "(one oracle call per layer and head), scaled by the layer count"
                                         % (used, L, el, cores)}
    comp.close()
    # the other four configurations, briefly: 3 warm-up steps, 10 timed, same accounting
    if world == 1 and args.config == DEFAULT_CONFIG and not args.layers and not args.seqlens and not args.no_all_configs:
        del Kd, Vd
        torch.cuda.empty_cache()
        out["all_configs"] = {args.config: {"ms_per_step": ms_per_step, "value": value, "unit": UNIT,
                                            "roofline_step_frac": roof_step["frac"]}}
        for name in ("cfg1", "cfg2", "cfg4", "cfg5"):
            out["all_configs"][name] = quick_config(torch, binding, S, name, dev, peaks, alu_peak)
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
