#!/usr/bin/env python
"""Benchmark of the RT prefill hot path on synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4|c2|c3|c5_N<len>] [--sched tiled|naive]
    python bench.py --impl reference ...          # times the fp64 CPU oracle instead

A step is one pass of the whole hot path (pre-pass, every leaf launch, every cross tile) over
one batch.  `value` counts tokens/s with inputs resident in HBM; `e2e` runs the same call with
the batch coming from pinned host memory and the layer output read back, copies inside the
timed region.  With N > 1 (torchrun) every rank runs an independent replica of the workload on
its own GPU -- the path shards over the batch only, so there is no collective on the data
path -- and the line reports all ranks' tokens over the slowest rank's time.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "rt_prefill_tokens_per_s"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 256 << 20


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


def leaf_traffic_table():
    """DRAM bytes (read + write) of ONE leaf launch per workload, from single-launch ncu captures; the table lives in
    profiles/leaf_mma_kernel_dram_bytes.md as rows `| workload | bytes |` (a launch stages its weight rows once,
    everything else stays in L2).  Workloads without a row report null."""
    out = {}
    path = os.path.join(ROOT, "profiles", "leaf_mma_kernel_dram_bytes.md")
    if os.path.exists(path):
        for ln in open(path):
            f = [t.strip() for t in ln.strip().strip("|").split("|")]
            if len(f) >= 2 and f[1].isdigit():
                out[f[0]] = int(f[1])
    return out


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def mark(self, wait_s=2.0):
        """Waits for nvidia-smi's first line (its start-up can outlast a short timed region), then drops what
        was sampled so far: only samples taken after this call count."""
        t0 = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - t0 < wait_s:
            time.sleep(0.01)
        self.skip = len(self.lines)

    def count(self):
        return len(self.lines) - getattr(self, "skip", 0)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines[getattr(self, "skip", 0):]:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def alibi_slopes(n_heads, max_bias=8.0):
    """Geometric slopes 2^(-max_bias h / H), h = 1..H (the paper's experiments: maximum bias 8)."""
    return [2.0 ** (-max_bias * (h + 1) / n_heads) for h in range(n_heads)]


def get_workload(name, batch=0):
    import dataclasses
    from paper_2604_21215_b200 import inputs
    wl = inputs.sweep(int(name[4:])) if name.startswith("c5_N") else inputs.WORKLOADS[name]
    return dataclasses.replace(wl, B=batch) if batch else wl


def config_dict(wl, sched, extra=None):
    c = {"workload": wl.name, "n_layers": wl.n_layers, "B": wl.B, "N": wl.N, "d_model": wl.d_model,
         "n_heads": wl.n_heads, "d_ff": wl.d_ff, "vocab": wl.vocab, "sched": sched,
         "l2": f"flushed between timed steps ({L2_FLUSH_BYTES >> 20} MiB write)"}
    if extra:
        c.update(extra)
    return c


# ------------------------------------------------------------------------------------ oracle arm

def oracle_sample(wl, data, n_pos, recur_block=0):
    """Runs the oracle, as it stands, on the first n_pos positions of the workload; returns seconds."""
    from oracle import RTConfig, RTWeights, layer_blockrec, layer_seq, stack_prefill
    cfg = RTConfig(wl.d_model, wl.n_heads, wl.head_dim, wl.d_ff, residual_scale=wl.residual_scale,
                   alibi_slopes=data["layers"][0].get("alibi_slopes"))
    layers = [RTWeights(**{k: v for k, v in lw.items() if k != "alibi_slopes"}) for lw in data["layers"]]
    t0 = time.perf_counter()
    if wl.vocab:
        stack_prefill(cfg, layers, data["emb"], None, data["ids"][:, :n_pos])
    elif recur_block > 1:
        layer_blockrec(cfg, layers[0], data["x"][:, :n_pos], recur_block)
    else:
        layer_seq(cfg, layers[0], data["x"][:, :n_pos])
    return time.perf_counter() - t0


def oracle_cores():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def sample_positions(wl):
    # about 10-30 s of CPU work: the first positions of every sequence of the batch
    n = 1024 if wl.d_model <= 768 else 512
    if wl.n_layers > 1:
        n = max(32, n // wl.n_layers)
    if wl.B > 64:                                      # wide batches: keep the sample near 16 k tokens
        n = max(8, 16384 // wl.B)
    return min(wl.N, n)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2604_21215_b200 import inputs
    wl = get_workload(args.workload, args.batch)
    data = inputs.make_inputs(wl)
    n_pos = sample_positions(wl)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(wl, data, min(n_pos, 64))
    times = [oracle_sample(wl, data, n_pos) for _ in range(args.steps)]
    tot = sum(times)
    value = wl.B * n_pos * args.steps / tot
    cores = oracle_cores()
    sample = (f"fp64 oracle (numpy + BLAS) on the first {n_pos} of {wl.N} positions of all {wl.B} sequences per step "
              "(the positions the CUDA arm's cpu_baseline times); later positions cost more (longer prefixes), so the "
              "full workload would be slower per token")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(wl, "oracle", {"l2": "n/a (CPU)"}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------ CUDA arm

def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2604_21215_b200 import inputs, replicas, rt

    world, rank, local = replicas.world_info(os.environ)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = get_workload(args.workload, args.batch)
    data = inputs.make_inputs(wl)
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    leaf_kw = {"leaf": args.leaf} if args.leaf else {}
    if args.recur_block > 1:
        leaf_kw["recur_block"] = args.recur_block
    stream = torch.cuda.current_stream(dev)

    if args.alibi:                                     # the same slopes for every layer
        for lw in data["layers"]:
            lw["alibi_slopes"] = alibi_slopes(wl.n_heads)
    if wl.vocab:
        model = rt.Stack(wl.n_layers, wl.d_model, wl.n_heads, wl.d_ff, wl.vocab, dtype=wl.dtype, device=str(dev),
                         sched=args.sched, residual_scale=wl.residual_scale, **leaf_kw)
        model.set_weights(data["layers"], data["emb"])
        model.reserve(wl.B, wl.N)
        host_in = torch.from_numpy(data["ids"]).pin_memory()
        dev_in = host_in.to(dev)
        dev_out = torch.empty((wl.B, wl.N, wl.d_model), dtype=tdt, device=dev)
        logits = torch.empty((wl.B, wl.vocab), dtype=torch.float32, device=dev)
        host_out = torch.empty((wl.B, wl.vocab), dtype=torch.float32).pin_memory()
        call = lambda inp: model.prefill_device(inp, dev_out, logits)
        result = logits
    else:
        model = rt.Layer(wl.d_model, wl.n_heads, wl.d_ff, dtype=wl.dtype, device=str(dev), sched=args.sched,
                         residual_scale=wl.residual_scale, **leaf_kw)
        model.set_weights(data["layers"][0])
        model.reserve(wl.B, wl.N)
        host_in = torch.from_numpy(data["x"]).to(tdt).pin_memory()
        dev_in = host_in.to(dev)
        dev_out = torch.empty((wl.B, wl.N, wl.d_model), dtype=tdt, device=dev)
        host_out = torch.empty((wl.B, wl.N, wl.d_model), dtype=tdt).pin_memory()
        call = lambda inp: model.prefill_device(inp, dev_out)
        result = dev_out
    dev_in2 = torch.empty_like(dev_in)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    tokens = wl.B * wl.N

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize(dev)

    def timed(fn, steps):
        """Each step bracketed by its own pair of CUDA events on the launching stream; L2 flushed between."""
        evs = []
        for _ in range(steps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize(dev)
        return [a.elapsed_time(b) for a, b in evs]

    def e2e_step():
        dev_in2.copy_(host_in, non_blocking=True)
        call(dev_in2)
        host_out.copy_(result, non_blocking=True)

    if args.profile_one_call:
        # profiling mode (for ncu byte counters): exactly one call, no warm-up, no bench line
        call(dev_in)
        torch.cuda.synchronize(dev)
        c = rt.rt_plan_counters(model.cfg, wl.B, wl.N, wl.n_layers, wl.vocab)
        print(json.dumps({"profile_one_call": wl.name, "sched": args.sched, "status": int(model.status()),
                          "model_bytes": c["model_bytes_read"] + c["model_bytes_written"],
                          "model_kv_bytes_read": c["kv_bytes_read"], "leaf_kv_bytes_l2": c["leaf_kv_bytes_l2"]}))
        return 0
    for _ in range(max(args.warmup, 3)):
        call(dev_in)
    torch.cuda.synchronize(dev)
    if model.status() != rt.RT_OK:
        raise SystemExit("device status after warm-up: " + rt.rt_status_string(model.status()))

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        sampler.mark()
    barrier()
    rt.rt_profile_enable(True)
    rt.rt_profile_read()
    wall0 = time.perf_counter()
    ms = timed(lambda: call(dev_in), args.steps)
    barrier()
    wall = time.perf_counter() - wall0
    prof = rt.rt_profile_read()
    rt.rt_profile_enable(False)
    total_ms = sum(ms)
    # end to end: pinned host input -> device, the call, result -> pinned host
    e2e_step(); torch.cuda.synchronize(dev)
    barrier()
    e2e_ms = timed(e2e_step, args.steps)
    barrier()
    if rank == 0 and sampler.proc is not None and sampler.count() == 0:
        # both timed regions ended inside one sampling period: keep the same step running (untimed) until a sample lands
        t0 = time.perf_counter()
        while sampler.count() == 0 and time.perf_counter() - t0 < 1.0:
            call(dev_in)
            torch.cuda.synchronize(dev)
    clocks = sampler.stop() if rank == 0 else None
    e2e_total = sum(e2e_ms)
    if model.status() != rt.RT_OK:
        raise SystemExit("device status after the timed region: " + rt.rt_status_string(model.status()))

    total_ms, e2e_total = replicas.max_over_ranks([total_ms, e2e_total], device=dev)

    if rank == 0:
        counters = rt.rt_plan_counters(model.cfg, wl.B, wl.N, wl.n_layers, wl.vocab)
        peaks = measured_peaks()
        e = 2 if wl.dtype == "bf16" else 4
        d, f, B = wl.d_model, wl.d_ff, wl.B
        # dominant kernel: the leaf recurrence.  Algorithmic bytes per token step = the chain
        # weights once (shared by the B sequences) + activation rows; per launch x the leaf length.
        chain_w = (3 * d * d + 2 * d * f) * e
        act = (7 * e + 4) * d * B
        n_leaf = max(prof["leaf"]["launches"], 1)
        tok_steps_per_launch = wl.N * wl.n_layers * args.steps / n_leaf
        leaf_ms = prof["leaf"]["ms"] / n_leaf
        alg_bytes = (chain_w + act) * tok_steps_per_launch
        achieved = alg_bytes / (leaf_ms * 1e-3) / 1e9 if leaf_ms > 0 else 0.0
        roofline = {"kernel": "leaf_mma_kernel" if (wl.dtype == "bf16" and args.sched == "tiled") else "leaf_kernel", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "traffic": leaf_traffic_table().get(wl.name),
                    "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_ms": leaf_ms,
                    "us_per_token_step": 1e3 * leaf_ms / max(tok_steps_per_launch, 1),
                    "note": "weights stay in shared memory for a whole launch, so the kernel is bound by the "
                            "latency of its five all-to-all exchanges per token step (L2 round trips), not by HBM; "
                            "the fraction is the effective weight+activation stream against the HBM copy peak and "
                            "traffic is the DRAM bytes ncu counted for one launch"}
        if wl.B > 64:
            # wide batches: the token step is a chain of dense products over the B rows (tcgen05), one position at
            # a time; the leaf class of the profile holds them together with the small in-leaf attention kernels
            tf_peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))).get("bf16_tflops_sustained", 1403.5)) \
                if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else 1400.0
            flops = 2.0 * B * (5 * d * d + 2 * d * f) * wl.N * wl.n_layers * args.steps      # W_o, W_up, W_down, W_k, W_v per step
            ms_all = prof["leaf"]["ms"]
            achieved = flops / (ms_all * 1e-3) / 1e12 if ms_all > 0 else 0.0
            roofline = {"kernel": "dense_tc_kernel (wide-batch token steps, with their small kernels)", "bound": "tensor",
                        "achieved": achieved, "peak": tf_peak, "unit": "TFLOP/s", "frac": achieved / tf_peak,
                        "peak_source": "measured (sustained)", "traffic": None,
                        "us_per_token_step": 1e3 * ms_all / max(wl.N * wl.n_layers * args.steps, 1),
                        "note": "M = B rows per product: each token step is seven short dependent launches, so launch latency "
                                "and the L2 stream of the weights, not the tensor pipe, set the time"}
        if args.recur_block > 1:
            # recurrence over blocks: every block is a parallel sweep of dense products and attention tiles
            tf_peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))).get("bf16_tflops_sustained", 1403.5)) \
                if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else 1400.0
            tok_all = B * wl.N * wl.n_layers * args.steps
            flops = 2.0 * tok_all * (5 * d * d + 2 * d * f) + 6.0 * tok_all * d * d + 2.0 * B * d * wl.N * (wl.N - 1) * wl.n_layers * args.steps
            ms_all = prof["leaf"]["ms"] + prof["tile"]["ms"] + prof["prepass"]["ms"]
            achieved = flops / (ms_all * 1e-3) / 1e12 if ms_all > 0 else 0.0
            roofline = {"kernel": "dense_tc_kernel + tile_tc_kernel (recurrence over blocks)", "bound": "tensor",
                        "achieved": achieved, "peak": tf_peak, "unit": "TFLOP/s", "frac": achieved / tf_peak,
                        "peak_source": "measured (sustained)", "traffic": None,
                        "us_per_token_step": 1e3 * ms_all / max(wl.N * wl.n_layers * args.steps, 1),
                        "note": "all products of a call (projections, chain, attention) over the summed kernel time"}
        tile_ms = prof["tile"]["ms"]
        tile_tflops = (counters["flops_tile"] * args.steps / (tile_ms * 1e-3) / 1e12) if tile_ms > 0 else None
        n_pos = sample_positions(wl)
        oracle_sample(wl, data, min(n_pos, 16), args.recur_block)         # untimed: starts the BLAS threads
        t_cpu = oracle_sample(wl, data, n_pos, args.recur_block)
        cpu = {"value": wl.B * n_pos / t_cpu, "unit": UNIT, "cores": oracle_cores(), "kind": "oracle",
               "sample": f"first {n_pos} of {wl.N} positions, all {wl.B} sequences, one warmed run ({t_cpu:.1f} s); "
                         "`--impl reference` times the same positions"}
        launches = sum(v["launches"] for v in prof.values())
        # the pre-pass group is three kernels, every other group one
        gpu_launches = int(launches + 2 * prof["prepass"]["launches"])
        if wl.B > 64:
            # wide batches: per position one in-leaf attention launch (which also leaves c = o/l), three dense products
            # (W_o and W_down split at this shape: + a reduction each, which also leaves the row norms) and the K/V
            # projection; per call the pre-pass (3) and one cross tile per leaf boundary
            lf = int(model.cfg.leaf) or 32
            n_leaves = (wl.N + lf - 1) // lf
            per_call = wl.N + 3 * wl.N + 2 * wl.N + wl.N + 3 + (n_leaves - 1)
            gpu_launches = int(per_call * wl.n_layers * args.steps)
        h2d = host_in.numel() * host_in.element_size()
        d2h = host_out.numel() * host_out.element_size()
        line = {"metric": METRIC, "value": replicas.aggregate_tokens_per_s(tokens, args.steps, world, total_ms), "unit": UNIT,
                "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16/f32-accumulate" if wl.dtype == "bf16" else "f32",
                "data": "synthetic", "config": config_dict(wl, args.sched, {"alibi": bool(args.alibi), "recur_block": int(args.recur_block), "leaf": int(model.cfg.leaf) or (32 if wl.B > 64 else 64),
                                                                            "parallelism": f"replicas x{world}"}),
                "clocks": clocks,
                "e2e": {"value": replicas.aggregate_tokens_per_s(tokens, args.steps, world, e2e_total), "unit": UNIT,
                        "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
                "gpu_launches": gpu_launches,
                "roofline": roofline, "cpu_baseline": cpu,
                "kernels": {k: {"ms_per_step": v["ms"] / args.steps, "launches_per_step": v["launches"] / args.steps}
                            for k, v in prof.items()},
                "tile_tflops": tile_tflops,
                "model": {"hbm_bytes_per_step": counters["model_bytes_read"] + counters["model_bytes_written"],
                          "kv_bytes_read_per_step": counters["kv_bytes_read"],
                          "flops_tile": counters["flops_tile"], "flops_leaf": counters["flops_leaf"],
                          "flops_gemm": counters["flops_gemm"]},
                "wall_s_timed_region": wall}
        if world == 1 and args.also:
            line["also"] = measure_also([n for n in args.also.split(",") if n and n != wl.name], 3, dev, stream, flush)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def measure_also(names, steps, dev, stream, flush):
    """Tokens/s of other single-layer workloads in this process (few steps each; same timing rules as the main line)."""
    import torch
    from paper_2604_21215_b200 import inputs, rt
    out = {}
    for name in names:
        wl = get_workload(name)
        data = inputs.make_inputs(wl)
        tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        layer = rt.Layer(wl.d_model, wl.n_heads, wl.d_ff, dtype=wl.dtype, device=str(dev), residual_scale=wl.residual_scale)
        layer.set_weights(data["layers"][0])
        layer.reserve(wl.B, wl.N)
        x = torch.from_numpy(data["x"]).to(tdt).to(dev)
        z = torch.empty_like(x)
        for _ in range(3):
            layer.prefill_device(x, z)
        torch.cuda.synchronize(dev)
        rt.rt_profile_enable(True)
        rt.rt_profile_read()
        evs = []
        for _ in range(steps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); layer.prefill_device(x, z); b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize(dev)
        prof = rt.rt_profile_read()
        rt.rt_profile_enable(False)
        if layer.status() != rt.RT_OK:
            out[name] = {"error": rt.rt_status_string(layer.status())}
            continue
        ms = sum(a.elapsed_time(b) for a, b in evs) / steps
        out[name] = {"tokens_per_s": wl.B * wl.N / (ms * 1e-3), "ms_per_step": ms, "steps": steps, "B": wl.B, "N": wl.N,
                     "d_model": wl.d_model, "us_per_token_step": 1e3 * prof["leaf"]["ms"] / (wl.N * steps),
                     "tile_ms_per_step": prof["tile"]["ms"] / steps}
        del layer, x, z
        torch.cuda.empty_cache()
    return out


def run_tile_bench(args):
    """Times Algorithm 2 alone (rt_update_tile) per tile size, in the shape the workload's prefill uses it:
    queries [P, 2P) against the pairs [0, P) for all B*H (sequence, head) pairs; prints one JSON object."""
    import torch
    from paper_2604_21215_b200 import rt
    wl = get_workload(args.workload, args.batch)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(
        os.path.join(ROOT, "MEASURED_PEAKS.json")) else {"bf16_tflops": 1590.0}
    cfg = rt.make_config(wl.d_model, wl.n_heads, wl.d_ff, dtype=wl.dtype)
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    ws = torch.zeros(256, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)
    out = []
    g = torch.Generator(device=dev); g.manual_seed(BASE_TILE_SEED)
    slopes = torch.tensor(alibi_slopes(wl.n_heads), dtype=torch.float32, device=dev) if args.alibi else None
    alibi_ptr = slopes.data_ptr() if args.alibi else None
    for P in (64, 128, 256, 512, 1024, 2048, 4096):
        if P > wl.N // 2 and not args.tile_bench_all:
            break
        rows = 2 * P
        q = torch.randn((rows, wl.B, wl.d_model), generator=g, device=dev).to(tdt)
        k = torch.randn((rows, wl.B, wl.d_model), generator=g, device=dev).to(tdt)
        v = torch.randn((rows, wl.B, wl.d_model), generator=g, device=dev).to(tdt)
        o = torch.zeros((rows, wl.B, wl.d_model), dtype=torch.float32, device=dev)
        m = torch.zeros((rows, wl.B, wl.n_heads), dtype=torch.float32, device=dev)
        l = torch.ones((rows, wl.B, wl.n_heads), dtype=torch.float32, device=dev)
        call = lambda: rt.rt_update_tile(cfg, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), m.data_ptr(),
                                         l.data_ptr(), wl.B, rows, rows, P, 2 * P, 0, P, alibi_ptr, ws.data_ptr(), stream.cuda_stream)
        for _ in range(3):
            assert call() == rt.RT_OK
        evs = []
        for _ in range(args.steps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); call(); b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize(dev)
        assert rt.rt_get_status(ws.data_ptr()) == rt.RT_OK
        ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
        flops = 4.0 * P * P * 64 * wl.B * wl.n_heads
        tf = flops / (ms * 1e-3) / 1e12
        out.append({"P": P, "ms": ms, "tflops": tf, "frac_of_measured_bf16_peak": tf / peaks["bf16_tflops"]})
    print(json.dumps({"tile_bench": wl.name, "B": wl.B, "H": wl.n_heads, "dtype": wl.dtype, "alibi": bool(args.alibi),
                      "peak_tflops": peaks["bf16_tflops"], "tiles": out}))
    return 0


def run_decode_bench(args):
    """Times rt_decode_step (one new token per sequence through every layer, attention over the whole cache) at a
    given cache length, in the stack shape of the workload; prints one JSON object.  The caches are filled with
    seeded random values (the step's cost does not depend on them)."""
    import torch
    from paper_2604_21215_b200 import inputs, rt
    wl = get_workload(args.workload, args.batch)
    if not wl.vocab:
        raise SystemExit("--decode-bench needs a stack workload (c4)")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    data = inputs.make_inputs(wl, N=8)
    st = rt.Stack(wl.n_layers, wl.d_model, wl.n_heads, wl.d_ff, wl.vocab, dtype=wl.dtype, residual_scale=wl.residual_scale)
    st.set_weights(data["layers"], data["emb"])
    out = []
    g = torch.Generator(device=dev); g.manual_seed(BASE_TILE_SEED + 1)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)
    esz = 2 if wl.dtype == "bf16" else 4
    for pos in (1024, 4096, 16384):
        n_max = pos + args.steps + 4
        st.k_caches = []
        st.reserve(wl.B, 1, n_max)
        for t in st.k_caches + st.v_caches:
            t.copy_(torch.randn(t.shape, generator=g, device=dev).to(t.dtype))
        need = rt.rt_workspace_bytes(st.cfg, wl.B, 1, wl.n_layers)
        if st.ws is None or st.ws.numel() < need:
            st.ws = torch.zeros(need, dtype=torch.uint8, device=dev)
        ids = torch.randint(0, wl.vocab, (wl.B,), generator=g, device=dev, dtype=torch.int32)
        logits = torch.empty((wl.B, wl.vocab), dtype=torch.float32, device=dev)

        def step(p):
            rt._check(rt.rt_decode_step(st.cfg, wl.n_layers, st.layers, st.emb.data_ptr(), None, wl.vocab, ids.data_ptr(),
                                        wl.B, p, logits.data_ptr(), st._kp, st._vp, st.N_max, st.ws.data_ptr(),
                                        st.ws.numel(), stream.cuda_stream), "rt_decode_step")
        for i in range(3):
            step(pos + i)
        evs = []
        for i in range(args.steps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); step(pos + 3 + i); b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize(dev)
        assert st.status() == rt.RT_OK
        ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
        cache_bytes = 2.0 * pos * wl.B * wl.d_model * esz * wl.n_layers
        weight_bytes = (4 * wl.d_model ** 2 + 2 * wl.d_model * wl.d_ff) * esz * wl.n_layers + wl.vocab * wl.d_model * esz
        gbs = (cache_bytes + weight_bytes) / (ms * 1e-3) / 1e9
        out.append({"pos": pos, "ms_per_step": ms, "tokens_per_s": wl.B / (ms * 1e-3), "cache_bytes": cache_bytes,
                    "weight_bytes": weight_bytes, "achieved_gbs": gbs, "frac_of_measured_hbm_peak": gbs / peaks["hbm_gbs"]})
    print(json.dumps({"decode_bench": wl.name, "B": wl.B, "n_layers": wl.n_layers, "dtype": wl.dtype,
                      "peak_gbs": peaks["hbm_gbs"], "points": out}))
    return 0


def run_recompute_bench(args):
    """Times rt_layer_recompute (the parallel sweep of Sec. 6: all positions at once, given the outputs) on the
    workload's single-layer shape; prints one JSON object with the per-class kernel times and the tensor rate."""
    import torch
    from paper_2604_21215_b200 import inputs, rt
    wl = get_workload(args.workload, args.batch)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(
        os.path.join(ROOT, "MEASURED_PEAKS.json")) else {"bf16_tflops": 1590.0}
    import dataclasses
    if wl.vocab:
        wl = dataclasses.replace(wl, vocab=0, n_layers=1)
    data = inputs.make_inputs(wl)
    lw = data["layers"][0]
    if args.alibi:
        lw["alibi_slopes"] = alibi_slopes(wl.n_heads)
    layer = rt.Layer(wl.d_model, wl.n_heads, wl.d_ff, dtype=wl.dtype, residual_scale=wl.residual_scale)
    layer.set_weights(lw)
    layer.reserve(wl.B, wl.N)
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    x = torch.from_numpy(data["x"]).to(tdt).to(dev)
    g = torch.Generator(device=dev); g.manual_seed(BASE_TILE_SEED + 2)
    zc = (x.float() + 0.5 * torch.randn(x.shape, generator=g, device=dev)).to(tdt)
    zo = torch.empty_like(x)
    need = rt.rt_recompute_workspace_bytes(layer.cfg, wl.B, wl.N)
    ws = torch.zeros(need, dtype=torch.uint8, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    def call():
        rt._check(rt.rt_layer_recompute(layer.cfg, layer.w, x.data_ptr(), zc.data_ptr(), wl.B, wl.N, zo.data_ptr(),
                                        layer.k_cache.data_ptr(), layer.v_cache.data_ptr(), layer.N_max, ws.data_ptr(),
                                        ws.numel(), stream.cuda_stream), "rt_layer_recompute")
    for _ in range(max(3, args.warmup)):
        call()
    torch.cuda.synchronize(dev)
    rt.rt_profile_enable(True)
    rt.rt_profile_read()
    evs = []
    for _ in range(args.steps):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); call(); b.record(stream)
        evs.append((a, b))
    torch.cuda.synchronize(dev)
    prof = rt.rt_profile_read()
    rt.rt_profile_enable(False)
    assert rt.rt_get_status(ws.data_ptr()) == rt.RT_OK
    ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
    tok, d, f = wl.B * wl.N, wl.d_model, wl.d_ff
    flops_proj = 10.0 * tok * d * d
    flops_chain = 2.0 * tok * d * d + 4.0 * tok * d * f
    flops_attn = 2.0 * wl.B * d * wl.N * (wl.N - 1)
    tf = (flops_proj + flops_chain + flops_attn) / (ms * 1e-3) / 1e12
    per = {k: v["ms"] / args.steps for k, v in prof.items()}
    print(json.dumps({"recompute_bench": wl.name, "B": wl.B, "N": wl.N, "d_model": d, "d_ff": f, "dtype": wl.dtype,
                      "alibi": bool(args.alibi), "ms_per_call": ms, "tokens_per_s": tok / (ms * 1e-3), "tflops": tf,
                      "frac_of_measured_bf16_peak": tf / peaks["bf16_tflops"], "peak_tflops": peaks["bf16_tflops"],
                      "gflop": {"projections": flops_proj / 1e9, "chain": flops_chain / 1e9, "attention": flops_attn / 1e9},
                      "ms_by_class": {"projections": per.get("prepass"), "attention": per.get("tile"),
                                      "chain": per.get("other")}}))
    return 0


def run_backward_bench(args):
    """Times rt_layer_backward (Sec. 6, the backward pass: parallel sweep of the intermediates, reverse loop over the
    positions, batched products) next to the forward pass on the workload's single-layer shape; one JSON object."""
    import dataclasses
    import torch
    from paper_2604_21215_b200 import inputs, rt
    wl = get_workload(args.workload, args.batch)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    if wl.vocab:
        wl = dataclasses.replace(wl, vocab=0, n_layers=1)
    data = inputs.make_inputs(wl)
    lw = data["layers"][0]
    if args.alibi:
        lw["alibi_slopes"] = alibi_slopes(wl.n_heads)
    layer = rt.Layer(wl.d_model, wl.n_heads, wl.d_ff, dtype=wl.dtype, residual_scale=wl.residual_scale)
    layer.set_weights(lw)
    layer.reserve(wl.B, wl.N)
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    d, f = wl.d_model, wl.d_ff
    x = torch.from_numpy(data["x"]).to(tdt).to(dev)
    z = torch.empty_like(x)
    g = torch.Generator(device=dev); g.manual_seed(BASE_TILE_SEED + 3)
    dz = torch.randn(x.shape, generator=g, device=dev, dtype=torch.float32)
    dx = torch.empty_like(dz)
    ws = torch.zeros(rt.rt_backward_workspace_bytes(layer.cfg, wl.B, wl.N), dtype=torch.uint8, device=dev)
    grads, keep = rt.RtLayerGrads(), []
    for n, shape in (("w_q", (d, d)), ("w_k", (d, d)), ("w_v", (d, d)), ("w_o", (d, d)), ("w_up", (f, d)), ("w_down", (d, f))):
        keep.append(torch.empty(shape, dtype=torch.float32, device=dev))
        setattr(grads, n, keep[-1].data_ptr())
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    def timed(fn):
        for _ in range(max(3, args.warmup)):
            fn()
        torch.cuda.synchronize(dev)
        evs = []
        for _ in range(args.steps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize(dev)
        return sum(a.elapsed_time(b) for a, b in evs) / len(evs)

    bwd = lambda: layer.backward_device(x, z, dz, dx, grads, ws)
    if args.profile_one_call:
        # profiling mode (launch list under ncu): the forward pass once for z, ONE backward call, no bench line
        layer.prefill_device(x, z)
        bwd()
        torch.cuda.synchronize(dev)
        print(json.dumps({"profile_one_call": "backward " + wl.name, "status": int(rt.rt_get_status(ws.data_ptr()))}))
        return 0
    fwd_ms = timed(lambda: layer.prefill_device(x, z))
    assert layer.status() == rt.RT_OK
    bwd_ms = timed(bwd)
    rt.rt_profile_enable(True)
    rt.rt_profile_read()
    bwd(); torch.cuda.synchronize(dev)
    prof = rt.rt_profile_read()
    rt.rt_profile_enable(False)
    assert rt.rt_get_status(ws.data_ptr()) == rt.RT_OK and bool(torch.isfinite(dx).all())
    tok = wl.B * wl.N
    # products of the backward pass proper (twice the forward's) plus the recomputed forward products
    flops_fwd = 12.0 * tok * d * d + 4.0 * tok * d * f + 2.0 * wl.B * d * wl.N * (wl.N + 1)
    print(json.dumps({"backward_bench": wl.name, "B": wl.B, "N": wl.N, "d_model": d, "d_ff": f, "dtype": wl.dtype,
                      "alibi": bool(args.alibi), "forward_ms": fwd_ms, "backward_ms": bwd_ms,
                      "backward_tokens_per_s": tok / (bwd_ms * 1e-3), "backward_over_forward": bwd_ms / fwd_ms,
                      "us_per_position_reverse_loop": prof["leaf"]["ms"] * 1e3 / wl.N,
                      "gflop": 3.0 * flops_fwd / 1e9, "tflops": 3.0 * flops_fwd / (bwd_ms * 1e-3) / 1e12,
                      "arithmetic": "reverse loop and attention terms fp32 on CUDA cores; products over all rows on the tensor cores "
                                    "for bf16 storage",
                      "ms_by_phase": {"sweep_of_intermediates": prof["prepass"]["ms"], "reverse_loop_steps": prof["leaf"]["ms"],
                                      "reverse_loop_tiles": prof["tile"]["ms"], "products_over_all_rows": prof["other"]["ms"]},
                      "workspace_gb": ws.numel() / 1e9}))
    return 0


BASE_TILE_SEED = 20260421


def spawn_replicas(args):
    """`python bench.py --gpus N` without a launcher: start one replica process per GPU (the launch line the contract
    gives for N > 1) and pass rank 0's JSON line through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c4",
                    help="c4 (default: the 8-layer stack, the largest single-GPU configuration), c2, c3, c5_N<len>, p512")
    ap.add_argument("--also", default="c2,c3",
                    help="single-layer workloads also timed in the same process and reported under `also` ('' = none)")
    ap.add_argument("--sched", default="tiled", choices=["tiled", "naive"])
    ap.add_argument("--leaf", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (sweeps)")
    ap.add_argument("--profile-one-call", action="store_true",
                    help="run one call and exit (used under ncu to count DRAM / L2 bytes of a whole call)")
    ap.add_argument("--tile-bench", action="store_true", help="time Algorithm 2 alone per tile size and exit")
    ap.add_argument("--tile-bench-all", action="store_true", help="with --tile-bench: also sizes beyond N/2")
    ap.add_argument("--recur-block", type=int, default=0,
                    help="recurrence over blocks of this many positions (config.recur_block); 0 = the layer as defined")
    ap.add_argument("--alibi", action="store_true",
                    help="add ALiBi distances (slopes 2^(-8 h / H), h = 1..H) to the attention logits")
    ap.add_argument("--recompute-bench", action="store_true",
                    help="time rt_layer_recompute (parallel sweep given the outputs) and exit")
    ap.add_argument("--decode-bench", action="store_true", help="time rt_decode_step at several cache lengths and exit")
    ap.add_argument("--backward-bench", action="store_true", help="time rt_layer_backward next to the forward pass and exit")
    args = ap.parse_args()
    if args.tile_bench:
        return run_tile_bench(args)
    if args.decode_bench:
        return run_decode_bench(args)
    if args.recompute_bench:
        return run_recompute_bench(args)
    if args.backward_bench:
        return run_backward_bench(args)
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_replicas(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
